"""CPU oracle: per-layer kernel eligibility and cold-cost selection (integers).

TEST INFRASTRUCTURE ONLY -- never imported by the product path.

Follows the paper's kernel-selection and transformation-bypass knobs (its
Sections 3.1.1 and 3.1.2, Table 2) and the candidate filter that opens its
Algorithm 1: a candidate is dropped when another one is at least as fast in
both preparation and execution and strictly faster in one.  For each kernel
(variant, math) there are two arms ("2 * c_i" combinations per operator in its
Section 3.3): read raw weights and transform them, or read the cached
post-transform weights and skip the transform.

    prep(raw)    = h2d_raw + xform
    prep(cached) = h2d_cached
    cold cost    = prep + exec                   (one layer, nothing overlapped)

All costs are unsigned integers (nanoseconds); every comparison is exact.
Ties are broken by the total order rank = (variant, math, cached).
"""

# variant ids (the enum order is the tie-break order)
DIRECT, IM2COL, GEMM1X1, DEPTHWISE, WINO_F2, WINO_F4, WINO_F6 = range(7)
FP32, TF32, BF16 = range(3)


def has_transform(variant):
    """DIRECT and DEPTHWISE consume raw weights: no transform, no cached arm."""
    return variant not in (DIRECT, DEPTHWISE)


def eligible(L):
    """Variants that can execute conv layer L (dict with C,K,R,S,stride,pad,groups)."""
    out = []
    dense = L["groups"] == 1
    if dense:
        out.append(DIRECT)
        out.append(IM2COL)
        if L["R"] == 1 and L["S"] == 1 and L["pad"] == 0:
            out.append(GEMM1X1)
    if L["groups"] == L["C"] and L["C"] == L["K"] and L["groups"] > 1:
        out.append(DEPTHWISE)
    if dense and L["R"] == 3 and L["S"] == 3 and L["stride"] == 1:
        out += [WINO_F2, WINO_F4, WINO_F6]
    return sorted(out)


def math_modes(variant):
    """Arithmetic modes a variant exists in."""
    if variant in (DIRECT, DEPTHWISE):
        return [FP32]
    if variant in (WINO_F4, WINO_F6):
        return [TF32]          # one bf16 pass in these Winograd domains misses the 1e-2 tolerance
    return [TF32, BF16]


def options_from_costs(rows, allow_cached):
    """rows: iterable of dicts (variant, math, h2d_raw_ns, xform_ns, h2d_cached_ns, exec_ns).

    Returns a list of (rank, prep, exec) with rank = (variant, math, cached).
    """
    opts = []
    for r in rows:
        v, mth = int(r["variant"]), int(r["math"])
        opts.append(((v, mth, 0), int(r["h2d_raw_ns"]) + int(r["xform_ns"]), int(r["exec_ns"])))
        if (int(allow_cached) & 1) and has_transform(v):
            opts.append(((v, mth, 1), int(r["h2d_cached_ns"]), int(r["exec_ns"])))
        # third arm (bit 1 of allow_cached): read and transform fused into one operation whose time is zc_ns
        if (int(allow_cached) & 2) and has_transform(v) and int(r.get("zc_ns", 0)) > 0:
            opts.append(((v, mth, 2), int(r["zc_ns"]), int(r["exec_ns"])))
    return opts


def pareto_filter(opts):
    """Keep options not dominated in (prep, exec); of exact duplicates keep the lowest rank."""
    keep = []
    for o in opts:
        dominated = False
        for p in opts:
            if p is o:
                continue
            if p[1] <= o[1] and p[2] <= o[2]:
                if p[1] < o[1] or p[2] < o[2]:
                    dominated = True
                elif p[0] < o[0]:                 # exact duplicate with a lower rank
                    dominated = True
            if dominated:
                break
        if not dominated:
            keep.append(o)
    return sorted(keep)


def choose(opts):
    """argmin of prep + exec over the Pareto survivors; ties -> lowest rank."""
    surv = pareto_filter(opts)
    best = None
    for o in surv:                                # surv is sorted by rank
        if best is None or o[1] + o[2] < best[1] + best[2]:
            best = o
    return best


def select_kernels(layers, costs, allow_cached):
    """Per conv layer, the chosen (variant, math, cached); None for non-conv layers.

    costs: list of dicts with key 'layer' plus the cost fields.
    """
    out = []
    for i, L in enumerate(layers):
        if L["op"] != 0:
            out.append(None)
            continue
        rows = [r for r in costs if int(r["layer"]) == i]
        el = eligible(L)
        for r in rows:
            if int(r["variant"]) not in el or int(r["math"]) not in math_modes(int(r["variant"])):
                raise ValueError("cost row for a kernel the layer cannot use")
        if not rows:
            raise ValueError("no cost rows for layer %d" % i)
        out.append(choose(options_from_costs(rows, allow_cached))[0])
    return out


def choose_warm(rows):
    """Of one layer's cost rows, the kernel with the least execution time; ties -> lowest (variant, math).

    Warm inference has every weight prepared already, so only the execution column counts: this is
    the paper's K_warm (its Section 3.5, "the kernels with the fastest warm inference")."""
    best = None
    for r in sorted(rows, key=lambda r: (int(r["variant"]), int(r["math"]))):
        if best is None or int(r["exec_ns"]) < int(best["exec_ns"]):
            best = r
    return (int(best["variant"]), int(best["math"]))


def select_warm(layers, costs):
    """K_warm per conv layer as (variant, math, prepared): prepared = 1 when the kernel reads
    transformed weights (they stay resident after the first inference), 0 when it reads raw ones."""
    out = []
    for i, L in enumerate(layers):
        if L["op"] != 0:
            out.append(None)
            continue
        rows = [r for r in costs if int(r["layer"]) == i]
        if not rows:
            raise ValueError("no cost rows for layer %d" % i)
        v, m = choose_warm(rows)
        out.append((v, m, 1 if has_transform(v) else 0))
    return out


def switch_set(k_cold, k_warm):
    """Layers of K_warm - K_cold (Section 3.5): their warm kernel differs from the cold one, so its
    weights are still to be prepared (read, transformed) while or after the cold inference runs.
    A warm kernel without a transform needs no preparation beyond the raw weights."""
    out = []
    for i, (c, w) in enumerate(zip(k_cold, k_warm)):
        if c is None or w is None:
            continue
        if (c[0], c[1]) != (w[0], w[1]) and has_transform(w[0]):
            out.append(i)
    return out
