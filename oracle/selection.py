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
        if allow_cached and has_transform(v):
            opts.append(((v, mth, 1), int(r["h2d_cached_ns"]), int(r["exec_ns"])))
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
