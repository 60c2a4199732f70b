"""Pins for oracle/selection.py (CPU only)."""
import itertools
import os

import numpy as np

from oracle import selection as sel

GOLD = os.path.join(os.path.dirname(__file__), "golden", "table2_costs.txt")


def _table2():
    rows = []
    for line in open(GOLD):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        name, rr, wt, rc, ex = line.split()
        rows.append((name, int(rr), int(wt), int(rc), int(ex)))
    return rows


def _table2_options(allow_cached):
    """Kernel i of the table gets variant id i; kernels with a zero transform have no cached arm."""
    opts = []
    for i, (name, rr, wt, rc, ex) in enumerate(_table2()):
        opts.append(((i, 0, 0), rr + wt, ex))
        if allow_cached and wt > 0:
            opts.append(((i, 0, 1), rc, ex))
    return opts


def test_table2_serial_cold_costs():
    """Sums of the paper's Table 2 columns (us): raw = read+transform+exec, cached = read cache+exec."""
    want_raw = {"3x3s1-winograd-pack4": 41910, "sgemm-pack4": 11050, "pack4": 21550,
                "3x3s1-winograd": 69740, "3x3s1": 8710, "general": 87820}
    want_cached = {"3x3s1-winograd-pack4": 8210, "sgemm-pack4": 8840, "pack4": 19330, "3x3s1-winograd": 7490}
    for name, rr, wt, rc, ex in _table2():
        assert rr + wt + ex == want_raw[name]
        if name in want_cached:
            assert rc + ex == want_cached[name]
    # the paper's text: sgemm-pack4 has a lower total cost than the default winograd-pack4 kernel
    assert want_raw["sgemm-pack4"] < want_raw["3x3s1-winograd-pack4"]


def test_table2_choice_and_pareto_set():
    names = [r[0] for r in _table2()]
    best = sel.choose(_table2_options(True))
    assert names[best[0][0]] == "3x3s1-winograd" and best[0][2] == 1 and best[1] + best[2] == 7490
    best_raw = sel.choose(_table2_options(False))
    assert names[best_raw[0][0]] == "3x3s1" and best_raw[0][2] == 0 and best_raw[1] + best_raw[2] == 8710
    surv = sel.pareto_filter(_table2_options(True))
    got = {(names[o[0][0]], o[0][2], o[1], o[2]) for o in surv}
    assert got == {("3x3s1-winograd-pack4", 1, 5230, 2980), ("3x3s1-winograd", 1, 4120, 3370), ("3x3s1", 0, 700, 8010)}


def test_brute_force_random_tables():
    """On small random integer tables: survivors are exactly the non-dominated options (lowest rank among
    duplicates), and the choice is the lexicographic minimum of (cost, rank) over ALL options."""
    rng = np.random.default_rng(11)
    for _ in range(300):
        n = int(rng.integers(1, 7))
        opts = []
        for i in range(n):
            opts.append(((int(rng.integers(0, 4)), int(rng.integers(0, 2)), int(rng.integers(0, 2)), i),
                         int(rng.integers(0, 6)), int(rng.integers(0, 6))))
        surv = sel.pareto_filter(opts)
        for o in opts:
            strictly = any((p[1] <= o[1] and p[2] <= o[2]) and (p[1] < o[1] or p[2] < o[2]) for p in opts)
            dup_lower = any(p[1] == o[1] and p[2] == o[2] and p[0] < o[0] for p in opts)
            assert (o in surv) == (not strictly and not dup_lower)
        best = sel.choose(opts)
        assert (best[1] + best[2], best[0]) == min((o[1] + o[2], o[0]) for o in opts)


def test_eligibility_rules():
    base = dict(op=0, C=64, K=64, R=3, S=3, stride=1, pad=1, groups=1)
    assert sel.eligible(base) == [sel.DIRECT, sel.IM2COL, sel.WINO_F2, sel.WINO_F4, sel.WINO_F6]
    assert sel.eligible(dict(base, stride=2)) == [sel.DIRECT, sel.IM2COL]
    assert sel.eligible(dict(base, R=1, S=1, pad=0)) == [sel.DIRECT, sel.IM2COL, sel.GEMM1X1]
    assert sel.eligible(dict(base, R=1, S=1, pad=0, stride=2)) == [sel.DIRECT, sel.IM2COL, sel.GEMM1X1]
    assert sel.eligible(dict(base, groups=64)) == [sel.DEPTHWISE]
    assert sel.eligible(dict(base, R=7, S=7, stride=2, pad=3, C=3)) == [sel.DIRECT, sel.IM2COL]
    assert sel.eligible(dict(base, groups=2)) == []


def test_select_kernels_over_layers():
    layers = [dict(op=0, C=8, K=8, R=3, S=3, stride=1, pad=1, groups=1),
              dict(op=1, C=8, K=8, R=2, S=2, stride=2, pad=0, groups=1),
              dict(op=0, C=8, K=8, R=3, S=3, stride=1, pad=1, groups=8)]
    costs = [dict(layer=0, variant=sel.DIRECT, math=sel.FP32, h2d_raw_ns=10, xform_ns=0, h2d_cached_ns=10, exec_ns=100),
             dict(layer=0, variant=sel.WINO_F2, math=sel.TF32, h2d_raw_ns=10, xform_ns=80, h2d_cached_ns=40, exec_ns=30),
             dict(layer=0, variant=sel.WINO_F2, math=sel.BF16, h2d_raw_ns=10, xform_ns=80, h2d_cached_ns=20, exec_ns=50),
             dict(layer=2, variant=sel.DEPTHWISE, math=sel.FP32, h2d_raw_ns=1, xform_ns=0, h2d_cached_ns=1, exec_ns=5)]
    assert sel.select_kernels(layers, costs, True) == [(sel.WINO_F2, sel.TF32, 1), None, (sel.DEPTHWISE, sel.FP32, 0)]
    assert sel.select_kernels(layers, costs, False) == [(sel.DIRECT, sel.FP32, 0), None, (sel.DEPTHWISE, sel.FP32, 0)]


def test_table2_warm_kernel_and_switch_set():
    """Table 2's execution column: the fastest-executing kernel is winograd-pack4 (2.98 ms), while the cold
    choice is the unpacked Winograd from the cache (7.49 ms) or, without caching, the untransformed 3x3s1
    kernel (8.71 ms): K_warm differs from K_cold in both modes, the situation Section 3.5 describes."""
    names = [r[0] for r in _table2()]
    rows = [dict(layer=0, variant=i, math=0, h2d_raw_ns=rr, xform_ns=wt, h2d_cached_ns=rc, exec_ns=ex)
            for i, (name, rr, wt, rc, ex) in enumerate(_table2())]
    v, m = sel.choose_warm(rows)
    assert names[v] == "3x3s1-winograd-pack4" and rows[v]["exec_ns"] == 2980
    assert min(r["exec_ns"] for r in rows) == 2980
    cold_cached = sel.choose(_table2_options(True))[0]
    cold_raw = sel.choose(_table2_options(False))[0]
    assert (cold_cached[0], cold_cached[1]) != (v, m) and (cold_raw[0], cold_raw[1]) != (v, m)


def test_warm_selection_and_switch_set_properties():
    """Brute force on random tables: K_warm minimises the summed execution time over all combinations;
    the switch set is empty iff the kernels agree (or the warm kernel has no transform)."""
    rng = np.random.default_rng(21)
    layer = dict(op=0, C=8, K=8, R=3, S=3, stride=1, pad=1, groups=1)
    kernels = [(sel.DIRECT, sel.FP32), (sel.IM2COL, sel.TF32), (sel.IM2COL, sel.BF16), (sel.WINO_F2, sel.TF32),
               (sel.WINO_F4, sel.TF32)]
    for _ in range(100):
        n = int(rng.integers(1, 4))
        layers = [layer] * n
        costs = []
        for i in range(n):
            for (v, m) in kernels:
                costs.append(dict(layer=i, variant=v, math=m, h2d_raw_ns=int(rng.integers(1, 9)),
                                  xform_ns=0 if v == sel.DIRECT else int(rng.integers(0, 9)),
                                  h2d_cached_ns=int(rng.integers(1, 9)), exec_ns=int(rng.integers(1, 6))))
        warm = sel.select_warm(layers, costs)
        ex = {(c["layer"], c["variant"], c["math"]): c["exec_ns"] for c in costs}
        total = sum(ex[(i, w[0], w[1])] for i, w in enumerate(warm))
        for combo in itertools.product(kernels, repeat=n):
            assert total <= sum(ex[(i, k[0], k[1])] for i, k in enumerate(combo))
        for i, w in enumerate(warm):                      # ties go to the lowest (variant, math)
            assert (w[0], w[1]) == min(k for k in kernels if ex[(i, k[0], k[1])] == ex[(i, w[0], w[1])])
            assert w[2] == (0 if w[0] == sel.DIRECT else 1)
        cold = sel.select_kernels(layers, costs, True)
        sw = sel.switch_set(cold, warm)
        for i in range(n):
            differs = (cold[i][0], cold[i][1]) != (warm[i][0], warm[i][1])
            assert (i in sw) == (differs and warm[i][0] != sel.DIRECT)
        assert sel.switch_set(warm, warm) == []


def test_third_arm_fused_read_and_transform():
    """The zero-copy arm (rank 2): offered only when allowed (bit 1) and profiled (zc_ns > 0), for kernels with a
    transform; it competes on prep = zc_ns.  Hand table: one layer, two kernels."""
    rows = [dict(variant=sel.IM2COL, math=sel.TF32, h2d_raw_ns=70, xform_ns=30, h2d_cached_ns=90, exec_ns=50, zc_ns=80),
            dict(variant=sel.DIRECT, math=sel.FP32, h2d_raw_ns=70, xform_ns=0, h2d_cached_ns=70, exec_ns=200, zc_ns=40)]
    ranks = lambda allow: [o[0] for o in sel.options_from_costs(rows, allow)]
    assert ranks(0) == [(sel.IM2COL, sel.TF32, 0), (sel.DIRECT, sel.FP32, 0)]
    assert ranks(1) == [(sel.IM2COL, sel.TF32, 0), (sel.IM2COL, sel.TF32, 1), (sel.DIRECT, sel.FP32, 0)]
    assert ranks(2) == [(sel.IM2COL, sel.TF32, 0), (sel.IM2COL, sel.TF32, 2), (sel.DIRECT, sel.FP32, 0)]   # DIRECT: no transform, no arm
    assert len(ranks(3)) == 4
    # raw: 70 + 30 + 50 = 150; cached: 90 + 50 = 140; fused: 80 + 50 = 130
    assert sel.choose(sel.options_from_costs(rows, 0))[0] == (sel.IM2COL, sel.TF32, 0)
    assert sel.choose(sel.options_from_costs(rows, 1))[0] == (sel.IM2COL, sel.TF32, 1)
    assert sel.choose(sel.options_from_costs(rows, 3))[0] == (sel.IM2COL, sel.TF32, 2)
    # the fused arm dominates the raw arm of its kernel (80 <= 100, same execution): the filter drops the raw one
    surv = [o[0] for o in sel.pareto_filter(sel.options_from_costs(rows, 2))]
    assert (sel.IM2COL, sel.TF32, 2) in surv and (sel.IM2COL, sel.TF32, 0) not in surv
    rows[0]["zc_ns"] = 0                                       # not profiled: not offered
    assert ranks(3) == ranks(1)
