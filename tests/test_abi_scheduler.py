"""CPU-only: the library's Algorithm 1 entry points (nnv_simulate, nnv_schedule_queues, nnv_schedule)
agree with oracle/scheduler.py exactly on random integer cost tables."""
import numpy as np
import pytest

import workloads as wl
from oracle import scheduler as osch
from oracle import selection as osel
from paper_2206_07446_b200 import binding as nb
from test_abi_host import _plan, _random_costs

NETS = [wl.tiny_net, wl.cfg2_resnet18, wl.cfg3_mobilenetv2, wl.cfg5_vgg16, wl.cfg4_resnet50]


def _random_times(layers, rng, hi):
    n = len(layers)
    pl = [int(rng.integers(0, hi)) for _ in range(n)]
    pb = [int(p * int(rng.integers(30, 101)) // 100) for p in pl]
    ex = [int(rng.integers(0, hi)) for _ in range(n)]
    return pl, pb, ex


@pytest.mark.parametrize("seed", range(20))
def test_simulate_and_schedule_queues_match_oracle(seed):
    rng = np.random.default_rng(100 + seed)
    layers = NETS[seed % len(NETS)]()
    plan = _plan(layers)
    hi = [8, 1000, 10 ** 9][seed % 3]
    for m in (1, 2, 3, 7):
        pl, pb, ex = _random_times(layers, rng, hi)
        if seed % 4 == 0:                       # preparation-heavy: B grows
            pl = [p * 20 for p in pl]
        queue_of = [int(rng.integers(0, m + 1)) if L["op"] == wl.OP_CONV else -1 for L in layers]
        assert nb.nnv_simulate(plan, pl, pb, ex, queue_of, m) == osch.simulate(layers, pl, pb, ex, queue_of, m)
        for eps in (0, hi // 4):
            want_q, want_t = osch.schedule(layers, pl, pb, ex, m, eps)
            got_q, got_t = nb.nnv_schedule_queues(plan, pl, pb, ex, m, eps)
            assert got_q == want_q and got_t == want_t


def _oracle_search(layers, costs, allow, m, eps, big_pct, limit, pool):
    options = []
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            options.append(None)
            continue
        rows = [c for c in costs if c["layer"] == i]
        options.append(osel.pareto_filter(osel.options_from_costs(rows, allow)))
    return osch.search(layers, options, m, eps, big_pct=big_pct, exhaustive_limit=limit, pool_t=pool)


@pytest.mark.parametrize("seed", range(12))
def test_schedule_matches_oracle_search(seed):
    rng = np.random.default_rng(200 + seed)
    layers = [wl.tiny_net, wl.cfg1, wl.cfg2_resnet18][seed % 3]()
    plan = _plan(layers)
    costs = _random_costs(layers, rng, hi=[9, 500, 10 ** 6][seed % 3])
    if seed % 2:                                # make preparation dominate so that queue 0 takes some of it
        for c in costs:
            c["h2d_raw_ns"] *= 6
            c["h2d_cached_ns"] *= 6
    pool = [0 if L["op"] == wl.OP_CONV else int(rng.integers(0, 9)) for L in layers]
    for allow in (0, 1):
        for m, big_pct, limit in ((1, 100, 4096), (2, 60, 4096), (3, 100, 0)):
            if len(layers) > 8 and limit:       # exhaustive search only where the oracle finishes quickly
                limit = 64
            want = _oracle_search(layers, costs, allow, m, 0, big_pct, limit, pool)
            got = nb.nnv_schedule(plan, costs, allow, m, 0, big_pct, limit, pool)
            assert got[0] == want[0] and got[1] == want[1] and got[2] == want[2]


def test_schedule_never_worse_than_sequential_selection():
    """Scheduling the per-layer argmin combination on the queues cannot beat what nnv_schedule returns,
    and running everything on queue 0 (no pipelining) is an upper bound on both."""
    rng = np.random.default_rng(7)
    layers = wl.cfg2_resnet18()
    plan = _plan(layers)
    costs = _random_costs(layers, rng, hi=1000)
    choices, queue_of, t = nb.nnv_schedule(plan, costs, 1, 2, combo_limit=0)
    start = nb.nnv_select_kernels(plan, costs, 1)
    by_key = {}
    for c in costs:
        by_key[(c["layer"], c["variant"], c["math"], 0)] = (c["h2d_raw_ns"] + c["xform_ns"], c["exec_ns"])
        by_key[(c["layer"], c["variant"], c["math"], 1)] = (c["h2d_cached_ns"], c["exec_ns"])

    def times(ch):
        pl = [0 if c is None else by_key[(i,) + c][0] for i, c in enumerate(ch)]
        ex = [0 if c is None else by_key[(i,) + c][1] for i, c in enumerate(ch)]
        return pl, ex

    pl0, ex0 = times(start)
    _, t_start = nb.nnv_schedule_queues(plan, pl0, pl0, ex0, 2)
    assert t <= t_start <= sum(pl0) + sum(ex0)
    pl, ex = times(choices)
    assert nb.nnv_simulate(plan, pl, pl, ex, queue_of, 2) == t


def test_scheduler_argument_errors():
    layers = wl.tiny_net()
    plan = _plan(layers)
    n = len(layers)
    z = [1] * n
    with pytest.raises(nb.NnvError):
        nb.nnv_simulate(plan, z, z, z, [5] * n, 2)          # queue outside 0..n_little
    with pytest.raises(nb.NnvError):
        nb.nnv_schedule_queues(plan, z, z, z, 0)            # no little queue
    with pytest.raises(nb.NnvError):
        nb.nnv_schedule(plan, [], 1, 2)                     # no cost rows


# ---- shared host link, calibration, epsilon -----------------------------------------------------------
@pytest.mark.parametrize("seed", range(12))
def test_simulate_link_matches_oracle(seed):
    rng = np.random.default_rng(300 + seed)
    layers = NETS[seed % len(NETS)]()
    plan = _plan(layers)
    hi = [8, 1000, 10 ** 9][seed % 3]
    n = len(layers)
    for m in (1, 2, 3, 7):
        rd, xl, xb, ex = ([int(rng.integers(0, hi)) for _ in range(n)] for _ in range(4))
        queue_of = [int(rng.integers(0, m + 1)) if L["op"] == wl.OP_CONV else -1 for L in layers]
        assert nb.nnv_simulate_link(plan, rd, xl, xb, ex, queue_of, m) == osch.simulate_link(layers, rd, xl, xb, ex, queue_of, m)
        zero = [0] * n
        assert nb.nnv_simulate_link(plan, zero, xl, xb, ex, queue_of, m) == nb.nnv_simulate(plan, xl, xb, ex, queue_of, m)


@pytest.mark.parametrize("seed", range(8))
def test_schedule_link_matches_oracle_search(seed):
    rng = np.random.default_rng(400 + seed)
    layers = [wl.tiny_net, wl.cfg1, wl.cfg2_resnet18][seed % 3]()
    plan = _plan(layers)
    costs = _random_costs(layers, rng, hi=[9, 500, 10 ** 6][seed % 3])
    pool = [0 if L["op"] == wl.OP_CONV else int(rng.integers(0, 9)) for L in layers]
    read_of = {}
    for c in costs:
        read_of[(c["layer"], c["variant"], c["math"], 0)] = c["h2d_raw_ns"]
        read_of[(c["layer"], c["variant"], c["math"], 1)] = c["h2d_cached_ns"]
    for allow in (0, 1):
        for m, big_pct, limit in ((1, 100, 4096), (2, 60, 4096), (3, 100, 0)):
            if len(layers) > 8 and limit:
                limit = 64
            options = []
            for i, L in enumerate(layers):
                if L["op"] != wl.OP_CONV:
                    options.append(None)
                    continue
                surv = osel.pareto_filter(osel.options_from_costs([c for c in costs if c["layer"] == i], allow))
                options.append([(o[0], o[1], o[2], read_of[(i,) + tuple(o[0])]) for o in surv])
            want = osch.search(layers, options, m, 0, big_pct=big_pct, exhaustive_limit=limit, pool_t=pool, link=True)
            got = nb.nnv_schedule(plan, costs, allow, m, 0, big_pct, limit, pool, link=True)
            assert got[0] == want[0] and got[1] == want[1] and got[2] == want[2]


@pytest.mark.parametrize("seed", range(10))
def test_calibrate_and_eps_match_oracle(seed):
    rng = np.random.default_rng(500 + seed)
    layers = NETS[seed % len(NETS)]()
    plan = _plan(layers)
    hi = [9, 5000, 10 ** 9][seed % 3]
    costs = _random_costs(layers, rng, hi=hi)
    for allow in (0, 1):
        choices = nb.nnv_select_kernels(plan, costs, allow)
        tm = []
        for i, L in enumerate(layers):
            a, b, c = (int(rng.integers(0, hi)) for _ in range(3))
            tm.append(dict(h2d_start_ns=5, h2d_end_ns=5 + a, xform_start_ns=7, xform_end_ns=7 + (b if seed % 4 else 0),
                           exec_start_ns=9, exec_end_ns=9 + c))
        for kinds in (7, 6, 5, 0):
            want_rows, want_fac = osch.calibrate(costs, choices, tm, kinds=[bool(kinds & 1), bool(kinds & 2), bool(kinds & 4)])
            got_rows, got_fac = nb.nnv_calibrate_costs(plan, costs, choices, tm, kinds)
            assert got_fac == [tuple(f) for f in want_fac]
            assert got_rows == [{k: r[k] for k in got_rows[0]} for r in want_rows]
        iso = {(c["layer"], c["variant"], c["math"]): c for c in costs}
        for pct in (0, 1, 7, 100):
            ex = [iso[(i,) + ch[:2]]["exec_ns"] for i, ch in enumerate(choices) if ch is not None]
            assert nb.nnv_schedule_eps(plan, costs, allow, pct) == osch.schedule_eps(ex, pct)


def test_calibrate_errors():
    layers = wl.tiny_net()
    plan = _plan(layers)
    costs = _random_costs(layers, np.random.default_rng(1), hi=100)
    choices = nb.nnv_select_kernels(plan, costs, 0)
    tm = [dict(h2d_start_ns=0, h2d_end_ns=1, xform_start_ns=0, xform_end_ns=1, exec_start_ns=0, exec_end_ns=1) for _ in layers]
    conv = next(i for i, L in enumerate(layers) if L["op"] == wl.OP_CONV)
    with pytest.raises(nb.NnvError) as e:                   # the chosen kernel's row is missing
        nb.nnv_calibrate_costs(plan, [c for c in costs if c["layer"] != conv], choices, tm)
    assert e.value.status == 3
    bad = [dict(t) for t in tm]
    bad[conv]["exec_end_ns"], bad[conv]["exec_start_ns"] = 1, 5
    with pytest.raises(nb.NnvError):
        nb.nnv_calibrate_costs(plan, costs, choices, bad)
