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
