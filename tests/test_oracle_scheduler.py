"""Pins for oracle/scheduler.py (CPU only): the makespan simulator and the Algorithm 1 heuristic."""
import itertools

import numpy as np

from oracle import scheduler as sch


def _chain(n):
    return [dict(op=0, in0=i - 1, in1=-1) for i in range(n)]


def _tick_simulator(layers, pl, pb, ex, queue_of, n_little):
    """Independent check (all durations >= 1): advance time one unit at a time; every queue works on the
    first unfinished operation of its list if that operation's precursors ended by now (Eq. (2):
    precursors first, one operation per queue at a time)."""
    n = len(layers)
    lists = [[] for _ in range(n_little + 1)]
    for i in range(n):
        if layers[i]["op"] == 0 and queue_of[i] == 0:
            lists[0].append(("p", i))
        lists[0].append(("e", i))
        if layers[i]["op"] == 0 and queue_of[i] > 0:
            lists[queue_of[i]].append(("p", i))
    left = {("e", i): ex[i] for i in range(n)}
    left.update({("p", i): (pb[i] if queue_of[i] == 0 else pl[i]) for i in range(n) if layers[i]["op"] == 0})
    done_at = {}

    def deps(op):
        kind, i = op
        if kind == "p":
            return []
        d = [("p", i)] if layers[i]["op"] == 0 else []
        return d + [("e", s) for s in (layers[i]["in0"], layers[i]["in1"]) if s >= 0]

    t = 0
    while ("e", n - 1) not in done_at:
        running = []
        for q in range(n_little + 1):
            todo = [op for op in lists[q] if op not in done_at]
            if todo and all(d in done_at and done_at[d] <= t for d in deps(todo[0])):
                running.append(todo[0])
        for op in running:
            left[op] -= 1
            if left[op] == 0:
                done_at[op] = t + 1
        t += 1
        assert t < 10000
    return done_at[("e", n - 1)]


def test_simulate_hand_examples():
    L = _chain(3)
    assert sch.simulate(_chain(1), [7], [4], [3], [0], 1) == 7                      # p_big + e
    assert sch.simulate(L, [9, 9, 9], [2, 3, 4], [5, 6, 7], [0, 0, 0], 1) == 27     # everything on queue 0
    assert sch.simulate(L, [5, 4, 4], [5, 9, 9], [3, 3, 3], [0, 1, 1], 1) == 14     # execution-bound
    assert sch.simulate(L, [1, 10, 10], [1, 1, 1], [1, 1, 1], [0, 1, 1], 1) == 21   # preparation-bound
    assert sch.simulate(L, [1, 10, 10], [1, 1, 1], [1, 1, 1], [0, 1, 2], 2) == 12   # two little queues
    # a residual edge: layer 2 also waits for layer 0's execution (already implied here) and a pool in between
    D = [dict(op=0, in0=-1, in1=-1), dict(op=1, in0=0, in1=-1), dict(op=0, in0=1, in1=0)]
    assert sch.simulate(D, [2, 0, 3], [2, 0, 3], [4, 1, 5], [0, -1, 1], 1) == 12    # 2+4, pool 1, then 5


def test_simulate_matches_independent_tick_simulator():
    rng = np.random.default_rng(3)
    for _ in range(300):
        n = int(rng.integers(1, 7))
        layers = []
        for i in range(n):
            op = 0 if (i == 0 or rng.random() < 0.8) else 1
            in1 = int(rng.integers(-1, i)) if (i > 1 and op == 0 and rng.random() < 0.3) else -1
            layers.append(dict(op=op, in0=i - 1, in1=in1))
        m = int(rng.integers(1, 4))
        pl = [int(rng.integers(1, 7)) for _ in range(n)]
        pb = [int(rng.integers(1, 7)) for _ in range(n)]
        ex = [int(rng.integers(1, 7)) for _ in range(n)]
        q = [int(rng.integers(0, m + 1)) if layers[i]["op"] == 0 else -1 for i in range(n)]
        assert sch.simulate(layers, pl, pb, ex, q, m) == _tick_simulator(layers, pl, pb, ex, q, m)


def test_balance_little_reaches_its_fixed_point():
    rng = np.random.default_rng(4)
    for _ in range(200):
        n = int(rng.integers(1, 12))
        m = int(rng.integers(1, 5))
        eps = int(rng.integers(0, 4))
        items = [(i, int(rng.integers(0, 20))) for i in range(n)]
        a = sch.balance_little(items, m, eps)
        assert sorted(a) == list(range(n)) and all(1 <= q <= m for q in a.values())
        tot = [sum(t for i, t in items if a[i] == q) for q in range(1, m + 1)]
        gap = max(tot) - min(tot)
        if gap > eps:                                   # stopped because no operation of a longest queue may move
            jmax = tot.index(max(tot)) + 1
            assert all(2 * t >= gap for i, t in items if a[i] == jmax)
    assert sch.balance_little([(0, 5), (1, 5), (2, 5), (3, 5)], 2, 0) == {0: 1, 2: 1, 1: 2, 3: 2}
    # round-robin gives [10,1 | 1]; the 1 moves from the long queue (2*1 < 9), the 10 cannot (20 >= 9)
    assert sch.balance_little([(0, 10), (1, 1), (2, 1)], 2, 0) == {0: 1, 1: 2, 2: 2}


def test_schedule_hand_examples():
    L = _chain(3)
    q, t = sch.schedule(L, [2, 10, 10], [1, 3, 3], [5, 5, 5], 1, 0)
    assert q == [0, 1, 1] and t == 25                   # gap 4: no layer has t_big + t_little < 4
    q, t = sch.schedule(L, [2, 6, 30], [1, 1, 5], [5, 5, 5], 1, 0)
    assert q == [0, 0, 1] and t == 35                   # layer 1 moves to queue 0 (7 < 20), layer 2 cannot (35 >= 13)
    q, t = sch.schedule(L, [1, 1, 1], [1, 1, 1], [9, 9, 9], 2, 0)
    assert q[0] == 0 and t == 28                        # execution-bound: p_1 + all executions


def test_schedule_properties_and_brute_force_bound():
    rng = np.random.default_rng(5)
    for _ in range(150):
        n = int(rng.integers(1, 6))
        L = _chain(n)
        m = int(rng.integers(1, 3))
        pl = [int(rng.integers(0, 30)) for _ in range(n)]
        pb = [max(0, p - int(rng.integers(0, 5))) for p in pl]
        ex = [int(rng.integers(1, 15)) for _ in range(n)]
        q, t = sch.schedule(L, pl, pb, ex, m, 0)
        assert q[0] == 0 and all(0 <= v <= m for v in q)
        assert t == sch.simulate(L, pl, pb, ex, q, m)
        best = min(sch.simulate(L, pl, pb, ex, [0] + list(rest), m)
                   for rest in itertools.product(range(m + 1), repeat=n - 1))
        assert best <= t                                # the heuristic never beats the exhaustive optimum
        assert t >= pb[0] + sum(ex)                     # queue 0 runs p_1 and every execution


def test_search_exhaustive_and_descent():
    rng = np.random.default_rng(6)
    for _ in range(40):
        n = int(rng.integers(1, 5))
        L = _chain(n)
        options = [[((v, 0, 0), int(rng.integers(0, 40)), int(rng.integers(1, 40))) for v in range(int(rng.integers(1, 4)))]
                   for _ in range(n)]
        ranks, q, t = sch.search(L, options, 2, 0)
        # exhaustive: no single combination does better
        for combo in itertools.product(*[range(len(o)) for o in options]):
            pl = [options[i][c][1] for i, c in enumerate(combo)]
            ex = [options[i][c][2] for i, c in enumerate(combo)]
            assert sch.schedule(L, pl, pl, ex, 2, 0)[1] >= t
        # forced coordinate descent ends no worse than where it starts, and no better than the exhaustive optimum
        r2, q2, t2 = sch.search(L, options, 2, 0, exhaustive_limit=0)
        start = [min(range(len(o)), key=lambda c: (o[c][1] + o[c][2], c)) for o in options]
        t0 = sch.schedule(L, [options[i][c][1] for i, c in enumerate(start)], [options[i][c][1] for i, c in enumerate(start)],
                          [options[i][c][2] for i, c in enumerate(start)], 2, 0)[1]
        assert t <= t2 <= t0


# ---- one shared host link ------------------------------------------------------------------------------
def _tick_simulator_link(layers, rd, xl, xb, ex, queue_of, n_little):
    """Independent check of simulate_link (all durations >= 1): unit time steps; a queue works on the first
    unfinished operation of its list; a read additionally needs the link, which goes to the waiting read of the
    lowest layer and stays with it until that read is finished."""
    n = len(layers)
    lists = [[] for _ in range(n_little + 1)]
    for i in range(n):
        if layers[i]["op"] == 0 and queue_of[i] == 0:
            lists[0] += [("r", i), ("x", i)]
        lists[0].append(("e", i))
        if layers[i]["op"] == 0 and queue_of[i] > 0:
            lists[queue_of[i]] += [("r", i), ("x", i)]
    left = {("e", i): ex[i] for i in range(n)}
    for i in range(n):
        if layers[i]["op"] == 0:
            left[("r", i)] = rd[i]
            left[("x", i)] = xb[i] if queue_of[i] == 0 else xl[i]
    done_at = {}
    link_owner = None

    def deps(op):
        kind, i = op
        if kind == "r":
            return []
        if kind == "x":
            return [("r", i)]
        d = [("x", i)] if layers[i]["op"] == 0 else []
        return d + [("e", s) for s in (layers[i]["in0"], layers[i]["in1"]) if s >= 0]

    t = 0
    while ("e", n - 1) not in done_at:
        heads = []
        for q in range(n_little + 1):
            todo = [op for op in lists[q] if op not in done_at]
            if todo and all(d in done_at and done_at[d] <= t for d in deps(todo[0])):
                heads.append(todo[0])
        if link_owner is None:
            reads = sorted(op[1] for op in heads if op[0] == "r")
            if reads:
                link_owner = ("r", reads[0])
        for op in heads:
            if op[0] == "r" and op != link_owner:
                continue
            left[op] -= 1
            if left[op] == 0:
                done_at[op] = t + 1
                if op == link_owner:
                    link_owner = None
        t += 1
        assert t < 20000
    return done_at[("e", n - 1)]


def test_simulate_link_hand_examples():
    L = _chain(3)
    # one little queue, everything on it: the link never has two reads waiting, so read + transform behave as one bundle
    assert sch.simulate_link(L, [2, 3, 4], [1, 1, 1], [9, 9, 9], [1, 1, 1], [1, 1, 1], 1) == \
        sch.simulate(L, [3, 4, 5], [9, 9, 9], [1, 1, 1], [1, 1, 1], 1) == 13
    # two little queues: reads 10 and 10 serialise on the link (ends 10 and 20), where separate links would end both at 10
    assert sch.simulate(L, [1, 11, 11], [1, 1, 1], [1, 1, 1], [0, 1, 2], 2) == 13
    assert sch.simulate_link(L, [1, 10, 10], [0, 1, 1], [0, 1, 1], [1, 1, 1], [0, 1, 2], 2) == 23
    # the lower layer's read goes first when both wait: layer 1 (queue 2) before layer 2 (queue 1)
    assert sch.simulate_link(L, [1, 5, 7], [0, 0, 0], [0, 0, 0], [1, 1, 1], [0, 2, 1], 2) == 14
    # no reads at all: the plain makespan
    assert sch.simulate_link(L, [0, 0, 0], [5, 4, 4], [5, 9, 9], [3, 3, 3], [0, 1, 1], 1) == 14


def test_simulate_link_matches_independent_tick_simulator():
    rng = np.random.default_rng(13)
    for _ in range(300):
        n = int(rng.integers(1, 7))
        layers = []
        for i in range(n):
            op = 0 if (i == 0 or rng.random() < 0.8) else 1
            in1 = int(rng.integers(-1, i)) if (i > 1 and op == 0 and rng.random() < 0.3) else -1
            layers.append(dict(op=op, in0=i - 1, in1=in1))
        m = int(rng.integers(1, 4))
        rd, xl, xb, ex = ([int(rng.integers(1, 7)) for _ in range(n)] for _ in range(4))
        q = [int(rng.integers(0, m + 1)) if layers[i]["op"] == 0 else -1 for i in range(n)]
        assert sch.simulate_link(layers, rd, xl, xb, ex, q, m) == _tick_simulator_link(layers, rd, xl, xb, ex, q, m)
        # a shared link can only delay: never below the model with a link per queue
        pl = [rd[i] + xl[i] for i in range(n)]
        pb = [rd[i] + xb[i] for i in range(n)]
        assert sch.simulate_link(layers, rd, xl, xb, ex, q, m) >= sch.simulate(layers, pl, pb, ex, q, m)


def test_calibrate_hand_table():
    rows = [dict(layer=0, variant=1, math=1, h2d_raw_ns=100, xform_ns=40, h2d_cached_ns=300, exec_ns=50),
            dict(layer=0, variant=4, math=1, h2d_raw_ns=100, xform_ns=90, h2d_cached_ns=500, exec_ns=20),
            dict(layer=1, variant=0, math=0, h2d_raw_ns=10, xform_ns=0, h2d_cached_ns=10, exec_ns=70),
            dict(layer=2, variant=1, math=1, h2d_raw_ns=200, xform_ns=60, h2d_cached_ns=700, exec_ns=30)]
    choices = [(1, 1, 0), (0, 0, 0), (1, 1, 1)]
    tm = [dict(h2d_start_ns=0, h2d_end_ns=150, xform_start_ns=150, xform_end_ns=210, exec_start_ns=210, exec_end_ns=300),
          dict(h2d_start_ns=150, h2d_end_ns=165, xform_start_ns=0, xform_end_ns=0, exec_start_ns=300, exec_end_ns=370),
          dict(h2d_start_ns=165, h2d_end_ns=1065, xform_start_ns=0, xform_end_ns=0, exec_start_ns=1065, exec_end_ns=1100)]
    out, fac = sch.calibrate(rows, choices, tm)
    # read: (150 + 15 + 900) / (100 + 10 + 700) = 1065/810; transform: 60/40 (layer 2 read cached weights, layer 1 has none);
    # execution: (90 + 70 + 35) / (50 + 70 + 30) = 195/150
    assert fac == [(1065, 810), (60, 40), (195, 150)]
    assert [r["h2d_raw_ns"] for r in out] == [100 * 1065 // 810, 100 * 1065 // 810, 10 * 1065 // 810, 200 * 1065 // 810]
    assert [r["h2d_cached_ns"] for r in out] == [300 * 1065 // 810, 500 * 1065 // 810, 10 * 1065 // 810, 700 * 1065 // 810]
    assert [r["xform_ns"] for r in out] == [60, 135, 0, 90]
    assert [r["exec_ns"] for r in out] == [65, 26, 91, 39]
    # a kind switched off keeps its isolated costs, the others are scaled as before
    out6, fac6 = sch.calibrate(rows, choices, tm, kinds=(False, True, True))
    assert [r["h2d_raw_ns"] for r in out6] == [100, 100, 10, 200] and [r["exec_ns"] for r in out6] == [65, 26, 91, 39] and fac6 == fac
    # a run that measured nothing of a kind leaves that kind alone (no division by zero, no zeroed table)
    tm0 = [dict(t, xform_start_ns=0, xform_end_ns=0) for t in tm]
    out0, fac0 = sch.calibrate(rows, choices, tm0)
    assert [r["xform_ns"] for r in out0] == [40, 90, 0, 60] and fac0[1] == (0, 40)
    # the measured run equal to the isolated profile is a fixed point
    same = [dict(h2d_start_ns=0, h2d_end_ns=100, xform_start_ns=0, xform_end_ns=40, exec_start_ns=0, exec_end_ns=50),
            dict(h2d_start_ns=0, h2d_end_ns=10, xform_start_ns=0, xform_end_ns=0, exec_start_ns=0, exec_end_ns=70),
            dict(h2d_start_ns=0, h2d_end_ns=700, xform_start_ns=0, xform_end_ns=0, exec_start_ns=0, exec_end_ns=30)]
    assert sch.calibrate(rows, choices, same)[0] == rows
    assert sch.schedule_eps([50, 70, 30], 1) == 1 and sch.schedule_eps([50, 70, 30], 10) == 15
