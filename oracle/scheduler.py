"""CPU oracle: the paper's heuristic kernel scheduler (its Algorithm 1) and the makespan it minimises.

TEST INFRASTRUCTURE ONLY -- never imported by the product path.

Model (the paper's Section 3.2, Eq. (1)-(2), and the assumptions of Section 3.3).  Every layer i has a
bundled preparation operation p_i (read + transform of its weights, or read of the cached weights) and an
execution operation e_i.  Queue 0 ("big cores"; here: the execution stream) runs every e_i in layer order
and the preparation of the layers in the set B; queues 1..M ("little cores"; here: preparation streams)
run the remaining preparations.  A queue runs one operation at a time, in its listed order; an operation
starts when its queue is free and its precursors have ended: e_i needs p_i and the executions of the
layers that produce its inputs.  The cold latency is the end of the last execution.

All times are unsigned integers (nanoseconds); every comparison is exact.

Reading of Algorithm 1 used here (the listing is ambiguous about which statements the outer while encloses
and about the bookkeeping of s; this is the reading, in the listing's order):
  start      B = {first conv layer}; queue 0 = p_1 and all executions.
  spread     the preparations not in B go to queues 1..M round-robin in layer order.
  balance    while max - min of the little-queue totals exceeds eps: sort the longest queue's operations
             by time, descending, and move to the shortest queue every operation whose time is below half
             the current gap, updating the totals after each move; stop when a pass moves nothing.
  grow B     while the longest little queue exceeds queue 0's total by more than eps: take the first layer
             (in layer order) not in B with t_big + t_little < gap, add it to B, and redo spread and
             balance; stop when no layer qualifies.
  result     T_cold = makespan of the resulting queues.
Within queue 0 a layer's preparation sits directly before its execution; little queues keep layer order.
"""


def simulate(layers, prep_little, prep_big, exec_t, queue_of, n_little):
    """Makespan (end of the last execution) of one assignment.

    layers: list of dicts with 'op', 'in0', 'in1' (op 0 = conv; others have no preparation).
    prep_little / prep_big / exec_t: per-layer integer times (prep entries of non-conv layers are ignored).
    queue_of: per-layer queue of the preparation: 0 = queue 0, 1..n_little = little queue; -1 for non-conv.
    """
    n = len(layers)
    free = [0] * (n_little + 1)
    prep_end = [0] * n
    exec_end = [0] * n
    # little queues: layer order
    for q in range(1, n_little + 1):
        for i in range(n):
            if layers[i]["op"] == 0 and queue_of[i] == q:
                start = free[q]
                prep_end[i] = start + prep_little[i]
                free[q] = prep_end[i]
    for i in range(n):
        if layers[i]["op"] == 0 and queue_of[i] == 0:
            start = free[0]
            prep_end[i] = start + prep_big[i]
            free[0] = prep_end[i]
        ready = free[0]
        if layers[i]["op"] == 0:
            ready = max(ready, prep_end[i])
        for src in (layers[i]["in0"], layers[i]["in1"]):
            if src >= 0:
                ready = max(ready, exec_end[src])
        exec_end[i] = ready + exec_t[i]
        free[0] = exec_end[i]
    return exec_end[n - 1]


def balance_little(items, n_little, eps):
    """The spread and balance steps: round-robin start, then move operations from the longest to the shortest queue.

    items: list of (layer, time) in layer order.  Returns {layer: queue in 1..n_little}.
    """
    queues = [[] for _ in range(n_little)]
    for k, it in enumerate(items):
        queues[k % n_little].append(it)
    tot = [sum(t for _, t in q) for q in queues]
    while max(tot) - min(tot) > eps:
        jmax = max(range(n_little), key=lambda j: (tot[j], -j))      # ties: lowest index
        jmin = min(range(n_little), key=lambda j: (tot[j], j))
        moved = False
        for it in sorted(queues[jmax], key=lambda it: (-it[1], it[0])):
            if 2 * it[1] < tot[jmax] - tot[jmin]:
                queues[jmax].remove(it)
                queues[jmin].append(it)
                tot[jmax] -= it[1]
                tot[jmin] += it[1]
                moved = True
        if not moved:
            break
    out = {}
    for j, q in enumerate(queues):
        for layer, _ in q:
            out[layer] = j + 1
    return out


def schedule(layers, prep_little, prep_big, exec_t, n_little, eps):
    """The inner part of Algorithm 1 for one kernel combination.  Returns (queue_of, T_cold)."""
    n = len(layers)
    conv = [i for i in range(n) if layers[i]["op"] == 0]
    B = {conv[0]}
    while True:
        rest = [(i, prep_little[i]) for i in conv if i not in B]
        assign = balance_little(rest, n_little, eps) if rest else {}
        tot_little = [0] * (n_little + 1)
        for i, q in assign.items():
            tot_little[q] += prep_little[i]
        t_little = max(tot_little)
        t0 = sum(prep_big[i] for i in B) + sum(exec_t)
        if t_little <= t0 + eps:
            break
        gap = t_little - t0
        pick = None
        for i in conv:
            if i not in B and prep_big[i] + prep_little[i] < gap:
                pick = i
                break
        if pick is None:
            break
        B.add(pick)
    queue_of = [-1] * n
    for i in conv:
        queue_of[i] = 0 if i in B else assign[i]
    return queue_of, simulate(layers, prep_little, prep_big, exec_t, queue_of, n_little)


def option_times(opt, big_pct):
    """(prep_little, prep_big, exec) of one option (rank, prep, exec); the big queue runs a preparation in
    big_pct percent of the little-queue time (integer arithmetic, rounded down)."""
    return opt[1], opt[1] * big_pct // 100, opt[2]


def search(layers, options, n_little, eps, big_pct=100, exhaustive_limit=4096, pool_t=None, link=False):
    """The outer loop of Algorithm 1 over the filtered candidates.

    With link=True every option is (rank, prep, exec, read) -- read is the part of prep that crosses the host
    link -- the queues still come from schedule() on the bundled times, but the latency that is compared and
    returned is simulate_link()'s (transform on queue 0 = (prep - read) * big_pct // 100).

    options: per layer, the list of surviving (rank, prep, exec) options in rank order (None for non-conv
    layers; pool_t gives their execution time).  With at most `exhaustive_limit` combinations every one is
    scheduled; otherwise coordinate descent from the per-layer cold-cost minimum: sweep the layers in
    order, adopt the first option (in rank order) that strictly lowers T_cold, repeat until a sweep
    changes nothing (at most 8 sweeps).  Ties keep the earlier combination.
    Returns (chosen rank per layer, queue_of, T_cold).
    """
    n = len(layers)
    conv = [i for i in range(n) if layers[i]["op"] == 0]

    def evaluate(pick):
        pl, pb, ex = [0] * n, [0] * n, [0] * n
        for i in range(n):
            if layers[i]["op"] == 0:
                pl[i], pb[i], ex[i] = option_times(options[i][pick[i]], big_pct)
            else:
                ex[i] = pool_t[i] if pool_t else 0
        q, t = schedule(layers, pl, pb, ex, n_little, eps)
        if link:
            rd = [options[i][pick[i]][3] if layers[i]["op"] == 0 else 0 for i in range(n)]
            xl = [pl[i] - rd[i] for i in range(n)]
            xb = [xl[i] * big_pct // 100 for i in range(n)]
            t = simulate_link(layers, rd, xl, xb, ex, q, n_little)
        return t, q

    total = 1
    for i in conv:
        total *= len(options[i])
        if total > exhaustive_limit:
            break
    best_pick, best_t, best_q = None, None, None
    if total <= exhaustive_limit:
        import itertools
        for combo in itertools.product(*[range(len(options[i])) for i in conv]):
            pick = [0] * n
            for i, c in zip(conv, combo):
                pick[i] = c
            t, q = evaluate(pick)
            if best_t is None or t < best_t:
                best_pick, best_t, best_q = pick, t, q
    else:
        pick = [0] * n
        for i in conv:
            pick[i] = min(range(len(options[i])), key=lambda c: (options[i][c][1] + options[i][c][2], c))
        best_t, best_q = evaluate(pick)
        best_pick = pick
        for _ in range(8):
            changed = False
            for i in conv:
                for c in range(len(options[i])):
                    if c == best_pick[i]:
                        continue
                    trial = list(best_pick)
                    trial[i] = c
                    t, q = evaluate(trial)
                    if t < best_t:
                        best_pick, best_t, best_q = trial, t, q
                        changed = True
                        break
            if not changed:
                break
    ranks = [options[i][best_pick[i]][0] if layers[i]["op"] == 0 else None for i in range(n)]
    return ranks, best_q, best_t


# ---- one host link shared by every queue's reads ------------------------------------------------------
def simulate_link(layers, read_t, xf_little, xf_big, exec_t, queue_of, n_little):
    """Makespan when the reads of ALL queues pass through one link (a reading of the model for a machine
    where every queue's weights arrive over the same host link: Eq. (1)-(2) give each queue its own
    processor for the whole bundled preparation; here only the transform part runs on the queue alone).

    A preparation is now two operations on its queue, read then transform.  The link carries one read at a
    time; a read is waiting from the moment the operation before it on its queue has ended; whenever the
    link is free it takes, among the waiting reads, the one of the lowest layer (the order the reads were
    issued in); a read occupies its queue and the link for read_t.  Everything else is as in simulate():
    queue 0 runs, in layer order, [read, transform] of its own layers directly before their execution and
    every execution; queues 1..n_little run their layers' [read, transform] in layer order; an execution
    needs its transform and the executions of its producers.  Times are integers; returns the end of the
    last execution.
    """
    n = len(layers)
    conv = [layers[i]["op"] == 0 for i in range(n)]
    ops = [[] for _ in range(n_little + 1)]                    # per queue: (kind, layer, duration)
    for i in range(n):
        if conv[i] and queue_of[i] == 0:
            ops[0].append(("r", i, read_t[i]))
            ops[0].append(("x", i, xf_big[i]))
        ops[0].append(("e", i, exec_t[i]))
        if conv[i] and queue_of[i] > 0:
            ops[queue_of[i]].append(("r", i, read_t[i]))
            ops[queue_of[i]].append(("x", i, xf_little[i]))
    head = [0] * (n_little + 1)                                # index of the next operation to start
    busy_until = [0] * (n_little + 1)                          # end of the operation that was started last
    end = {}                                                   # (kind, layer) -> end time, once started
    link_free = 0
    t = 0
    while ("e", n - 1) not in end:
        progressed = True
        while progressed:                                      # start everything that can start at time t
            progressed = False
            waiting = []
            for q in range(n_little + 1):
                if head[q] >= len(ops[q]) or busy_until[q] > t:
                    continue
                kind, i, dur = ops[q][head[q]]
                if kind == "r":
                    waiting.append((i, q, dur))
                    continue
                deps = [("r", i)] if kind == "x" else ([("x", i)] if conv[i] else []) + \
                    [("e", s) for s in (layers[i]["in0"], layers[i]["in1"]) if s >= 0]
                if all(d in end and end[d] <= t for d in deps):
                    end[(kind, i)] = t + dur
                    busy_until[q] = t + dur
                    head[q] += 1
                    progressed = True
            if waiting and link_free <= t:
                i, q, dur = min(waiting)
                end[("r", i)] = t + dur
                busy_until[q] = t + dur
                link_free = t + dur
                head[q] += 1
                progressed = True
        later = [v for v in list(end.values()) + [link_free] if v > t]
        if ("e", n - 1) in end:
            break
        t = min(later)
    return end[("e", n - 1)]


def calibrate(rows, choices, timings, kinds=(True, True, True)):
    """The re-profiling step of Algorithm 1 (its profiling of operations happens with the other queues
    busy; Section 3.3's remark on interference): scale the isolated cost table by how much slower each KIND
    of operation ran in a run of the schedule than it did alone.

    rows: cost rows as dicts (layer, variant, math, h2d_raw_ns, xform_ns, h2d_cached_ns, exec_ns).
    choices: per layer (variant, math, cached) or None.  timings: per layer dict with h2d/xform/exec start and
    end stamps of that run.  For kind k in (read, transform, execution): num_k = sum over the chosen kernels
    of the measured interval, den_k = sum of their isolated costs (read: the cached or the raw read, whichever
    the choice made; transform: only where the choice transformed).  Every row's costs of kind k become
    floor(cost * num_k / den_k); a kind with num_k = 0 or den_k = 0 stays as it is, and so does a kind whose
    entry in `kinds` (read, transform, execution) is False -- under the shared-link model the reads' waiting for
    one another is what simulate_link() itself accounts for, so their measured intervals must not be fed back.
    Returns (new rows, [(num, den) for read, transform, execution]).
    """
    iso = {(r["layer"], r["variant"], r["math"]): r for r in rows}
    num = [0, 0, 0]
    den = [0, 0, 0]
    for i, ch in enumerate(choices):
        if ch is None:
            continue
        r, t = iso[(i, ch[0], ch[1])], timings[i]
        has_xf = ch[0] not in (0, 3)                           # DIRECT and DEPTHWISE read raw weights as they are
        cached = ch[2] == 1 and has_xf
        fused = ch[2] == 2 and has_xf                          # read + transform as one operation (zc_ns): counts as a transform
        if not fused:
            num[0] += t["h2d_end_ns"] - t["h2d_start_ns"]
            den[0] += r["h2d_cached_ns"] if cached else r["h2d_raw_ns"]
        if has_xf and not cached:
            num[1] += t["xform_end_ns"] - t["xform_start_ns"]
            den[1] += r.get("zc_ns", 0) if fused else r["xform_ns"]
        num[2] += t["exec_end_ns"] - t["exec_start_ns"]
        den[2] += r["exec_ns"]

    def scale(v, k):
        return v if num[k] == 0 or den[k] == 0 or not kinds[k] else v * num[k] // den[k]

    out = [dict(r, h2d_raw_ns=scale(r["h2d_raw_ns"], 0), h2d_cached_ns=scale(r["h2d_cached_ns"], 0),
                xform_ns=scale(r["xform_ns"], 1), exec_ns=scale(r["exec_ns"], 2),
                **({"zc_ns": scale(r["zc_ns"], 1)} if "zc_ns" in r else {})) for r in rows]
    return out, list(zip(num, den))


def schedule_eps(exec_of_choice, eps_pct):
    """Algorithm 1's epsilon: eps_pct percent (rounded down) of the summed execution time of the per-layer
    cold-cost choice; exec_of_choice lists those execution times."""
    return sum(exec_of_choice) * eps_pct // 100
