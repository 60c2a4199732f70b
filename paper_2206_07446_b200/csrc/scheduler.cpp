// The paper's heuristic kernel scheduler (its Algorithm 1) and the makespan it minimises
// (Eq. (1)-(2) of its Section 3.2), on integer nanosecond costs.  Host logic only.
//
// Queue 0 (the execution stream; the paper's big cores) runs every execution in layer order and
// the preparation (read + transform, or read of cached weights) of the layers in the set B;
// queues 1..M (preparation streams; the paper's little cores) run the other preparations in layer
// order.  An operation starts when its queue is free and its precursors have ended: an execution
// needs its own preparation and the executions of the layers that feed it.
#include <algorithm>
#include <vector>

#include "nnv_internal.h"

namespace nnv {

// End of the last execution for one assignment of preparations to queues.
static uint64_t makespan(const nnv_plan& p, const uint64_t* pl, const uint64_t* pb, const uint64_t* ex,
                         const int32_t* queue_of, int n_little) {
    const int n = (int)p.layers.size();
    std::vector<uint64_t> free_at(n_little + 1, 0), prep_end(n, 0), exec_end(n, 0);
    for (int q = 1; q <= n_little; ++q)
        for (int i = 0; i < n; ++i)
            if (p.layers[i].op == NNV_OP_CONV && queue_of[i] == q) {
                prep_end[i] = free_at[q] + pl[i];
                free_at[q] = prep_end[i];
            }
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p.layers[i];
        if (L.op == NNV_OP_CONV && queue_of[i] == 0) {
            prep_end[i] = free_at[0] + pb[i];
            free_at[0] = prep_end[i];
        }
        uint64_t ready = free_at[0];
        if (L.op == NNV_OP_CONV) ready = std::max(ready, prep_end[i]);
        if (L.in0 >= 0) ready = std::max(ready, exec_end[L.in0]);
        if (L.in1 >= 0) ready = std::max(ready, exec_end[L.in1]);
        exec_end[i] = ready + ex[i];
        free_at[0] = exec_end[i];
    }
    return exec_end[n - 1];
}

// The same latency on a machine where every queue's weights arrive over ONE host link.  A
// preparation is two operations on its queue, read then transform; the link carries one read at a
// time, and when it is free it takes, among the reads whose turn on their own queue has come, the
// one of the lowest layer (reads are issued in layer order).  Event-driven: operations are started
// as soon as they can be, time jumps to the next end.
static uint64_t makespan_link(const nnv_plan& p, const uint64_t* rd, const uint64_t* xl, const uint64_t* xb, const uint64_t* ex,
                              const int32_t* queue_of, int n_little) {
    const int n = (int)p.layers.size();
    enum { READ = 0, XFORM = 1, EXEC = 2 };
    struct Op { int kind, layer; uint64_t dur; };
    std::vector<std::vector<Op>> ops(n_little + 1);
    for (int i = 0; i < n; ++i) {
        const bool conv = p.layers[i].op == NNV_OP_CONV;
        if (conv && queue_of[i] == 0) { ops[0].push_back({READ, i, rd[i]}); ops[0].push_back({XFORM, i, xb[i]}); }
        ops[0].push_back({EXEC, i, ex[i]});
        if (conv && queue_of[i] > 0) { ops[queue_of[i]].push_back({READ, i, rd[i]}); ops[queue_of[i]].push_back({XFORM, i, xl[i]}); }
    }
    constexpr uint64_t NOT_YET = ~0ull;
    std::vector<uint64_t> end_of[3];
    for (auto& v : end_of) v.assign(n, NOT_YET);
    std::vector<size_t> head(n_little + 1, 0);
    std::vector<uint64_t> busy(n_little + 1, 0);
    uint64_t link_free = 0, t = 0;
    auto ended = [&](int kind, int layer) { return end_of[kind][layer] != NOT_YET && end_of[kind][layer] <= t; };
    while (end_of[EXEC][n - 1] == NOT_YET) {
        bool progressed = true;
        while (progressed) {
            progressed = false;
            int wq = -1;                                         // queue of the waiting read of the lowest layer
            for (int q = 0; q <= n_little; ++q) {
                if (head[q] >= ops[q].size() || busy[q] > t) continue;
                const Op& o = ops[q][head[q]];
                if (o.kind == READ) {
                    if (wq < 0 || o.layer < ops[wq][head[wq]].layer) wq = q;
                    continue;
                }
                bool ok;
                if (o.kind == XFORM) {
                    ok = ended(READ, o.layer);
                } else {
                    const nnv_layer_desc_t& L = p.layers[o.layer];
                    ok = (L.op != NNV_OP_CONV || ended(XFORM, o.layer)) && (L.in0 < 0 || ended(EXEC, L.in0)) &&
                         (L.in1 < 0 || ended(EXEC, L.in1));
                }
                if (!ok) continue;
                end_of[o.kind][o.layer] = busy[q] = t + o.dur;
                ++head[q];
                progressed = true;
            }
            if (wq >= 0 && link_free <= t) {
                const Op& o = ops[wq][head[wq]];
                end_of[READ][o.layer] = busy[wq] = link_free = t + o.dur;
                ++head[wq];
                progressed = true;
            }
        }
        if (end_of[EXEC][n - 1] != NOT_YET) break;
        uint64_t next = NOT_YET;                                 // the earliest end after t
        for (const auto& v : end_of)
            for (uint64_t e : v)
                if (e != NOT_YET && e > t) next = std::min(next, e);
        if (next == NOT_YET) break;                              // cannot happen for a topologically ordered plan
        t = next;
    }
    return end_of[EXEC][n - 1];
}

// Algorithm 1's little-core balancing step: round-robin start in layer order, then move operations
// from the longest to the shortest little queue while one shorter than half the gap exists.
struct Item { int layer; uint64_t t; };
static void balance_little(const std::vector<Item>& items, int n_little, uint64_t eps, std::vector<int32_t>* queue_of) {
    std::vector<std::vector<Item>> qs(n_little);
    std::vector<uint64_t> tot(n_little, 0);
    for (size_t k = 0; k < items.size(); ++k) {
        qs[k % n_little].push_back(items[k]);
        tot[k % n_little] += items[k].t;
    }
    for (;;) {
        int jmax = 0, jmin = 0;
        for (int j = 1; j < n_little; ++j) {
            if (tot[j] > tot[jmax]) jmax = j;                   // ties: lowest index
            if (tot[j] < tot[jmin]) jmin = j;
        }
        if (tot[jmax] - tot[jmin] <= eps) break;
        std::vector<Item> sorted = qs[jmax];
        std::sort(sorted.begin(), sorted.end(), [](const Item& a, const Item& b) {
            return a.t != b.t ? a.t > b.t : a.layer < b.layer;
        });
        bool moved = false;
        for (const Item& it : sorted) {
            if (2 * it.t < tot[jmax] - tot[jmin]) {
                auto pos = std::find_if(qs[jmax].begin(), qs[jmax].end(), [&](const Item& x) { return x.layer == it.layer; });
                qs[jmax].erase(pos);
                qs[jmin].push_back(it);
                tot[jmax] -= it.t;
                tot[jmin] += it.t;
                moved = true;
            }
        }
        if (!moved) break;
    }
    for (int j = 0; j < n_little; ++j)
        for (const Item& it : qs[j]) (*queue_of)[it.layer] = j + 1;
}

// Algorithm 1's body for one kernel combination: grow B while the little queues outlast queue 0.
static uint64_t schedule_queues(const nnv_plan& p, const uint64_t* pl, const uint64_t* pb, const uint64_t* ex,
                                int n_little, uint64_t eps, std::vector<int32_t>* queue_of) {
    const int n = (int)p.layers.size();
    std::vector<int> conv;
    uint64_t exec_sum = 0;
    for (int i = 0; i < n; ++i) {
        if (p.layers[i].op == NNV_OP_CONV) conv.push_back(i);
        exec_sum += ex[i];
    }
    queue_of->assign(n, -1);
    if (conv.empty()) return makespan(p, pl, pb, ex, queue_of->data(), n_little);
    std::vector<char> inB(n, 0);
    inB[conv[0]] = 1;
    for (;;) {
        std::vector<Item> rest;
        for (int i : conv)
            if (!inB[i]) rest.push_back({i, pl[i]});
        for (int i : conv) (*queue_of)[i] = 0;
        if (!rest.empty()) balance_little(rest, n_little, eps, queue_of);
        std::vector<uint64_t> tot(n_little + 1, 0);
        uint64_t t0 = exec_sum;
        for (int i : conv) {
            if (inB[i]) t0 += pb[i];
            else tot[(*queue_of)[i]] += pl[i];
        }
        const uint64_t t_little = *std::max_element(tot.begin(), tot.end());
        if (t_little <= t0 + eps) break;
        const uint64_t gap = t_little - t0;
        int pick = -1;
        for (int i : conv)
            if (!inB[i] && pb[i] + pl[i] < gap) { pick = i; break; }
        if (pick < 0) break;
        inB[pick] = 1;
    }
    return makespan(p, pl, pb, ex, queue_of->data(), n_little);
}

// Outer loop of Algorithm 1 over the filtered candidates: exhaustive up to `limit` combinations,
// else coordinate descent from the per-layer cold-cost minimum (first strict improvement in rank
// order per layer, at most 8 sweeps).  Ties keep the earlier combination.
// With `reads` (per layer and option, the part of the preparation that crosses the host link) the latency
// compared and returned is makespan_link's; the queues still come from the heuristic on the bundled times.
static uint64_t search(const nnv_plan& p, const std::vector<std::vector<Option>>& options, const uint64_t* pool_ns,
                       int n_little, uint64_t eps, int big_pct, uint64_t limit, std::vector<int>* pick_out,
                       std::vector<int32_t>* queue_out, const std::vector<std::vector<uint64_t>>* reads = nullptr) {
    const int n = (int)p.layers.size();
    std::vector<int> conv;
    for (int i = 0; i < n; ++i)
        if (p.layers[i].op == NNV_OP_CONV) conv.push_back(i);
    std::vector<uint64_t> pl(n), pb(n), ex(n);
    auto evaluate = [&](const std::vector<int>& pick, std::vector<int32_t>* q) {
        for (int i = 0; i < n; ++i) {
            if (p.layers[i].op == NNV_OP_CONV) {
                const Option& o = options[i][pick[i]];
                pl[i] = o.prep; pb[i] = o.prep * (uint64_t)big_pct / 100; ex[i] = o.exec;
            } else {
                pl[i] = pb[i] = 0; ex[i] = pool_ns ? pool_ns[i] : 0;
            }
        }
        const uint64_t t = schedule_queues(p, pl.data(), pb.data(), ex.data(), n_little, eps, q);
        if (!reads) return t;
        std::vector<uint64_t> rd(n, 0), xl(n, 0), xb(n, 0);
        for (int i = 0; i < n; ++i)
            if (p.layers[i].op == NNV_OP_CONV) {
                rd[i] = (*reads)[i][pick[i]];
                xl[i] = pl[i] - rd[i];
                xb[i] = xl[i] * (uint64_t)big_pct / 100;
            }
        return makespan_link(p, rd.data(), xl.data(), xb.data(), ex.data(), q->data(), n_little);
    };
    uint64_t total = 1;
    for (int i : conv) {
        total *= options[i].size();
        if (total > limit) break;
    }
    std::vector<int> best(n, 0);
    std::vector<int32_t> bq, q;
    uint64_t bt = 0;
    if (total <= limit) {
        std::vector<int> pick(n, 0);
        bool first = true;
        for (;;) {
            const uint64_t t = evaluate(pick, &q);
            if (first || t < bt) { bt = t; best = pick; bq = q; first = false; }
            int k = (int)conv.size() - 1;                       // odometer, last layer fastest
            while (k >= 0 && ++pick[conv[k]] == (int)options[conv[k]].size()) pick[conv[k--]] = 0;
            if (k < 0) break;
        }
    } else {
        for (int i : conv) {
            int arg = 0;
            for (int c = 1; c < (int)options[i].size(); ++c)
                if (options[i][c].prep + options[i][c].exec < options[i][arg].prep + options[i][arg].exec) arg = c;
            best[i] = arg;
        }
        bt = evaluate(best, &bq);
        for (int sweep = 0; sweep < 8; ++sweep) {
            bool changed = false;
            for (int i : conv) {
                for (int c = 0; c < (int)options[i].size(); ++c) {
                    if (c == best[i]) continue;
                    std::vector<int> trial = best;
                    trial[i] = c;
                    const uint64_t t = evaluate(trial, &q);
                    if (t < bt) { bt = t; best = trial; bq = q; changed = true; break; }
                }
            }
            if (!changed) break;
        }
    }
    *pick_out = best;
    *queue_out = bq;
    return bt;
}

static nnv_status_t check_queues(const nnv_plan& p, const int32_t* queue_of, int n_little) {
    for (int i = 0; i < (int)p.layers.size(); ++i)
        if (p.layers[i].op == NNV_OP_CONV)
            NNV_REQUIRE(queue_of[i] >= 0 && queue_of[i] <= n_little, NNV_ERR_INVALID_ARG,
                        "layer %d: queue %d outside 0..%d", i, queue_of[i], n_little);
    return NNV_OK;
}

}  // namespace nnv

using namespace nnv;

extern "C" {

nnv_status_t nnv_simulate(const nnv_plan_t* p, const uint64_t* prep_little_ns, const uint64_t* prep_big_ns,
                          const uint64_t* exec_ns, const int32_t* queue_of, int32_t n_little, uint64_t* t_cold_ns) {
    NNV_REQUIRE(p && prep_little_ns && prep_big_ns && exec_ns && queue_of && t_cold_ns, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(n_little >= 1 && n_little <= NNV_MAX_QUEUES, NNV_ERR_INVALID_ARG, "n_little %d outside 1..%d", n_little, NNV_MAX_QUEUES);
    NNV_TRY(check_queues(*p, queue_of, n_little));
    *t_cold_ns = makespan(*p, prep_little_ns, prep_big_ns, exec_ns, queue_of, n_little);
    return NNV_OK;
}

nnv_status_t nnv_schedule_queues(const nnv_plan_t* p, const uint64_t* prep_little_ns, const uint64_t* prep_big_ns,
                                 const uint64_t* exec_ns, int32_t n_little, uint64_t eps_ns, int32_t* queue_of,
                                 uint64_t* t_cold_ns) {
    NNV_REQUIRE(p && prep_little_ns && prep_big_ns && exec_ns && queue_of && t_cold_ns, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(n_little >= 1 && n_little <= NNV_MAX_QUEUES, NNV_ERR_INVALID_ARG, "n_little %d outside 1..%d", n_little, NNV_MAX_QUEUES);
    std::vector<int32_t> q;
    *t_cold_ns = schedule_queues(*p, prep_little_ns, prep_big_ns, exec_ns, n_little, eps_ns, &q);
    std::copy(q.begin(), q.end(), queue_of);
    return NNV_OK;
}

nnv_status_t nnv_simulate_link(const nnv_plan_t* p, const uint64_t* read_ns, const uint64_t* xform_little_ns,
                               const uint64_t* xform_big_ns, const uint64_t* exec_ns, const int32_t* queue_of, int32_t n_little,
                               uint64_t* t_cold_ns) {
    NNV_REQUIRE(p && read_ns && xform_little_ns && xform_big_ns && exec_ns && queue_of && t_cold_ns, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(n_little >= 1 && n_little <= NNV_MAX_QUEUES, NNV_ERR_INVALID_ARG, "n_little %d outside 1..%d", n_little, NNV_MAX_QUEUES);
    NNV_TRY(check_queues(*p, queue_of, n_little));
    *t_cold_ns = makespan_link(*p, read_ns, xform_little_ns, xform_big_ns, exec_ns, queue_of, n_little);
    return NNV_OK;
}

static nnv_status_t schedule_impl(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                                  const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                                  uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns, bool link);

nnv_status_t nnv_schedule(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                          const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                          uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns) {
    return schedule_impl(p, costs, n_costs, allow_cached, pool_ns, n_little, eps_ns, big_pct, combo_limit, out, queue_of, t_cold_ns, false);
}

nnv_status_t nnv_schedule_link(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                               const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                               uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns) {
    return schedule_impl(p, costs, n_costs, allow_cached, pool_ns, n_little, eps_ns, big_pct, combo_limit, out, queue_of, t_cold_ns, true);
}

nnv_status_t nnv_schedule_eps(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                              int32_t eps_pct, uint64_t* eps_ns) {
    NNV_REQUIRE(p && costs && eps_ns, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(eps_pct >= 0 && eps_pct <= 100, NNV_ERR_INVALID_ARG, "eps_pct %d outside 0..100", eps_pct);
    const int n = (int)p->layers.size();
    std::vector<nnv_choice_t> ch(n);
    NNV_TRY(nnv_select_kernels(p, costs, n_costs, allow_cached, ch.data()));
    uint64_t sum = 0;
    for (int i = 0; i < n; ++i) {
        if (p->layers[i].op != NNV_OP_CONV) continue;
        for (int r = 0; r < n_costs; ++r)
            if (costs[r].layer == i && costs[r].variant == ch[i].variant && costs[r].math == ch[i].math) { sum += costs[r].exec_ns; break; }
    }
    *eps_ns = sum * (uint64_t)eps_pct / 100;
    return NNV_OK;
}

nnv_status_t nnv_calibrate_costs(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, const nnv_choice_t* choices,
                                 const nnv_timing_t* timings, int32_t kinds, nnv_cost_t* out, uint64_t* factors) {
    NNV_REQUIRE(p && costs && choices && timings && out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(kinds >= 0 && kinds <= 7, NNV_ERR_INVALID_ARG, "kinds %d is not a mask of read (1), transform (2), execution (4)", kinds);
    const int n = (int)p->layers.size();
    uint64_t num[3] = {0, 0, 0}, den[3] = {0, 0, 0};             // read, transform, execution
    for (int i = 0; i < n; ++i) {
        if (p->layers[i].op != NNV_OP_CONV) continue;
        NNV_TRY(check_choice(*p, i, choices[i].variant, choices[i].math));
        const nnv_cost_t* row = nullptr;
        for (int r = 0; r < n_costs && !row; ++r)
            if (costs[r].layer == i && costs[r].variant == choices[i].variant && costs[r].math == choices[i].math) row = &costs[r];
        NNV_REQUIRE(row, NNV_ERR_STATE, "no cost row for the kernel chosen for layer %d", i);
        const nnv_timing_t& t = timings[i];
        NNV_REQUIRE(t.h2d_end_ns >= t.h2d_start_ns && t.xform_end_ns >= t.xform_start_ns && t.exec_end_ns >= t.exec_start_ns,
                    NNV_ERR_INVALID_ARG, "layer %d: a timing interval ends before it starts", i);
        const bool has_xf = variant_has_transform(choices[i].variant);
        const bool cached = has_xf && choices[i].cached == NNV_ARM_CACHED;
        const bool zc = has_xf && choices[i].cached == NNV_ARM_ZERO_COPY;
        if (!zc) {                                               // a zero-copy preparation has no read of its own:
            num[0] += t.h2d_end_ns - t.h2d_start_ns;             // it is measured, and rescaled, as a transform
            den[0] += cached ? row->h2d_cached_ns : row->h2d_raw_ns;
        }
        if (has_xf && !cached) {
            num[1] += t.xform_end_ns - t.xform_start_ns;
            den[1] += zc ? row->zc_ns : row->xform_ns;
        }
        num[2] += t.exec_end_ns - t.exec_start_ns;
        den[2] += row->exec_ns;
    }
    auto scale = [&](uint64_t v, int k) -> uint64_t {
        if (num[k] == 0 || den[k] == 0 || !((kinds >> k) & 1)) return v;
        return (uint64_t)((unsigned __int128)v * num[k] / den[k]);
    };
    for (int r = 0; r < n_costs; ++r) {
        nnv_cost_t c = costs[r];
        c.h2d_raw_ns = scale(c.h2d_raw_ns, 0);
        c.h2d_cached_ns = scale(c.h2d_cached_ns, 0);
        c.xform_ns = scale(c.xform_ns, 1);
        c.zc_ns = scale(c.zc_ns, 1);
        c.exec_ns = scale(c.exec_ns, 2);
        out[r] = c;
    }
    if (factors)
        for (int k = 0; k < 3; ++k) { factors[2 * k] = num[k]; factors[2 * k + 1] = den[k]; }
    return NNV_OK;
}

static nnv_status_t schedule_impl(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                                  const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                                  uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns, bool link) {
    NNV_REQUIRE(p && costs && out && queue_of && t_cold_ns, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(n_little >= 1 && n_little <= NNV_MAX_QUEUES, NNV_ERR_INVALID_ARG, "n_little %d outside 1..%d", n_little, NNV_MAX_QUEUES);
    NNV_REQUIRE(big_pct >= 0 && big_pct <= 1000, NNV_ERR_INVALID_ARG, "big_pct %d outside 0..1000", big_pct);
    const int n = (int)p->layers.size();
    std::vector<std::vector<Option>> options(n);
    for (int i = 0; i < n; ++i) {
        if (p->layers[i].op != NNV_OP_CONV) continue;
        std::vector<Option> all;
        NNV_TRY(gather_options(*p, i, costs, n_costs, allow_cached, &all));
        NNV_REQUIRE(!all.empty(), NNV_ERR_STATE, "no cost rows for conv layer %d", i);
        pareto(all, &options[i]);
    }
    std::vector<std::vector<uint64_t>> reads(n);                 // per option, the part of prep that is the read
    if (link) {
        for (int i = 0; i < n; ++i)
            for (const Option& o : options[i]) {
                uint64_t rd = 0;
                for (int r = 0; r < n_costs; ++r)
                    if (costs[r].layer == i && costs[r].variant == o.variant && costs[r].math == o.math) {
                        // a zero-copy preparation holds the link for its whole length
                        rd = o.cached == NNV_ARM_CACHED ? costs[r].h2d_cached_ns : o.cached == NNV_ARM_ZERO_COPY ? costs[r].zc_ns : costs[r].h2d_raw_ns;
                        break;
                    }
                reads[i].push_back(rd);
            }
    }
    std::vector<int> pick;
    std::vector<int32_t> q;
    *t_cold_ns = search(*p, options, pool_ns, n_little, eps_ns, big_pct, combo_limit, &pick, &q, link ? &reads : nullptr);
    for (int i = 0; i < n; ++i) {
        queue_of[i] = q[i];
        if (p->layers[i].op == NNV_OP_CONV) {
            const Option& o = options[i][pick[i]];
            out[i] = nnv_choice_t{o.variant, o.math, o.cached};
        } else {
            out[i] = nnv_choice_t{-1, -1, 0};
        }
    }
    return NNV_OK;
}

}  // extern "C"
