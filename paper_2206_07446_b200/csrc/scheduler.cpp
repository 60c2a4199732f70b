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
static uint64_t search(const nnv_plan& p, const std::vector<std::vector<Option>>& options, const uint64_t* pool_ns,
                       int n_little, uint64_t eps, int big_pct, uint64_t limit, std::vector<int>* pick_out,
                       std::vector<int32_t>* queue_out) {
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
        return schedule_queues(p, pl.data(), pb.data(), ex.data(), n_little, eps, q);
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

nnv_status_t nnv_schedule(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                          const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                          uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns) {
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
    std::vector<int> pick;
    std::vector<int32_t> q;
    *t_cold_ns = search(*p, options, pool_ns, n_little, eps_ns, big_pct, combo_limit, &pick, &q);
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
