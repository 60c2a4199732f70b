// Whole-model cold run (three-stream layer pipeline) and per-operation profiling.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <condition_variable>
#include <cstring>
#include <functional>
#include <mutex>
#include <thread>

#include "nnv_internal.h"

namespace nnv {
nnv_status_t do_transform(const nnv_plan& p, int layer, int v, int math, const void* d_raw, void* d_out, cudaStream_t st, bool host_src = false);
nnv_status_t do_exec(const nnv_plan& p, int layer, int v, int math, const void* d_in, const void* d_add,
                     const void* d_wt, const void* d_bias, void* d_out, void* d_ws, uint64_t ws_bytes, cudaStream_t st);
nnv_status_t do_pool(const nnv_plan& p, int layer, const void* d_in, void* d_out, cudaStream_t st);

static nnv_status_t ensure_events(nnv_plan& p, bool timing) {
    const size_t n = p.layers.size();
    const size_t ne = 3 * n + 8 + NNV_MAX_QUEUES;                   // + fork, join(copy), join(transform), 3 transform groups, queue joins, input ready, side join
    if (p.ev.size() != ne) {
        p.ev.resize(ne, nullptr);
        for (size_t i = 0; i < ne; ++i) NNV_CUDA(cudaEventCreateWithFlags(&p.ev[i], cudaEventDisableTiming));
    }
    if (timing && p.tev.size() != 6 * n + 7) {                     // + start / end of the 3 transform groups
        p.tev.resize(6 * n + 7, nullptr);
        for (size_t i = 0; i < 6 * n + 7; ++i) NNV_CUDA(cudaEventCreate(&p.tev[i]));
    }
    return NNV_OK;
}

static inline uint64_t ms_to_ns(float ms) { return ms <= 0.f ? 0ull : (uint64_t)((double)ms * 1e6 + 0.5); }

}  // namespace nnv

using namespace nnv;
namespace nnv {

// One pass over the layer list.  `resident` = the read stage is already done: weights, cached
// blob, input and output are device buffers and nothing crosses the host link.
// Continuous mode (the paper's Section 3.5): where the warm kernel set K_warm is to be left behind.
// d_warm holds a copy of the raw weight blob (same offsets as the host blob) followed, at
// xf_region, by the transformed weights of K_warm laid out by nnv_cached_layout().
struct WarmCtx {
    const nnv_choice_t* warm;
    uint8_t* d_warm;
    uint64_t xf_region;
    std::vector<uint64_t> woff;
};

// True when kernels can read `h` in place: pinned (page-locked) host memory under unified addressing.
static bool host_blob_is_mapped(const void* h) {
    cudaPointerAttributes at{};
    if (cudaPointerGetAttributes(&at, h) != cudaSuccess) { cudaGetLastError(); return false; }
    return at.type == cudaMemoryTypeHost && at.devicePointer == h;
}

static XformDesc make_xform_desc(const nnv_plan& p, int i, const nnv_choice_t& ch, const void* src, void* dst) {
    const nnv_layer_desc_t& L = p.layers[i];
    XformDesc d{};
    d.src = src;
    d.dst = dst;
    d.K = L.K; d.C = L.C; d.Cp = p.geom[i].Cp; d.RS = L.R * L.S; d.Qp = p.geom[i].Qp;
    d.bf16 = ch.math == NNV_MATH_BF16;
    const int m = wino_m(ch.variant);
    d.kind = m == 2 ? XF_WINO2 : m == 4 ? XF_WINO4 : m == 6 ? XF_WINO6 : (d.RS == 1 ? XF_PACK1X1 : XF_PACK);
    return d;
}

static bool same_kernel(const nnv_choice_t& a, const nnv_choice_t& b) { return a.variant == b.variant && a.math == b.math; }

static nnv_status_t run_model(nnv_plan* p, const nnv_choice_t* choices, const void* weights, uint64_t w_bytes,
                              const void* cached_blob, uint64_t c_bytes, const float* input, float* output,
                              void* d_arena, uint64_t arena_bytes, cudaStream_t s_copy, cudaStream_t s_xform,
                              cudaStream_t s_exec, int depth, nnv_timing_t* timings, bool resident,
                              const int32_t* queue_of = nullptr, const cudaStream_t* s_prep = nullptr, int n_little = 0,
                              int io_host = -1, const WarmCtx* wc = nullptr, bool wait_warm = false,
                              const std::function<nnv_status_t(int)>* before_read = nullptr) {
    const int n = (int)p->layers.size();
    const bool queued = queue_of != nullptr;        // preparations follow a schedule: queue 0 = s_exec, j = s_prep[j-1]
    const bool host_io = io_host < 0 ? !resident : io_host != 0;   // input / output are host buffers
    ArenaLayout A;
    NNV_TRY(layout_arena(*p, choices, depth, &A));
    NNV_REQUIRE(arena_bytes >= A.total, NNV_ERR_WORKSPACE_TOO_SMALL, "arena needs %llu bytes, got %llu",
                (unsigned long long)A.total, (unsigned long long)arena_bytes);
    std::vector<uint64_t> coff(n, 0);
    uint64_t ctotal = 0;
    NNV_TRY(nnv_cached_layout(p, choices, coff.data(), &ctotal));
    NNV_REQUIRE(ctotal == 0 || (cached_blob && c_bytes >= ctotal), NNV_ERR_INVALID_ARG,
                "cached blob needs %llu bytes", (unsigned long long)ctotal);
    NNV_REQUIRE(!resident || (aligned256(weights) && (!cached_blob || aligned256(cached_blob))), NNV_ERR_INVALID_ARG,
                "device-resident blobs must be 256-byte aligned");
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p->layers[i];
        if (L.op != NNV_OP_CONV) continue;
        NNV_REQUIRE(L.w_off + raw_weight_bytes(L) <= w_bytes && (!L.has_bias || L.b_off + 4ull * L.K <= w_bytes),
                    NNV_ERR_INVALID_ARG, "layer %d: weights lie outside the weight blob", i);
    }
    if (!resident && !wc) {
        bool any_zc = false;
        for (int i = 0; i < n; ++i)
            any_zc = any_zc || (p->layers[i].op == NNV_OP_CONV && variant_has_transform(choices[i].variant) && choices[i].cached == NNV_ARM_ZERO_COPY);
        NNV_REQUIRE(!any_zc || host_blob_is_mapped(weights), NNV_ERR_INVALID_ARG,
                    "the zero-copy arm needs the weight blob in pinned host memory that kernels can address");
    }
    NNV_TRY(ensure_events(*p, timings != nullptr));
    if (wc && p->warm_ev.size() != (size_t)n) {
        p->warm_ev.assign(n, nullptr);
        for (int i = 0; i < n; ++i) NNV_CUDA(cudaEventCreateWithFlags(&p->warm_ev[i], cudaEventDisableTiming));
    }
    if (!p->h_status) NNV_CUDA(cudaHostAlloc((void**)&p->h_status, sizeof(int), cudaHostAllocDefault));
    p->last_layout = A;
    p->last_arena = d_arena;

    uint8_t* base = (uint8_t*)d_arena;
    auto EV = [&](int layer, int k) { return p->ev[3 * layer + k]; };       // 0 copied, 1 transformed, 2 executed
    auto TEV = [&](int layer, int k) { return p->tev[1 + 6 * layer + k]; };
    const bool tm = timings != nullptr;
    if (tm) std::memset(timings, 0, sizeof(nnv_timing_t) * n);
    NNV_TRY(gemm_tc_init());

    // Residual-branch layers (a conv whose output is only ever the addend of a later layer, e.g. the
    // 1x1 downsample of a ResNet block) run on a side stream of the plan's own, beside the main
    // branch, when they need no execution scratch (the one scratch buffer belongs to s_exec).
    std::vector<char> on_side(n, 0);
    bool any_side = false;
    const Tuning tn = tuning();
    if (!queued && tn.side) {
        for (int i = 0; i < n; ++i) {
            if (p->layers[i].op != NNV_OP_CONV || exec_ws_bytes(*p, i, choices[i].variant, choices[i].math) != 0) continue;
            bool as_input = false, as_addend = false;
            for (int j = i + 1; j < n; ++j) {
                as_input = as_input || p->layers[j].in0 == i;
                as_addend = as_addend || p->layers[j].in1 == i;
            }
            on_side[i] = (as_addend && !as_input && i != n - 1) ? 1 : 0;
            any_side = any_side || on_side[i];
        }
    }
    if (any_side && !p->s_side) {
        int prio = 0;
        NNV_CUDA(cudaStreamGetPriority(s_exec, &prio));
        NNV_CUDA(cudaStreamCreateWithPriority(&p->s_side, cudaStreamNonBlocking, prio));
    }
    cudaStream_t s_side = p->s_side;
    const cudaEvent_t ev_input = p->ev[3 * n + 6 + NNV_MAX_QUEUES], ev_side_join = p->ev[3 * n + 7 + NNV_MAX_QUEUES];

    // A host-to-device copy costs ~4 us on top of its bytes even when it directly follows another one on
    // its stream (measured: 96 MB as 1 MB copies moves at 45 GB/s, as 4 MB copies at 51, as 16 MB copies at 53, as one copy at
    // 55), so at depth 0 (where the arena mirrors the host blobs' layouts) consecutive layers whose source
    // and destination ranges line up are read by ONE copy.  The chunks start at 256 KB, so that execution
    // begins early, and double up to 16 MB (measured on the ResNet-50-shaped model: 1.84 ms with 4 MB chunks,
    // 1.80 ms with 16 MB ones, 1.71 ms for one bulk copy of the same bytes); all layers of a chunk become ready
    // when it lands, and their weight transforms are one grouped launch.
    struct CopyChunk { const uint8_t* src; uint8_t* dst; uint64_t bytes; int first, last; bool zero_copy; };
    std::vector<CopyChunk> chunks;
    std::vector<int> chunk_of(n, -1);
    bool merge = !resident && !queued && depth == 0 && !wc && tn.merge;
    // (Merging pays on every model shape measured once the copies go first: a MobileNetV2 shape, whose 52 layers hold only
    // 8.8 MB, went from 0.62 to 0.41 ms -- its run is bound by the host's API calls, and merged copies and grouped
    // transforms save two thirds of them.)
    if (merge) {
        const uint64_t kFirstTarget = (uint64_t)tn.chunk_first_kb << 10, kMaxTarget = (uint64_t)tn.chunk_max_kb << 10;
        constexpr uint64_t kMaxGap = 4096;
        uint64_t target = kFirstTarget;
        int cur_kind = -1, last_conv = -1;
        for (int i = 0; i < n; ++i)
            if (p->layers[i].op == NNV_OP_CONV) last_conv = i;
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p->layers[i];
            if (L.op != NNV_OP_CONV) continue;
            const nnv_choice_t ch = choices[i];
            const bool zc_l = variant_has_transform(ch.variant) && ch.cached == NNV_ARM_ZERO_COPY;   // read by its transform kernel, no copy
            const bool cached = variant_has_transform(ch.variant) && ch.cached == NNV_ARM_CACHED;
            const int kind = zc_l ? 2 : (int)cached;
            const uint8_t* src = cached ? (const uint8_t*)cached_blob + coff[i] : (const uint8_t*)weights + L.w_off;
            uint8_t* dst = (uint8_t*)d_arena + (cached ? A.xf_off[i] : A.raw_off[i]);
            const uint64_t len = cached ? transformed_bytes(*p, i, ch.variant, ch.math) : raw_weight_bytes(L);
            bool joined = false;
            if (!chunks.empty() && cur_kind == kind && i != last_conv) {   // the last layer's copy is its own: nothing but its
                                                                          // transform and execution then follows the last byte
                CopyChunk& c = chunks.back();
                if (src >= c.src + c.bytes && (uint64_t)(src - (c.src + c.bytes)) <= kMaxGap && src - c.src == dst - c.dst &&
                    c.bytes < target && i - c.first < XF_BATCH_MAX) {
                    c.bytes = (uint64_t)(src - c.src) + len;
                    c.last = i;
                    joined = true;
                }
            }
            if (!joined) {
                if (!chunks.empty()) target = std::min(target * 2, kMaxTarget);
                chunks.push_back(CopyChunk{src, dst, len, i, i, kind == 2});
                cur_kind = kind;
            }
            chunk_of[i] = (int)chunks.size() - 1;
        }
    }

    const bool grouped = resident && depth == 0 && tn.group;
    std::vector<cudaEvent_t> group_event(n, nullptr);

    // Kernel stamps: slot 2i for layer i's transform launch, 2i + 1 for its tensor-core kernel; two words each.
    unsigned long long* stamp_base = nullptr;
    if (p->opts.kernel_stamps && n <= STAMP_MAX_LAYERS) NNV_TRY(stamps_device_base(&stamp_base));
    auto stamp_for = [&](int layer, int which) {
        next_stamp() = stamp_base ? stamp_base + 2 * (STAMP_SLOTS_PER_LAYER * layer + which) : nullptr;
    };
    p->stamped_layers = stamp_base ? n : 0;

    // Everything the pass puts on the streams: fork from s_exec, the per-layer operations, join back.
    auto enqueue = [&]() -> nnv_status_t {
    if (stamp_base) NNV_CUDA(cudaMemsetAsync(stamp_base, 0, sizeof(unsigned long long) * 2 * STAMP_SLOTS_PER_LAYER * n, s_exec));
    if (tm) NNV_CUDA(cudaEventRecord(p->tev[0], s_exec));
    NNV_CUDA(cudaEventRecord(p->ev[3 * n], s_exec));
    if (queued) {
        for (int j = 0; j < n_little; ++j) NNV_CUDA(cudaStreamWaitEvent(s_prep[j], p->ev[3 * n], 0));
    } else {
        if (!resident) NNV_CUDA(cudaStreamWaitEvent(s_copy, p->ev[3 * n], 0));
        NNV_CUDA(cudaStreamWaitEvent(s_xform, p->ev[3 * n], 0));
    }

    // The merged reads.  Nothing orders a chunk's copy behind any kernel (at depth 0 every layer has its own place in
    // the arena), and the link is what the run waits for, so when the weights are already in host memory ALL copies go
    // on the copy stream before anything else is enqueued: the link then never waits for the host to get through the
    // launches of earlier layers (measured on the ResNet-50-shaped model: the second to fourth chunk used to land
    // 15-35 us late each).  With a storage reader in front the copies stay in layer order, each behind its arrival.
    std::vector<char> chunk_issued(chunks.size(), 0);
    auto issue_chunk_copy = [&](int ci) -> nnv_status_t {
        if (chunk_issued[ci]) return NNV_OK;
        chunk_issued[ci] = 1;
        const CopyChunk& c = chunks[ci];
        for (int k = c.first; k <= c.last; ++k)
            if (before_read && p->layers[k].op == NNV_OP_CONV) NNV_TRY((*before_read)(k));
        if (tm) NNV_CUDA(cudaEventRecord(TEV(c.first, 0), s_copy));
        if (!c.zero_copy) NNV_CUDA(cudaMemcpyAsync(c.dst, c.src, c.bytes, cudaMemcpyHostToDevice, s_copy));
        for (int k = c.first; k <= c.last; ++k) {
            const nnv_layer_desc_t& Lk = p->layers[k];
            if (Lk.op == NNV_OP_CONV && Lk.has_bias)
                NNV_CUDA(cudaMemcpyAsync(base + A.bias_off[k], (const uint8_t*)weights + Lk.b_off, 4ull * Lk.K, cudaMemcpyHostToDevice, s_copy));
        }
        if (tm) NNV_CUDA(cudaEventRecord(TEV(c.first, 1), s_copy));
        NNV_CUDA(cudaEventRecord(EV(c.first, 0), s_copy));
        return NNV_OK;
    };
    // model input: NCHW -> device NHWC, on the execution stream (its copy ahead of the weights': copies of one
    // direction are served in the order they were submitted, whatever their streams)
    const nnv_layer_desc_t& L0 = p->layers[0];
    const float* in_chw = input;
    if (host_io) {
        NNV_CUDA(cudaMemcpyAsync(base + A.in_chw, input, 4ull * L0.C * L0.H * L0.W, cudaMemcpyHostToDevice, s_exec));
        in_chw = (const float*)(base + A.in_chw);
    }
    if (merge && !before_read && tn.copies_first)
        for (size_t ci = 0; ci < chunks.size(); ++ci) NNV_TRY(issue_chunk_copy((int)ci));
    NNV_TRY(launch_chw_to_hwc(in_chw, (float*)(base + A.in_hwc), L0.C, L0.H, L0.W, s_exec));
    if (any_side) NNV_CUDA(cudaEventRecord(ev_input, s_exec));

    // Weights resident and no staging limit: nothing orders the transforms, so they are issued as up
    // to three multi-layer launches of growing size (the first ~1 MB of raw weights so that execution
    // can start at once, the next ~8 MB, then all the rest) instead of one small launch per layer.
    if (grouped) {
        std::vector<XformDesc> descs[3];
        int group_first[3] = {0, 0, 0};
        uint64_t first_bytes = 0;
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p->layers[i];
            if (L.op != NNV_OP_CONV) continue;
            const nnv_choice_t ch = choices[i];
            if (!variant_has_transform(ch.variant) || ch.cached == NNV_ARM_CACHED) continue;
            const XformDesc d = make_xform_desc(*p, i, ch, (const uint8_t*)weights + L.w_off, base + A.xf_off[i]);
            const int g = first_bytes < (1u << 20) ? 0 : first_bytes < (9u << 20) ? 1 : 2;
            first_bytes += raw_weight_bytes(L);
            if (descs[g].empty()) group_first[g] = i;
            descs[g].push_back(d);
            group_event[i] = p->ev[3 * n + 3 + g];
        }
        for (int g = 0; g < 3; ++g) {
            if (descs[g].empty()) continue;
            if (tm) NNV_CUDA(cudaEventRecord(p->tev[6 * n + 1 + 2 * g], s_xform));
            stamp_for(group_first[g], 0);
            NNV_TRY(launch_transform_batch(descs[g].data(), (int)descs[g].size(), s_xform));
            next_stamp() = nullptr;
            if (tm) NNV_CUDA(cudaEventRecord(p->tev[6 * n + 2 + 2 * g], s_xform));
            NNV_CUDA(cudaEventRecord(p->ev[3 * n + 3 + g], s_xform));
        }
    }

    std::vector<int> conv_ids;
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p->layers[i];
        const void* in = L.in0 < 0 ? base + A.in_hwc : base + A.act_off[L.in0];
        void* out = base + A.act_off[i];
        // order this layer after its producers when they ran on the other execution stream
        cudaStream_t se = on_side[i] ? s_side : s_exec;
        for (int prod : {L.in0, L.in1})
            if (prod >= 0 && on_side[prod] != on_side[i]) NNV_CUDA(cudaStreamWaitEvent(se, EV(prod, 2), 0));
        if (on_side[i] && L.in0 < 0) NNV_CUDA(cudaStreamWaitEvent(se, ev_input, 0));
        if (L.op != NNV_OP_CONV) {
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 4), s_exec));
            NNV_TRY(do_pool(*p, i, in, out, s_exec));
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 5), s_exec));
            NNV_CUDA(cudaEventRecord(EV(i, 2), s_exec));
            continue;
        }
        const nnv_choice_t ch = choices[i];
        const int j = (int)conv_ids.size();
        conv_ids.push_back(i);
        const int slot = depth ? j % depth : 0;
        const uint8_t* raw = depth ? base + A.raw_slot0 + (uint64_t)slot * A.raw_slot_bytes : base + A.raw_off[i];
        const uint8_t* bias = depth ? raw + A.raw_bias_off : base + A.bias_off[i];
        const uint8_t* xf = depth ? base + A.xf_slot0 + (uint64_t)slot * A.xf_slot_bytes : base + A.xf_off[i];
        const bool has_xf = variant_has_transform(ch.variant);
        const bool cached = has_xf && ch.cached == NNV_ARM_CACHED;
        // zero-copy arm: no copy, the transform kernel reads the host blob itself (with the weights already on the
        // device, or when the raw copy has to stay for warm runs, it is the raw arm)
        const bool zc = has_xf && ch.cached == NNV_ARM_ZERO_COPY && !resident && !wc;
        const uint64_t rbytes = raw_weight_bytes(L), tbytes = transformed_bytes(*p, i, ch.variant, ch.math);
        if (wc) {
            // raw weights and biases are read straight into the copy that stays; a kernel that is also
            // the warm one writes its transformed weights where the warm runs will look for them
            raw = wc->d_warm + L.w_off;
            bias = wc->d_warm + L.b_off;
            if (has_xf && same_kernel(ch, wc->warm[i])) xf = wc->d_warm + wc->xf_region + wc->woff[i];
        }
        cudaEvent_t ready = nullptr;
        uint64_t copied = 0;

        if (queued) {
            // the layer's bundled preparation (read, then transform) on the queue the schedule gave it
            cudaStream_t ps = queue_of[i] == 0 ? s_exec : s_prep[queue_of[i] - 1];
            if (before_read) NNV_TRY((*before_read)(i));
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 0), ps));
            if (zc) {
                // nothing to copy but the bias
            } else if (cached) {
                NNV_CUDA(cudaMemcpyAsync((void*)xf, (const uint8_t*)cached_blob + coff[i], tbytes, cudaMemcpyHostToDevice, ps));
                copied += tbytes;
            } else {
                NNV_CUDA(cudaMemcpyAsync((void*)raw, (const uint8_t*)weights + L.w_off, rbytes, cudaMemcpyHostToDevice, ps));
                copied += rbytes;
            }
            if (L.has_bias) {
                NNV_CUDA(cudaMemcpyAsync((void*)bias, (const uint8_t*)weights + L.b_off, 4ull * L.K, cudaMemcpyHostToDevice, ps));
                copied += 4ull * L.K;
            }
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 1), ps));
            if (has_xf && !cached) {
                if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 2), ps));
                stamp_for(i, 0);
                NNV_TRY(do_transform(*p, i, ch.variant, ch.math, zc ? (const uint8_t*)weights + L.w_off : raw, (void*)xf, ps, zc));
                next_stamp() = nullptr;
                if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 3), ps));
            }
            if (ps != s_exec) {
                NNV_CUDA(cudaEventRecord(EV(i, 1), ps));
                ready = EV(i, 1);
            }
        } else if (resident) {
            raw = (const uint8_t*)weights + L.w_off;
            bias = (const uint8_t*)weights + L.b_off;
            if (cached) xf = (const uint8_t*)cached_blob + coff[i];
        } else {
            // read: the staging slot is free once the layer that used it last has executed
            if (depth && j >= depth) NNV_CUDA(cudaStreamWaitEvent(s_copy, EV(conv_ids[j - depth], 2), 0));
            if (zc && !merge) {
                // fused preparation on the transform stream: (bias copy,) kernel reading the pinned host weights
                if (before_read) NNV_TRY((*before_read)(i));
                if (depth && j >= depth) NNV_CUDA(cudaStreamWaitEvent(s_xform, EV(conv_ids[j - depth], 2), 0));
                if (L.has_bias) {
                    NNV_CUDA(cudaMemcpyAsync((void*)bias, (const uint8_t*)weights + L.b_off, 4ull * L.K, cudaMemcpyHostToDevice, s_xform));
                    copied += 4ull * L.K;
                }
                if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 2), s_xform));
                stamp_for(i, 0);
                NNV_TRY(do_transform(*p, i, ch.variant, ch.math, (const uint8_t*)weights + L.w_off, (void*)xf, s_xform, true));
                next_stamp() = nullptr;
                if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 3), s_xform));
                NNV_CUDA(cudaEventRecord(EV(i, 1), s_xform));
                ready = EV(i, 1);
            } else if (merge) {
                const CopyChunk& c = chunks[chunk_of[i]];
                if (c.first == i) {                             // the chunk's one copy (unless issued ahead) ...
                    NNV_TRY(issue_chunk_copy(chunk_of[i]));
                    // the weight transforms of the chunk's layers: one grouped launch behind the copy
                    std::vector<XformDesc> descs;
                    for (int k = c.first; k <= c.last; ++k) {
                        const nnv_layer_desc_t& Lk = p->layers[k];
                        if (Lk.op != NNV_OP_CONV || !variant_has_transform(choices[k].variant) || choices[k].cached == NNV_ARM_CACHED) continue;
                        if ((choices[k].cached == NNV_ARM_ZERO_COPY) != c.zero_copy) continue;
                        XformDesc d = make_xform_desc(*p, k, choices[k], c.zero_copy ? (const void*)((const uint8_t*)weights + Lk.w_off)
                                                                                   : (const void*)(base + A.raw_off[k]), base + A.xf_off[k]);
                        d.host_src = c.zero_copy ? 1 : 0;
                        descs.push_back(d);
                    }
                    if (!descs.empty()) {
                        NNV_CUDA(cudaStreamWaitEvent(s_xform, EV(i, 0), 0));
                        if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 2), s_xform));
                        stamp_for(i, 0);
                        NNV_TRY(launch_transform_batch(descs.data(), (int)descs.size(), s_xform));
                        next_stamp() = nullptr;
                        if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 3), s_xform));
                        NNV_CUDA(cudaEventRecord(EV(i, 1), s_xform));
                    }
                }
                copied += (zc ? 0 : cached ? tbytes : rbytes) + (L.has_bias ? 4ull * L.K : 0);
                ready = (has_xf && !cached) ? EV(c.first, 1) : EV(c.first, 0);
            } else {
            if (before_read) NNV_TRY((*before_read)(i));         // the layer's bytes have arrived from storage
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 0), s_copy));
            if (cached) {
                NNV_CUDA(cudaMemcpyAsync((void*)xf, (const uint8_t*)cached_blob + coff[i], tbytes, cudaMemcpyHostToDevice, s_copy));
                copied += tbytes;
            } else {
                NNV_CUDA(cudaMemcpyAsync((void*)raw, (const uint8_t*)weights + L.w_off, rbytes, cudaMemcpyHostToDevice, s_copy));
                copied += rbytes;
            }
            if (L.has_bias) {
                NNV_CUDA(cudaMemcpyAsync((void*)bias, (const uint8_t*)weights + L.b_off, 4ull * L.K, cudaMemcpyHostToDevice, s_copy));
                copied += 4ull * L.K;
            }
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 1), s_copy));
            NNV_CUDA(cudaEventRecord(EV(i, 0), s_copy));
            ready = EV(i, 0);
            }
        }

        // transform
        if (queued) {
            // done above, inside the bundled preparation
        } else if (grouped) {
            if (has_xf && !cached) ready = group_event[i];
        } else if (merge || zc) {
            // done with the chunk's copy, or by the fused preparation above
        } else if (has_xf && !cached) {
            if (ready) NNV_CUDA(cudaStreamWaitEvent(s_xform, ready, 0));
            else if (depth && j >= depth) NNV_CUDA(cudaStreamWaitEvent(s_xform, EV(conv_ids[j - depth], 2), 0));
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 2), s_xform));
            stamp_for(i, 0);
            NNV_TRY(do_transform(*p, i, ch.variant, ch.math, raw, (void*)xf, s_xform));
            next_stamp() = nullptr;
            if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 3), s_xform));
            NNV_CUDA(cudaEventRecord(EV(i, 1), s_xform));
            ready = EV(i, 1);
        }

        // execute
        if (ready) NNV_CUDA(cudaStreamWaitEvent(se, ready, 0));
        if (wait_warm && i < (int)p->warm_ev.size() && p->warm_ev[i]) NNV_CUDA(cudaStreamWaitEvent(se, p->warm_ev[i], 0));
        if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 4), se));
        const void* add = L.in1 >= 0 ? base + A.act_off[L.in1] : nullptr;
        stamp_for(i, 1);
        NNV_TRY(do_exec(*p, i, ch.variant, ch.math, in, add, has_xf ? xf : raw, L.has_bias ? bias : nullptr, out,
                        base + A.ws_off, A.ws_bytes, se));
        next_stamp() = nullptr;
        if (tm) NNV_CUDA(cudaEventRecord(TEV(i, 5), se));
        NNV_CUDA(cudaEventRecord(EV(i, 2), se));
        if (tm) {
            timings[i].h2d_bytes = copied;
            timings[i].xform_bytes = (has_xf && !cached) ? rbytes + tbytes : 0;
            timings[i].exec_flops = exec_flops(*p, i, ch.variant);
            timings[i].choice = nnv_choice_t{ch.variant, ch.math, cached ? NNV_ARM_CACHED : zc ? NNV_ARM_ZERO_COPY : NNV_ARM_RAW};
        }
    }

    if (any_side) {                                           // the side stream rejoins the execution stream
        NNV_CUDA(cudaEventRecord(ev_side_join, s_side));
        NNV_CUDA(cudaStreamWaitEvent(s_exec, ev_side_join, 0));
    }
    // last layer's output: device NHWC -> NCHW
    const nnv_layer_desc_t& Ln = p->layers[n - 1];
    const LayerGeom& gn = p->geom[n - 1];
    float* out_chw = host_io ? (float*)(base + A.out_chw) : output;
    NNV_TRY(launch_hwc_to_chw((const float*)(base + A.act_off[n - 1]), out_chw, Ln.K, gn.OH, gn.OW, s_exec));
    if (host_io) NNV_CUDA(cudaMemcpyAsync(output, out_chw, 4ull * gn.P * Ln.K, cudaMemcpyDeviceToHost, s_exec));
    if (queued) {
        for (int j = 0; j < n_little; ++j) {
            NNV_CUDA(cudaEventRecord(p->ev[3 * n + 6 + j], s_prep[j]));
            NNV_CUDA(cudaStreamWaitEvent(s_exec, p->ev[3 * n + 6 + j], 0));
        }
    } else {
        if (!resident) {
            NNV_CUDA(cudaEventRecord(p->ev[3 * n + 1], s_copy));
            NNV_CUDA(cudaStreamWaitEvent(s_exec, p->ev[3 * n + 1], 0));
        }
        NNV_CUDA(cudaEventRecord(p->ev[3 * n + 2], s_xform));
        NNV_CUDA(cudaStreamWaitEvent(s_exec, p->ev[3 * n + 2], 0));
    }
    NNV_TRY(enqueue_status_read(p->h_status, s_exec));
    if (wc) {
        // K_warm - K_cold: behind everything the cold inference needs (the streams are idle from here
        // on, and s_exec no longer waits for them), read what was not read yet and transform it with
        // the warm kernel.  The first warm run waits for warm_ev[i] before executing layer i.
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p->layers[i];
            if (L.op != NNV_OP_CONV) continue;
            const nnv_choice_t ch = choices[i], wm = wc->warm[i];
            const bool cold_read_raw = !(variant_has_transform(ch.variant) && ch.cached == NNV_ARM_CACHED);
            const bool warm_xf = variant_has_transform(wm.variant);
            if (same_kernel(ch, wm) || (cold_read_raw && !warm_xf)) continue;     // nothing left to prepare
            uint8_t* raw = wc->d_warm + L.w_off;
            if (!cold_read_raw) {
                NNV_CUDA(cudaMemcpyAsync(raw, (const uint8_t*)weights + L.w_off, raw_weight_bytes(L), cudaMemcpyHostToDevice, s_copy));
                NNV_CUDA(cudaEventRecord(EV(i, 0), s_copy));
            }
            cudaEvent_t done = EV(i, 0);
            if (warm_xf) {
                NNV_CUDA(cudaStreamWaitEvent(s_xform, EV(i, 0), 0));
                NNV_TRY(do_transform(*p, i, wm.variant, wm.math, raw, wc->d_warm + wc->xf_region + wc->woff[i], s_xform));
                NNV_CUDA(cudaEventRecord(p->warm_ev[i], s_xform));
                done = p->warm_ev[i];
            } else {
                NNV_CUDA(cudaEventRecord(p->warm_ev[i], s_copy));
                done = p->warm_ev[i];
            }
            (void)done;
            p->warm_pending = true;
        }
    }
    return NNV_OK;
    };  // enqueue

    // Without per-operation timings the enqueue sequence is recorded once into a CUDA graph (keyed
    // by the choices and every buffer address) and replayed by later calls with the same arguments:
    // the host then issues one launch instead of a few hundred API calls.
    GraphKey key;
    key.tuning_gen = tn.generation;
    key.choices.assign(choices, choices + n);
    key.ptrs = {weights, cached_blob, input, output, d_arena};
    key.w_bytes = w_bytes; key.depth = depth; key.resident = resident; key.host_io = host_io;
    if (queued) {
        key.queues.assign(queue_of, queue_of + n);
        key.queues.push_back(n_little);
    }
    CachedGraph* cg = nullptr;
    if (!tm && p->opts.use_graphs && !wc && !wait_warm && !before_read) {
        for (CachedGraph& g : p->graphs)
            if (g.key == key) { cg = &g; break; }
        if (!cg) {
            CachedGraph fresh;
            fresh.key = key;
            cudaGraph_t graph = nullptr;
            if (cudaStreamBeginCapture(s_exec, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
                const nnv_status_t rc = enqueue();
                const cudaError_t ce = cudaStreamEndCapture(s_exec, &graph);
                if (rc == NNV_OK && ce == cudaSuccess && graph &&
                    cudaGraphInstantiate(&fresh.exec, graph, 0) == cudaSuccess) {
                    // recorded
                } else {
                    fresh.exec = nullptr;                       // this argument set runs eagerly from now on
                    cudaGetLastError();
                }
                if (graph) cudaGraphDestroy(graph);
            } else {
                cudaGetLastError();
            }
            p->graphs.push_back(fresh);
            cg = &p->graphs.back();
        }
    }
    const auto t_enq0 = std::chrono::steady_clock::now();
    if (cg && cg->exec) {
        NNV_CUDA(cudaGraphLaunch(cg->exec, s_exec));
    } else {
        NNV_TRY(enqueue());
    }
    p->last_enqueue_ns = (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t_enq0).count();
    NNV_CUDA(cudaStreamSynchronize(s_exec));

    if (tm) {
        auto stamp = [&](cudaEvent_t e, uint64_t* out) -> nnv_status_t {
            float ms = 0.f;
            NNV_CUDA(cudaEventElapsedTime(&ms, p->tev[0], e));
            *out = ms_to_ns(ms);
            return NNV_OK;
        };
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p->layers[i];
            NNV_TRY(stamp(TEV(i, 4), &timings[i].exec_start_ns));
            NNV_TRY(stamp(TEV(i, 5), &timings[i].exec_end_ns));
            if (L.op != NNV_OP_CONV) continue;
            const bool zc_i = !queued && !resident && !wc && !merge && variant_has_transform(choices[i].variant) &&
                              choices[i].cached == NNV_ARM_ZERO_COPY;
            if ((!resident || queued) && !zc_i) {
                const int hi = (merge && chunk_of[i] >= 0) ? chunks[chunk_of[i]].first : i;   // a merged copy's interval
                NNV_TRY(stamp(TEV(hi, 0), &timings[i].h2d_start_ns));
                NNV_TRY(stamp(TEV(hi, 1), &timings[i].h2d_end_ns));
            }
            if (timings[i].xform_bytes && grouped) {             // the interval of the layer's multi-layer launch
                const int g = group_event[i] == p->ev[3 * n + 3] ? 0 : group_event[i] == p->ev[3 * n + 4] ? 1 : 2;
                NNV_TRY(stamp(p->tev[6 * n + 1 + 2 * g], &timings[i].xform_start_ns));
                NNV_TRY(stamp(p->tev[6 * n + 2 + 2 * g], &timings[i].xform_end_ns));
            } else if (timings[i].xform_bytes) {
                const int xi = (merge && chunk_of[i] >= 0) ? chunks[chunk_of[i]].first : i;   // a chunk's grouped launch
                NNV_TRY(stamp(TEV(xi, 2), &timings[i].xform_start_ns));
                NNV_TRY(stamp(TEV(xi, 3), &timings[i].xform_end_ns));
            }
        }
    }
    if (*p->h_status != 0) {
        const int code = *p->h_status;
        int32_t dummy = 0;
        read_device_status(&dummy);                 // clears the device word
        return fail((nnv_status_t)code, "a device-side wait gave up during the run");
    }
    return NNV_OK;
}

}  // namespace nnv

extern "C" {

nnv_status_t nnv_cold_run(nnv_plan_t* p, const nnv_choice_t* choices, const void* h_weights, uint64_t w_bytes,
                          const void* h_cached, uint64_t c_bytes, const float* h_input, float* h_output,
                          void* d_arena, uint64_t arena_bytes, void* s_copy, void* s_xform, void* s_exec,
                          int32_t depth, nnv_timing_t* timings) {
    NNV_REQUIRE(p && choices && h_weights && h_input && h_output && d_arena, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(depth >= 0 && depth <= p->opts.max_depth, NNV_ERR_INVALID_ARG, "depth %d outside 0..%d", depth, p->opts.max_depth);
    NNV_REQUIRE(aligned256(d_arena), NNV_ERR_INVALID_ARG, "arena must be 256-byte aligned");
    NNV_REQUIRE(s_copy != s_xform && s_copy != s_exec && s_xform != s_exec, NNV_ERR_INVALID_ARG,
                "the three streams must be distinct");
    return run_model(p, choices, h_weights, w_bytes, h_cached, c_bytes, h_input, h_output, d_arena, arena_bytes,
                     (cudaStream_t)s_copy, (cudaStream_t)s_xform, (cudaStream_t)s_exec, depth, timings, false);
}

nnv_status_t nnv_cold_run_dio(nnv_plan_t* p, const nnv_choice_t* choices, const void* h_weights, uint64_t w_bytes,
                              const void* h_cached, uint64_t c_bytes, const float* d_input, float* d_output,
                              void* d_arena, uint64_t arena_bytes, void* s_copy, void* s_xform, void* s_exec,
                              int32_t depth, nnv_timing_t* timings) {
    NNV_REQUIRE(p && choices && h_weights && d_input && d_output && d_arena, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(depth >= 0 && depth <= p->opts.max_depth, NNV_ERR_INVALID_ARG, "depth %d outside 0..%d", depth, p->opts.max_depth);
    NNV_REQUIRE(aligned256(d_arena) && aligned256(d_input) && aligned256(d_output), NNV_ERR_INVALID_ARG,
                "device pointers must be 256-byte aligned");
    NNV_REQUIRE(s_copy != s_xform && s_copy != s_exec && s_xform != s_exec, NNV_ERR_INVALID_ARG,
                "the three streams must be distinct");
    return run_model(p, choices, h_weights, w_bytes, h_cached, c_bytes, d_input, d_output, d_arena, arena_bytes,
                     (cudaStream_t)s_copy, (cudaStream_t)s_xform, (cudaStream_t)s_exec, depth, timings, false, nullptr, nullptr,
                     0, 0);
}

nnv_status_t nnv_cold_run_queues(nnv_plan_t* p, const nnv_choice_t* choices, const int32_t* queue_of, int32_t n_little,
                                 const void* h_weights, uint64_t w_bytes, const void* h_cached, uint64_t c_bytes,
                                 const float* h_input, float* h_output, void* d_arena, uint64_t arena_bytes,
                                 void* const* streams, nnv_timing_t* timings) {
    NNV_REQUIRE(p && choices && queue_of && h_weights && h_input && h_output && d_arena && streams, NNV_ERR_INVALID_ARG,
                "null argument");
    NNV_REQUIRE(n_little >= 1 && n_little <= NNV_MAX_QUEUES, NNV_ERR_INVALID_ARG, "n_little %d outside 1..%d", n_little,
                NNV_MAX_QUEUES);
    NNV_REQUIRE(aligned256(d_arena), NNV_ERR_INVALID_ARG, "arena must be 256-byte aligned");
    cudaStream_t prep[NNV_MAX_QUEUES];
    for (int j = 0; j <= n_little; ++j) {
        for (int k = 0; k < j; ++k)
            NNV_REQUIRE(streams[j] != streams[k], NNV_ERR_INVALID_ARG, "the streams must be distinct");
        if (j) prep[j - 1] = (cudaStream_t)streams[j];
    }
    for (int i = 0; i < (int)p->layers.size(); ++i)
        if (p->layers[i].op == NNV_OP_CONV)
            NNV_REQUIRE(queue_of[i] >= 0 && queue_of[i] <= n_little, NNV_ERR_INVALID_ARG,
                        "layer %d: queue %d outside 0..%d", i, queue_of[i], n_little);
    return run_model(p, choices, h_weights, w_bytes, h_cached, c_bytes, h_input, h_output, d_arena, arena_bytes,
                     nullptr, nullptr, (cudaStream_t)streams[0], 0, timings, false, queue_of, prep, n_little);
}

nnv_status_t nnv_resident_run(nnv_plan_t* p, const nnv_choice_t* choices, const void* d_weights, uint64_t w_bytes,
                              const void* d_cached, uint64_t c_bytes, const float* d_input, float* d_output,
                              void* d_arena, uint64_t arena_bytes, void* s_xform, void* s_exec, int32_t depth,
                              nnv_timing_t* timings) {
    NNV_REQUIRE(p && choices && d_weights && d_input && d_output && d_arena, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(depth >= 0 && depth <= p->opts.max_depth, NNV_ERR_INVALID_ARG, "depth %d outside 0..%d", depth, p->opts.max_depth);
    NNV_REQUIRE(aligned256(d_arena) && aligned256(d_input) && aligned256(d_output), NNV_ERR_INVALID_ARG,
                "device pointers must be 256-byte aligned");
    NNV_REQUIRE(s_xform != s_exec, NNV_ERR_INVALID_ARG, "the two streams must be distinct");
    return run_model(p, choices, d_weights, w_bytes, d_cached, c_bytes, d_input, d_output, d_arena, arena_bytes,
                     nullptr, (cudaStream_t)s_xform, (cudaStream_t)s_exec, depth, timings, true);
}

// ---- continuous mode: cold inference that leaves K_warm behind, then warm inferences ----------
namespace {
// Warm choices with the `cached` flag normalised: kernels with a transform read the prepared copy.
nnv_status_t warm_layout(const nnv_plan& p, const nnv_choice_t* warm, uint64_t w_bytes, std::vector<nnv_choice_t>* norm,
                         std::vector<uint64_t>* woff, uint64_t* xf_region, uint64_t* total) {
    const int n = (int)p.layers.size();
    norm->assign(warm, warm + n);
    for (int i = 0; i < n; ++i) {
        if (p.layers[i].op != NNV_OP_CONV) continue;
        NNV_TRY(check_choice(p, i, warm[i].variant, warm[i].math));
        (*norm)[i].cached = variant_has_transform(warm[i].variant) ? 1 : 0;
    }
    woff->assign(n, 0);
    uint64_t xf_total = 0;
    NNV_TRY(nnv_cached_layout(&p, norm->data(), woff->data(), &xf_total));
    *xf_region = align_up(w_bytes, 1024);
    *total = *xf_region + xf_total;
    return NNV_OK;
}
}  // namespace

nnv_status_t nnv_warm_bytes(const nnv_plan_t* p, const nnv_choice_t* warm, uint64_t w_bytes, uint64_t* bytes) {
    NNV_REQUIRE(p && warm && bytes, NNV_ERR_INVALID_ARG, "null argument");
    std::vector<nnv_choice_t> norm;
    std::vector<uint64_t> woff;
    uint64_t region = 0;
    return warm_layout(*p, warm, w_bytes, &norm, &woff, &region, bytes);
}

nnv_status_t nnv_cold_run_continuous(nnv_plan_t* p, const nnv_choice_t* cold, const nnv_choice_t* warm,
                                     const void* h_weights, uint64_t w_bytes, const void* h_cached, uint64_t c_bytes,
                                     const float* h_input, float* h_output, void* d_arena, uint64_t arena_bytes,
                                     void* d_warm, uint64_t warm_bytes, void* s_copy, void* s_xform, void* s_exec,
                                     nnv_timing_t* timings) {
    NNV_REQUIRE(p && cold && warm && h_weights && h_input && h_output && d_arena && d_warm, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(aligned256(d_arena) && aligned256(d_warm), NNV_ERR_INVALID_ARG, "device buffers must be 256-byte aligned");
    NNV_REQUIRE(s_copy != s_xform && s_copy != s_exec && s_xform != s_exec, NNV_ERR_INVALID_ARG,
                "the three streams must be distinct");
    WarmCtx wc;
    std::vector<nnv_choice_t> norm;
    uint64_t need = 0;
    NNV_TRY(warm_layout(*p, warm, w_bytes, &norm, &wc.woff, &wc.xf_region, &need));
    NNV_REQUIRE(warm_bytes >= need, NNV_ERR_WORKSPACE_TOO_SMALL, "warm buffer needs %llu bytes, got %llu",
                (unsigned long long)need, (unsigned long long)warm_bytes);
    wc.warm = norm.data();
    wc.d_warm = (uint8_t*)d_warm;
    return run_model(p, cold, h_weights, w_bytes, h_cached, c_bytes, h_input, h_output, d_arena, arena_bytes,
                     (cudaStream_t)s_copy, (cudaStream_t)s_xform, (cudaStream_t)s_exec, 0, timings, false, nullptr, nullptr, 0,
                     -1, &wc, false);
}

nnv_status_t nnv_warm_run(nnv_plan_t* p, const nnv_choice_t* warm, const void* d_warm, uint64_t warm_bytes, uint64_t w_bytes,
                          const float* h_input, float* h_output, void* d_arena, uint64_t arena_bytes, void* s_xform,
                          void* s_exec, nnv_timing_t* timings) {
    NNV_REQUIRE(p && warm && d_warm && h_input && h_output && d_arena, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(aligned256(d_arena) && aligned256(d_warm), NNV_ERR_INVALID_ARG, "device buffers must be 256-byte aligned");
    NNV_REQUIRE(s_xform != s_exec, NNV_ERR_INVALID_ARG, "the two streams must be distinct");
    std::vector<nnv_choice_t> norm;
    std::vector<uint64_t> woff;
    uint64_t region = 0, need = 0;
    NNV_TRY(warm_layout(*p, warm, w_bytes, &norm, &woff, &region, &need));
    NNV_REQUIRE(warm_bytes >= need, NNV_ERR_WORKSPACE_TOO_SMALL, "warm buffer needs %llu bytes, got %llu",
                (unsigned long long)need, (unsigned long long)warm_bytes);
    const bool wait = p->warm_pending;
    const nnv_status_t rc = run_model(p, norm.data(), d_warm, w_bytes, (const uint8_t*)d_warm + region, need - region, h_input,
                                      h_output, d_arena, arena_bytes, nullptr, (cudaStream_t)s_xform, (cudaStream_t)s_exec, 0,
                                      timings, true, nullptr, nullptr, 0, 1, nullptr, wait);
    if (rc == NNV_OK) p->warm_pending = false;       // every preparation this run waited for has finished
    return rc;
}

// ---- cold run fed from the model file: storage -> pinned memory as a fourth pipeline stage -----
nnv_status_t nnv_cold_run_file(nnv_plan_t* p, const nnv_choice_t* choices, const nnv_cache_t* cache, void* h_stage_weights,
                               uint64_t stage_w_bytes, void* h_stage_cached, uint64_t stage_c_bytes, const float* h_input,
                               float* h_output, void* d_arena, uint64_t arena_bytes, void* s_copy, void* s_xform, void* s_exec,
                               int32_t depth, nnv_timing_t* timings, uint64_t* read_ns, uint64_t* read_bytes) {
    NNV_REQUIRE(p && choices && cache && h_stage_weights && h_input && h_output && d_arena, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(depth >= 0 && depth <= p->opts.max_depth, NNV_ERR_INVALID_ARG, "depth %d outside 0..%d", depth, p->opts.max_depth);
    NNV_REQUIRE(aligned256(d_arena), NNV_ERR_INVALID_ARG, "arena must be 256-byte aligned");
    NNV_REQUIRE(s_copy != s_xform && s_copy != s_exec && s_xform != s_exec, NNV_ERR_INVALID_ARG,
                "the three streams must be distinct");
    const int n = (int)p->layers.size();
    uint64_t raw_off, cached_off, w_bytes, c_bytes;
    const nnv_choice_t* file_choices;
    int file_n;
    cache_geometry(cache, &raw_off, &cached_off, &w_bytes, &c_bytes, &file_choices, &file_n);
    NNV_REQUIRE(file_n == n, NNV_ERR_INVALID_ARG, "the file describes %d layers, the plan %d", file_n, n);
    {
        // the file must describe THIS model: same layers, same places in the raw blob
        const nnv_layer_desc_t* fl = cache_layers(cache);
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& a = p->layers[i];
            const nnv_layer_desc_t& b = fl[i];
            const bool same = a.op == b.op && a.C == b.C && a.K == b.K && a.R == b.R && a.S == b.S && a.stride == b.stride &&
                              a.pad == b.pad && a.groups == b.groups && a.H == b.H && a.W == b.W && a.in0 == b.in0 && a.in1 == b.in1 &&
                              a.act == b.act && a.has_bias == b.has_bias &&
                              (a.op != NNV_OP_CONV || (a.w_off == b.w_off && (!a.has_bias || a.b_off == b.b_off)));
            NNV_REQUIRE(same, NNV_ERR_INVALID_ARG, "layer %d of the file differs from the plan's (another model's file?)", i);
        }
    }
    NNV_REQUIRE(stage_w_bytes >= w_bytes, NNV_ERR_WORKSPACE_TOO_SMALL, "weight staging needs %llu bytes", (unsigned long long)w_bytes);
    std::vector<uint64_t> coff(n), fcoff(n);
    uint64_t ctotal = 0, fctotal = 0;
    NNV_TRY(nnv_cached_layout(p, choices, coff.data(), &ctotal));
    if (ctotal) {
        // the cached blob in the file was laid out for the file's own choices: the layers read from it
        // must sit where this run's choices expect them
        NNV_TRY(nnv_cached_layout(p, file_choices, fcoff.data(), &fctotal));
        NNV_REQUIRE(h_stage_cached && stage_c_bytes >= ctotal && c_bytes >= ctotal, NNV_ERR_INVALID_ARG,
                    "the cached blob (file %llu bytes, staging %llu) is smaller than the %llu bytes these choices read",
                    (unsigned long long)c_bytes, (unsigned long long)stage_c_bytes, (unsigned long long)ctotal);
        for (int i = 0; i < n; ++i) {
            if (p->layers[i].op != NNV_OP_CONV || !(variant_has_transform(choices[i].variant) && choices[i].cached == NNV_ARM_CACHED)) continue;
            NNV_REQUIRE(file_choices[i].cached == NNV_ARM_CACHED && file_choices[i].variant == choices[i].variant && file_choices[i].math == choices[i].math &&
                            fcoff[i] == coff[i],
                        NNV_ERR_INVALID_ARG, "layer %d: the file holds no cached weights for this kernel at the expected place", i);
        }
    }

    for (int i = 0; i < n; ++i)
        if (p->layers[i].op == NNV_OP_CONV)
            NNV_REQUIRE(p->layers[i].w_off + raw_weight_bytes(p->layers[i]) <= w_bytes &&
                            (!p->layers[i].has_bias || p->layers[i].b_off + 4ull * p->layers[i].K <= w_bytes),
                        NNV_ERR_INVALID_ARG, "layer %d: weights lie outside the file's raw blob", i);

    // Reader threads.  The bytes each layer's choice reads (its cached blob entry, or its raw weights;
    // its bias) are cut into pieces of up to 2 MiB, listed in layer order; kReaders threads take the next
    // piece off the list and pread it from the file into the pinned staging buffers, at the blobs' own
    // offsets.  Several requests are then in flight at the storage device at once, which a single
    // buffered reader never achieves.  A layer is ready once all its pieces have arrived.
    struct Piece { uint64_t file_off; uint8_t* dst; uint64_t len; int layer; };
    constexpr uint64_t kPiece = 2u << 20;
    constexpr int kReaders = 4;
    std::vector<Piece> pieces;
    std::vector<int> left(n, 0);                              // pieces of layer i still to arrive
    uint64_t bytes_total = 0;
    auto add_range = [&](int i, uint64_t foff, uint8_t* dst, uint64_t len) {
        for (uint64_t o = 0; o < len; o += kPiece) {
            pieces.push_back(Piece{foff + o, dst + o, std::min(kPiece, len - o), i});
            ++left[i];
        }
        bytes_total += len;
    };
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p->layers[i];
        if (L.op != NNV_OP_CONV) continue;
        const nnv_choice_t ch = choices[i];
        if (variant_has_transform(ch.variant) && ch.cached == NNV_ARM_CACHED)
            add_range(i, cached_off + coff[i], (uint8_t*)h_stage_cached + coff[i], transformed_bytes(*p, i, ch.variant, ch.math));
        else
            add_range(i, raw_off + L.w_off, (uint8_t*)h_stage_weights + L.w_off, raw_weight_bytes(L));
        if (L.has_bias) add_range(i, raw_off + L.b_off, (uint8_t*)h_stage_weights + L.b_off, 4ull * L.K);
    }
    std::vector<int> ready(n, 0);
    for (int i = 0; i < n; ++i) ready[i] = left[i] == 0 ? 1 : 0;
    std::mutex mu;
    std::condition_variable cv;
    std::atomic<bool> stop{false};
    std::atomic<size_t> next{0};
    nnv_status_t reader_rc = NNV_OK;
    std::string reader_err;
    uint64_t bytes_read = 0, ns_read = 0;
    const auto t_read0 = std::chrono::steady_clock::now();
    auto reader_fn = [&] {
        for (;;) {
            const size_t k = next.fetch_add(1);
            if (k >= pieces.size() || stop.load()) return;
            const Piece& pc = pieces[k];
            const nnv_status_t rc = cache_read_range(cache, pc.file_off, pc.dst, pc.len);
            std::lock_guard<std::mutex> lk(mu);
            if (rc != NNV_OK) {
                if (reader_rc == NNV_OK) { reader_rc = rc; reader_err = nnv_last_error(); }
                stop = true;
                cv.notify_all();
                return;
            }
            bytes_read += pc.len;
            if (--left[pc.layer] == 0) { ready[pc.layer] = 1; cv.notify_all(); }
            if (bytes_read == bytes_total)
                ns_read = (uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t_read0).count();
        }
    };
    std::vector<std::thread> readers;
    for (int t = 0; t < kReaders; ++t) readers.emplace_back(reader_fn);
    struct Joiner {
        std::vector<std::thread>& ts; std::atomic<bool>& stop;
        void join() { stop = true; for (std::thread& t : ts) if (t.joinable()) t.join(); }
    } reader{readers, stop};
    const std::function<nnv_status_t(int)> gate = [&](int i) -> nnv_status_t {
        std::unique_lock<std::mutex> lk(mu);
        cv.wait(lk, [&] { return ready[i] != 0 || reader_rc != NNV_OK; });
        if (reader_rc != NNV_OK) return fail(reader_rc, "%s", reader_err.c_str());
        return NNV_OK;
    };
    const nnv_status_t rc = run_model(p, choices, h_stage_weights, w_bytes, h_stage_cached, stage_c_bytes, h_input, h_output, d_arena,
                                      arena_bytes, (cudaStream_t)s_copy, (cudaStream_t)s_xform, (cudaStream_t)s_exec, depth, timings,
                                      false, nullptr, nullptr, 0, -1, nullptr, false, &gate);
    reader.join();
    if (rc != NNV_OK) {
        cudaStreamSynchronize((cudaStream_t)s_copy);            // nothing of the failed pass may still touch the staging buffers
        cudaStreamSynchronize((cudaStream_t)s_xform);
        cudaStreamSynchronize((cudaStream_t)s_exec);
        return rc;
    }
    if (read_ns) *read_ns = ns_read;
    if (read_bytes) *read_bytes = bytes_read;
    return NNV_OK;
}

// Reads the stamp array of the plan's most recent run: per layer and slot, {start, end} in device-clock ns (0, 0 = no launch).
static nnv_status_t read_stamps(const nnv_plan_t* p, std::vector<uint64_t>* out) {
    NNV_REQUIRE(p, NNV_ERR_INVALID_ARG, "null argument");
    const int n = (int)p->layers.size();
    NNV_REQUIRE(p->opts.kernel_stamps && p->stamped_layers == n, NNV_ERR_STATE,
                "no run with kernel stamps has used this plan (create it with kernel_stamps = 1)");
    unsigned long long* base = nullptr;
    NNV_TRY(stamps_device_base(&base));
    std::vector<unsigned long long> h((size_t)2 * STAMP_SLOTS_PER_LAYER * n);
    NNV_CUDA(cudaDeviceSynchronize());
    NNV_CUDA(cudaMemcpy(h.data(), base, sizeof(unsigned long long) * h.size(), cudaMemcpyDeviceToHost));
    out->assign(h.size(), 0);
    for (size_t j = 0; j < h.size(); j += 2) {
        const uint64_t start = ~h[j], end = h[j + 1];       // the start slot holds the maximum of ~clock over the blocks
        if (h[j] != 0 && end >= start) { (*out)[j] = start; (*out)[j + 1] = end; }
    }
    return NNV_OK;
}

nnv_status_t nnv_kernel_times(const nnv_plan_t* p, uint64_t* xform_ns, uint64_t* exec_ns) {
    std::vector<uint64_t> h;
    NNV_TRY(read_stamps(p, &h));
    const int n = (int)p->layers.size();
    for (int i = 0; i < n; ++i)
        for (int w = 0; w < STAMP_SLOTS_PER_LAYER; ++w) {
            const size_t j = 2 * ((size_t)STAMP_SLOTS_PER_LAYER * i + w);
            uint64_t* dst = w == 0 ? xform_ns : exec_ns;
            if (dst) dst[i] = h[j + 1] - h[j];
        }
    return NNV_OK;
}

nnv_status_t nnv_kernel_spans(const nnv_plan_t* p, uint64_t* xform_span, uint64_t* exec_span) {
    std::vector<uint64_t> h;
    NNV_TRY(read_stamps(p, &h));
    const int n = (int)p->layers.size();
    uint64_t t0 = ~0ull;
    for (size_t j = 0; j < h.size(); j += 2)
        if (h[j + 1]) t0 = std::min(t0, h[j]);
    for (int i = 0; i < n; ++i)
        for (int w = 0; w < STAMP_SLOTS_PER_LAYER; ++w) {
            const size_t j = 2 * ((size_t)STAMP_SLOTS_PER_LAYER * i + w);
            uint64_t* dst = w == 0 ? xform_span : exec_span;
            if (!dst) continue;
            dst[2 * i] = h[j + 1] ? h[j] - t0 : 0;
            dst[2 * i + 1] = h[j + 1] ? h[j + 1] - t0 : 0;
        }
    return NNV_OK;
}

nnv_status_t nnv_last_enqueue_ns(const nnv_plan_t* p, uint64_t* ns) {
    NNV_REQUIRE(p && ns, NNV_ERR_INVALID_ARG, "null argument");
    *ns = p->last_enqueue_ns;
    return NNV_OK;
}

nnv_status_t nnv_layer_output(const nnv_plan_t* p, int32_t layer, const void** d_ptr, uint64_t* bytes) {
    NNV_REQUIRE(p && d_ptr && bytes, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(layer >= 0 && layer < (int)p->layers.size(), NNV_ERR_INVALID_ARG, "layer %d out of range", layer);
    NNV_REQUIRE(p->last_arena, NNV_ERR_STATE, "no cold run has used this plan yet");
    *d_ptr = (const uint8_t*)p->last_arena + p->last_layout.act_off[layer];
    *bytes = 4ull * p->geom[layer].P * p->layers[layer].K;
    return NNV_OK;
}

// ---- profiling ------------------------------------------------------------------------------
namespace {
constexpr uint64_t FLUSH_BYTES = 192ull << 20;     // larger than the L2

struct ProfLayout {
    std::vector<uint64_t> act_off;
    uint64_t in_chw, in_hwc, raw, bias, xf, ws, ws_bytes, flush, total;
};

nnv_status_t layout_profile(const nnv_plan& p, ProfLayout* out) {
    const int n = (int)p.layers.size();
    ProfLayout a;
    uint64_t pos = 0;
    auto take = [&](uint64_t b) { uint64_t o = pos; pos += align_up(b ? b : 1, 1024); return o; };
    const nnv_layer_desc_t& L0 = p.layers[0];
    a.in_chw = take(4ull * L0.C * L0.H * L0.W);
    a.in_hwc = take(4ull * L0.C * L0.H * L0.W);
    a.act_off.resize(n);
    uint64_t max_raw = 0, max_bias = 0, max_xf = 0, max_ws = 0;
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p.layers[i];
        a.act_off[i] = take(4ull * p.geom[i].P * L.K);
        if (L.op != NNV_OP_CONV) continue;
        max_raw = std::max(max_raw, raw_weight_bytes(L));
        max_bias = std::max<uint64_t>(max_bias, 4ull * L.K);
        for (int v = 0; v < NNV_NUM_VARIANTS; ++v) {
            if (!is_eligible(L, v)) continue;
            for (int m = 0; m < 3; ++m) {
                if (!math_valid_for(v, m)) continue;
                max_xf = std::max(max_xf, transformed_bytes(p, i, v, m));
                max_ws = std::max(max_ws, exec_ws_bytes(p, i, v, m));
            }
        }
    }
    a.raw = take(max_raw);
    a.bias = take(max_bias);
    a.xf = take(max_xf);
    a.ws_bytes = align_up(max_ws ? max_ws : 1, 1024);
    a.ws = take(a.ws_bytes);
    a.flush = take(FLUSH_BYTES);
    a.total = pos;
    *out = a;
    return NNV_OK;
}
}  // namespace

nnv_status_t nnv_profile_arena_bytes(const nnv_plan_t* p, uint64_t* bytes) {
    NNV_REQUIRE(p && bytes, NNV_ERR_INVALID_ARG, "null argument");
    ProfLayout a;
    NNV_TRY(layout_profile(*p, &a));
    *bytes = a.total;
    return NNV_OK;
}

nnv_status_t nnv_profile(nnv_plan_t* p, const void* h_weights, uint64_t w_bytes, const float* h_input, void* d_arena,
                         uint64_t arena_bytes, void* stream, int32_t reps, nnv_cost_t* out, int32_t cap,
                         int32_t* n_out) {
    NNV_REQUIRE(p && h_weights && h_input && d_arena && out && n_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(reps >= 1 && reps <= 1000, NNV_ERR_INVALID_ARG, "reps %d outside 1..1000", reps);
    NNV_REQUIRE(aligned256(d_arena), NNV_ERR_INVALID_ARG, "arena must be 256-byte aligned");
    ProfLayout A;
    NNV_TRY(layout_profile(*p, &A));
    NNV_REQUIRE(arena_bytes >= A.total, NNV_ERR_WORKSPACE_TOO_SMALL, "profiling arena needs %llu bytes, got %llu",
                (unsigned long long)A.total, (unsigned long long)arena_bytes);
    cudaStream_t st = (cudaStream_t)stream;
    uint8_t* base = (uint8_t*)d_arena;
    const int n = (int)p->layers.size();
    const bool host_mapped = host_blob_is_mapped(h_weights);      // the zero-copy arm needs kernels to see the host blob
    cudaEvent_t e0, e1;
    NNV_CUDA(cudaEventCreate(&e0));
    NNV_CUDA(cudaEventCreate(&e1));
    nnv_status_t rc = NNV_OK;
    std::vector<float> samples(reps);
    int cnt = 0;

    // Times `reps` repetitions of `op`, each after an L2 flush, and returns the median in ns.
    auto timed = [&](auto&& op, uint64_t* ns) -> nnv_status_t {
        for (int r = 0; r < reps; ++r) {
            NNV_CUDA(cudaMemsetAsync(base + A.flush, r & 0xff, FLUSH_BYTES, st));
            NNV_CUDA(cudaEventRecord(e0, st));
            NNV_TRY(op());
            NNV_CUDA(cudaEventRecord(e1, st));
            NNV_CUDA(cudaEventSynchronize(e1));
            NNV_CUDA(cudaEventElapsedTime(&samples[r], e0, e1));
        }
        std::sort(samples.begin(), samples.end());
        *ns = ms_to_ns(samples[reps / 2]);
        return NNV_OK;
    };

    auto body = [&]() -> nnv_status_t {
        const nnv_layer_desc_t& L0 = p->layers[0];
        NNV_CUDA(cudaMemcpyAsync(base + A.in_chw, h_input, 4ull * L0.C * L0.H * L0.W, cudaMemcpyHostToDevice, st));
        NNV_TRY(launch_chw_to_hwc((const float*)(base + A.in_chw), (float*)(base + A.in_hwc), L0.C, L0.H, L0.W, st));
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p->layers[i];
            const void* in = L.in0 < 0 ? base + A.in_hwc : base + A.act_off[L.in0];
            void* y = base + A.act_off[i];
            if (L.op != NNV_OP_CONV) {
                NNV_TRY(do_pool(*p, i, in, y, st));
                continue;
            }
            NNV_REQUIRE(L.w_off + raw_weight_bytes(L) <= w_bytes, NNV_ERR_INVALID_ARG, "layer %d: weights lie outside the host blob", i);
            const void* add = L.in1 >= 0 ? base + A.act_off[L.in1] : nullptr;
            const uint64_t rbytes = raw_weight_bytes(L);
            const void* hsrc = (const uint8_t*)h_weights + L.w_off;
            const void* bias = nullptr;
            if (L.has_bias) {
                NNV_CUDA(cudaMemcpyAsync(base + A.bias, (const uint8_t*)h_weights + L.b_off, 4ull * L.K, cudaMemcpyHostToDevice, st));
                bias = base + A.bias;
            }
            // A read is timed as one of kBurst back-to-back copies: in a cold run the link is busy all the time and a
            // copy costs its bytes plus ~4 us; a lone copy between two events costs ~10 us more than that.
            constexpr int kBurst = 4;
            uint64_t h2d_raw = 0;
            NNV_TRY(timed([&]() -> nnv_status_t {
                for (int b = 0; b < kBurst; ++b) NNV_CUDA(cudaMemcpyAsync(base + A.raw, hsrc, rbytes, cudaMemcpyHostToDevice, st));
                return NNV_OK;
            }, &h2d_raw));
            h2d_raw /= kBurst;
            for (int v = 0; v < NNV_NUM_VARIANTS; ++v) {
                if (!is_eligible(L, v)) continue;
                for (int m = 0; m < 3; ++m) {
                    if (!math_valid_for(v, m)) continue;
                    NNV_REQUIRE(cnt < cap, NNV_ERR_INVALID_ARG, "cost table capacity %d too small", cap);
                    nnv_cost_t c{};
                    c.layer = i; c.variant = v; c.math = m;
                    c.h2d_raw_ns = h2d_raw;
                    const bool has_xf = variant_has_transform(v);
                    const uint64_t tbytes = transformed_bytes(*p, i, v, m);
                    if (has_xf) {
                        NNV_TRY(timed([&]() { return do_transform(*p, i, v, m, base + A.raw, base + A.xf, st); }, &c.xform_ns));
                        if (host_mapped) NNV_TRY(timed([&]() { return do_transform(*p, i, v, m, hsrc, base + A.xf, st, true); }, &c.zc_ns));
                        // the cached blob is `tbytes` long; time a copy of that many bytes (scaled when the
                        // host blob is shorter than the layer's transformed weights)
                        const uint64_t cp = std::min<uint64_t>(tbytes, w_bytes);
                        uint64_t t = 0;
                        NNV_TRY(timed([&]() -> nnv_status_t {
                            for (int b = 0; b < kBurst; ++b)
                                NNV_CUDA(cudaMemcpyAsync(base + A.ws, h_weights, std::min<uint64_t>(cp, A.ws_bytes), cudaMemcpyHostToDevice, st));
                            return NNV_OK;
                        }, &t));
                        t /= kBurst;
                        const uint64_t done = std::min<uint64_t>(cp, A.ws_bytes);
                        c.h2d_cached_ns = done ? (uint64_t)((double)t * (double)tbytes / (double)done + 0.5) : 0;
                        // the timed copy overwrote nothing the exec needs: transformed weights live in A.xf
                    } else {
                        c.h2d_cached_ns = h2d_raw;
                    }
                    NNV_TRY(timed([&]() {
                        return do_exec(*p, i, v, m, in, add, has_xf ? base + A.xf : base + A.raw, bias, y, base + A.ws, A.ws_bytes, st);
                    }, &c.exec_ns));
                    out[cnt++] = c;
                }
            }
            // leave the layer's output computed by its lowest-numbered eligible fp32 kernel
            const int vbase = is_eligible(L, NNV_VAR_DIRECT) ? NNV_VAR_DIRECT : NNV_VAR_DEPTHWISE;
            NNV_TRY(do_exec(*p, i, vbase, NNV_MATH_FP32, in, add, base + A.raw, bias, y, base + A.ws, A.ws_bytes, st));
        }
        NNV_CUDA(cudaStreamSynchronize(st));
        return NNV_OK;
    };
    rc = body();
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc != NNV_OK) return rc;
    int32_t code = 0;
    NNV_TRY(read_device_status(&code));
    NNV_REQUIRE(code == 0, (nnv_status_t)code, "a device-side wait gave up during profiling");
    *n_out = cnt;
    return NNV_OK;
}

}  // extern "C"
