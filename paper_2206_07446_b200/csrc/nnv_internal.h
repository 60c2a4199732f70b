// Internal declarations shared by the host and device translation units of libnnv.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "nnv.h"

struct nnv_cache;

namespace nnv {

// ---- error plumbing -------------------------------------------------------------------------
nnv_status_t fail(nnv_status_t code, const char* fmt, ...);
#define NNV_REQUIRE(cond, code, ...)                       \
    do {                                                   \
        if (!(cond)) return ::nnv::fail((code), __VA_ARGS__); \
    } while (0)
#define NNV_CUDA(call)                                                                     \
    do {                                                                                   \
        cudaError_t e__ = (call);                                                          \
        if (e__ != cudaSuccess)                                                            \
            return ::nnv::fail(NNV_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e__)); \
    } while (0)
#define NNV_REQUIRE_OR(cond, cleanup, code, ...)            \
    do {                                                    \
        if (!(cond)) {                                      \
            cleanup;                                        \
            return ::nnv::fail((code), __VA_ARGS__);        \
        }                                                   \
    } while (0)
#define NNV_TRY(call)                         \
    do {                                      \
        nnv_status_t s__ = (call);            \
        if (s__ != NNV_OK) return s__;        \
    } while (0)

// ---- programmatic dependent launch ----------------------------------------------------------
// Every kernel is launched with the programmatic-stream-serialization attribute and starts with
// pdl_enter(): it lets the next kernel in the stream be launched at once (its blocks get scheduled
// and run their own preamble while this grid is still working) and then waits until the previous
// grid has completed and its writes are visible.  Because every kernel waits before it touches
// global memory, completion is transitive along the stream.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_trigger(); pdl_wait(); }

template <typename... Params, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}
// Same, as thread-block clusters of `cluster_z` consecutive CTAs along grid z (1 = no cluster).
template <typename... Params, typename... Args>
inline cudaError_t launch_pdl_cluster(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      int cluster_z, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 1;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = (unsigned)cluster_z;
    cfg.attrs = attr;
    cfg.numAttrs = cluster_z > 1 ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Params>(args)...);
}
#define NNV_LAUNCH(kernel, grid, block, smem, st, ...) \
    (void)::nnv::launch_pdl(kernel, dim3(grid), dim3(block), (size_t)(smem), st, __VA_ARGS__)
#endif

// ---- device-clock stamps of kernels ----------------------------------------------------------
// A kernel given a non-null `stamp` pointer records the device-wide nanosecond clock when its first
// block starts working (after the wait on the previous kernel) and when its last block has finished:
// stamp[0] = max over blocks of ~start (i.e. ~ of the earliest start), stamp[1] = max over blocks of
// end; both cleared to 0 before the run.  The launchers below take the pointer from
// next_stamp() -- set by the caller right before the launch, cleared by the launch that uses it.
#ifdef __CUDACC__
__device__ __forceinline__ unsigned long long device_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void stamp_start(unsigned long long* stamp) {
    if (stamp) atomicMax(stamp, ~device_ns());
}
__device__ __forceinline__ void stamp_end(unsigned long long* stamp) {
    if (stamp) atomicMax(stamp + 1, device_ns());
}
#endif
constexpr int STAMP_SLOTS_PER_LAYER = 2;                      // transform, execution
constexpr int STAMP_MAX_LAYERS = 4096;
unsigned long long*& next_stamp();                            // thread-local hand-over to the next stamped launch
nnv_status_t stamps_device_base(unsigned long long** base);  // the stamp array on the current device (2 words per slot)

static inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }
static inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

// ---- per-layer derived geometry -------------------------------------------------------------
struct LayerGeom {
    int OH, OW, P;        // output grid and pixel count
    int Cg;               // input channels per group
    int Q, Qp;            // im2col reduction length R*S*C and its padded row length
    int Cp;               // channels padded to a multiple of 8 (Winograd operands)
};

// ---- plan -----------------------------------------------------------------------------------
struct ArenaLayout {
    std::vector<uint64_t> act_off;     // NHWC output of each layer
    uint64_t in_chw = 0, in_hwc = 0, out_chw = 0;
    uint64_t raw_slot0 = 0, raw_slot_bytes = 0, raw_bias_off = 0;
    uint64_t xf_slot0 = 0, xf_slot_bytes = 0;
    std::vector<uint64_t> raw_off, bias_off, xf_off;   // depth 0: one buffer set per conv layer
    uint64_t ws_off = 0, ws_bytes = 0;
    uint64_t total = 0;
};

}  // namespace nnv

namespace nnv {
// Tuning overrides (nnv_tuning_set): process-wide, read when a launch is planned.  `generation`
// changes with every successful nnv_tuning_set call and is part of the key of a recorded graph, so a
// replay never runs with other tilings than an eager call made at the same time would.
struct Tuning {
    int gemm_bn = 0, gemm_splits = 0;         // 0 = the cost model decides
    int gemm_ring = 0;                        // 0 = default ring depth
    int gemm_prefill = 1;
    int conv3x3 = 0;                          // 0 auto, 1 off, 2 forced tiling below
    int conv_mt = 0, conv_bn = 0, conv_splits = 0, conv_na = 0, conv_nb = 0;
    int convp = 0;                            // persistent 3x3 kernel: 0 auto, 1 off, 2 forced with the values below
    int convp_bn = 0, convp_per_sm = 0, convp_na = 0, convp_nb = 0;
    int convw = 0;                            // weights-stationary 3x3 kernel: 0 the library decides, 1 off, 2 wherever it fits
    int side = 1, merge = 1, group = 1;       // pipeline features: side stream, merged reads, grouped transforms
    int copies_first = 1;                     // merged reads all enqueued before the first kernel
    int chunk_first_kb = 256, chunk_max_kb = 16384;   // merged reads: size target of the first chunk, doubling up to the maximum
    int winofused = -1;                       // the one-kernel F(2x2,3x3) path: -1 the library decides, 0 off, 1 on where it applies
    int bf16cvt = 1;                          // BF16 math straight from the fp32 activation (rounded inside the GEMM); 0: explicit bf16 im2col
    int smallp = 1;                           // the weights-on-rows kernel for layers with few pixels
    int smallp_splits = 0;                    // 0 = the cost model decides
    uint64_t generation = 0;
};
Tuning tuning();                              // a copy of the current overrides (thread safe)

struct GraphKey {
    uint64_t tuning_gen = 0;
    std::vector<nnv_choice_t> choices;
    std::vector<const void*> ptrs;
    uint64_t w_bytes = 0;
    int depth = 0;
    bool resident = false;
    bool host_io = false;
    std::vector<int32_t> queues;          // preparation queue per layer (scheduled runs), else empty
    bool operator==(const GraphKey& o) const {
        if (tuning_gen != o.tuning_gen || ptrs != o.ptrs || w_bytes != o.w_bytes || depth != o.depth || resident != o.resident || host_io != o.host_io ||
            queues != o.queues || choices.size() != o.choices.size())
            return false;
        for (size_t i = 0; i < choices.size(); ++i)
            if (choices[i].variant != o.choices[i].variant || choices[i].math != o.choices[i].math ||
                choices[i].cached != o.choices[i].cached)
                return false;
        return true;
    }
};
struct CachedGraph {
    GraphKey key;
    cudaGraphExec_t exec = nullptr;       // null: recording failed, this argument set runs eagerly
};
}  // namespace nnv

struct nnv_plan {
    std::vector<nnv_layer_desc_t> layers;
    std::vector<nnv::LayerGeom> geom;
    nnv_plan_opts_t opts;
    // runtime state of the most recent cold run
    std::vector<cudaEvent_t> ev;          // 3 ordering events per layer (copied, transformed, executed)
    std::vector<cudaEvent_t> tev;         // 6 timing events per layer + 1 origin
    nnv::ArenaLayout last_layout;
    const void* last_arena = nullptr;
    std::vector<nnv::CachedGraph> graphs;   // recorded passes, one per distinct argument set
    int* h_status = nullptr;              // pinned host word the device status is copied into
    cudaStream_t s_side = nullptr;        // the plan's own stream for residual-branch layers (created on first use)
    std::vector<cudaEvent_t> warm_ev;     // continuous mode: layer i's warm weights are prepared
    int stamped_layers = 0;               // layers whose kernels stamped the device clock in the last run (opts.kernel_stamps)
    uint64_t last_enqueue_ns = 0;         // host time the last run spent putting its work on the streams
    bool warm_pending = false;            // warm preparations may still be running (first warm run waits)
};

namespace nnv {

bool variant_has_transform(int variant);
bool math_valid_for(int variant, int math);
int wino_m(int variant);                                     // 2/4/6 or 0
bool is_eligible(const nnv_layer_desc_t& L, int variant);
uint64_t transformed_bytes(const nnv_plan& p, int layer, int variant, int math);
uint64_t exec_ws_bytes(const nnv_plan& p, int layer, int variant, int math);
// How the weights-on-rows kernel (gemm_sp.cuh) would run a layer: K splits, ring depth, padded pixel count and
// the scratch for the partial tiles; use = false when the layer does not qualify.
struct SmallPPlan { bool use; int splits, stages, Npad, nkb; uint32_t b_slot_bytes; uint64_t ws_bytes; };
SmallPPlan small_p_plan(const nnv_layer_desc_t& L, const LayerGeom& g, int variant, int math);
uint64_t raw_weight_bytes(const nnv_layer_desc_t& L);
uint64_t exec_flops(const nnv_plan& p, int layer, int variant);
nnv_status_t check_choice(const nnv_plan& p, int layer, int variant, int math);
// One way to run a layer: a kernel (variant, math), raw or cached weights, and its integer costs.
struct Option {
    int variant, math, cached;
    uint64_t prep, exec;
};
// Options of `layer` from the cost table, and the candidate filter over them (rank order out).
nnv_status_t gather_options(const nnv_plan& p, int layer, const nnv_cost_t* costs, int n_costs, int allow_cached,
                            std::vector<Option>* opts);
void pareto(const std::vector<Option>& in, std::vector<Option>* out);
nnv_status_t layout_arena(const nnv_plan& p, const nnv_choice_t* choices, int depth, ArenaLayout* out);

// ---- kernel launchers (device TUs) ----------------------------------------------------------
// Winograd filter transform: g[K][C][3][3] fp32 -> U[alpha^2][K][Cp] (fp32 or bf16).
nnv_status_t launch_filter_transform(int m, bool bf16, const float* d_g, void* d_U, int K, int C, int Cp,
                                     cudaStream_t st, bool host_src = false);
// GEMM-ready repack: W[K][C][R][S] -> P[K][Qp] (fp32 or bf16).
nnv_status_t launch_pack(bool bf16, const float* d_w, void* d_P, int K, int C, int RS, int Qp, cudaStream_t st,
                         bool host_src = false);

// Several layers' weight transforms in one launch.
enum { XF_PACK = 0, XF_PACK1X1 = 1, XF_WINO2 = 2, XF_WINO4 = 3, XF_WINO6 = 4 };
struct XformDesc {
    const void* src; void* dst;
    int K, C, Cp, RS, Qp;
    int kind, bf16, block0;
    int host_src;                    // src is pinned host memory read in place
};
constexpr int XF_BATCH_MAX = 56;
struct XformBatch { unsigned long long* stamp; int n; int total_blocks; int host_src; XformDesc d[XF_BATCH_MAX]; };
nnv_status_t launch_transform_batch(XformDesc* descs, int n, cudaStream_t st);

// Explicit im2col of an NHWC fp32 image: Xcol[P][Qp], q = (r*S+s)*C + c (fp32 or bf16).
nnv_status_t launch_im2col(bool bf16, const float* d_x, void* d_col, int C, int H, int W, int R, int S,
                           int stride, int pad, int OH, int OW, int Qp, cudaStream_t st);
// Winograd input transform V[alpha^2][T][Cp] = B^T d B per tile and channel.
nnv_status_t launch_wino_input(int m, bool bf16, const float* d_x, void* d_V, int C, int Cp, int H, int W,
                               int pad, int TH, int TW, cudaStream_t st);
// Winograd output transform Y = A^T M A with the layer epilogue.
nnv_status_t launch_wino_output(int m, const float* d_M, float* d_y, const float* d_bias, const float* d_add,
                                int act, int K, int OH, int OW, int TH, int TW, cudaStream_t st);
// fp32 direct convolution from raw OIHW weights (groups == 1).
nnv_status_t launch_direct(const float* d_x, const float* d_w, const float* d_bias, const float* d_add,
                           float* d_y, int act, int C, int H, int W, int K, int R, int S, int stride, int pad,
                           int OH, int OW, cudaStream_t st);
// fp32 depthwise convolution from raw [C][1][R][S] weights.
nnv_status_t launch_depthwise(const float* d_x, const float* d_w, const float* d_bias, const float* d_add,
                              float* d_y, int act, int C, int H, int W, int R, int S, int stride, int pad,
                              int OH, int OW, cudaStream_t st);
nnv_status_t launch_maxpool(const float* d_x, float* d_y, int C, int H, int W, int R, int stride, int pad,
                            int OH, int OW, cudaStream_t st);
nnv_status_t launch_gavgpool(const float* d_x, float* d_y, int C, int H, int W, cudaStream_t st);
nnv_status_t launch_chw_to_hwc(const float* d_in, float* d_out, int C, int H, int W, cudaStream_t st);
nnv_status_t launch_hwc_to_chw(const float* d_in, float* d_out, int C, int H, int W, cudaStream_t st);

// Winograd F(2x2,3x3), TF32, as one kernel (wino_fused.cuh): x NHWC, U[16][K][Cp] fp32, y NHWC.  Needs C % 8 == 0 and
// K % 8 == 0 (wino_fused_applies).
bool wino_fused_applies(const nnv_layer_desc_t& L, int variant, int math);
nnv_status_t launch_wino_f2_fused(const nnv_layer_desc_t& L, const LayerGeom& g, const float* x, const float* U, const float* bias,
                                  const float* addend, float* y, cudaStream_t st);

// Batched tensor-core GEMM  D[b][M][N] = A[b][M][Kd] * B[b][N][Kd]^T, both operands K-major
// (row-major with the reduction index innermost), fp32 accumulate, fp32 output with leading
// dimension ldd.  GEMM_TF32 / GEMM_X3: operands are fp32 words; GEMM_BF16: operands are bf16.  lda/ldb in elements,
// multiples of 16 bytes.  Optional epilogue: + bias[n], + addend[m*ldd+n], activation.
struct GemmArgs {
    const void* A; const void* B; float* D;
    int M, N, Kd, batch;
    int64_t lda, ldb, ldd;            // row strides (elements)
    int64_t strideA, strideB, strideD;  // batch strides (elements)
    const float* bias; const float* addend; int act;
    int mode;                         // GEMM_TF32, GEMM_BF16 or GEMM_X3
    // Implicit im2col: A is the NHWC fp32 activation (C % 4 == 0) read by the TMA in im2col mode;
    // B is the packed weight P[K][Qp] with Kd = Qp; M = OH*OW output pixels.  TF32 mode, batch 1.
    struct { int on, C, H, W, R, S, stride, pad, OW; } ic;
};
// GEMM_X3: fp32 operands; each is split on the fly into bf16 hi + lo and the product is formed
// as hi*hi + lo*hi + hi*lo on the bf16 tensor pipe (fp32-class accuracy, fp32 bytes in memory).
// GEMM_BF16_CVT: A is fp32 and is rounded to bf16 inside the kernel, B is bf16 (weights packed for BF16 math): the
// BF16 accuracy class without a bf16 copy of the activation (direct operand or implicit im2col; batch 1).
enum { GEMM_TF32 = 0, GEMM_BF16 = 1, GEMM_X3 = 2, GEMM_BF16_CVT = 3 };
nnv_status_t launch_gemm_tc(const GemmArgs& a, cudaStream_t st);
// Convolution of a layer with few pixels by the weights-on-rows kernel: x NHWC [H*W][C], wt packed P[K][Qp].
nnv_status_t launch_gemm_sp(const nnv_layer_desc_t& L, const LayerGeom& g, const SmallPPlan& sp, const float* x, const float* wt,
                            const float* bias, const float* addend, float* y, void* ws, cudaStream_t st);
// One-time host set-up of the GEMM (driver entry point, shared-memory attributes); call before
// stream capture.
nnv_status_t gemm_tc_init();

// Model file (cachefile.cpp): exact-range read, and where the two blobs sit in the file.
nnv_status_t cache_read_range(const nnv_cache* c, uint64_t off, void* dst, uint64_t n);
void cache_geometry(const nnv_cache* c, uint64_t* raw_off, uint64_t* cached_off, uint64_t* w_bytes, uint64_t* c_bytes,
                    const nnv_choice_t** file_choices, int* n_layers);

const nnv_layer_desc_t* cache_layers(const nnv_cache* c);      // the file's layer table (n_layers entries)

nnv_status_t read_device_status(int32_t* code);
// Enqueue a copy of the device status word into pinned host memory on `st` (no synchronisation).
nnv_status_t enqueue_status_read(int* h_pinned, cudaStream_t st);

}  // namespace nnv
