/*
 * nnv.h -- C ABI of the cold-start convolution path for NVIDIA B200 (sm_100a).
 *
 * The path is the one the NNV12 paper ("Boosting DNN Cold Inference on Devices")
 * optimises: for every convolution layer, raw fp32 weights are READ (here: copied
 * from pinned host memory to the GPU), TRANSFORMED into the layout the chosen
 * kernel wants, and the layer is EXECUTED (the paper's Section 2 stage list and
 * the read / transform / execute operation triple <r_i, w_i, e_i> of its
 * Section 3.2).  On top sit the three knobs of its Section 3.1: kernel selection
 * by cold cost, bypassing the transform with cached post-transform weights, and
 * pipelining the layers' operations.
 *
 * Conventions for every call
 *   - Plain C types only.  Pointers prefixed h_ are HOST pointers, d_ are DEVICE
 *     pointers.  Streams are cudaStream_t / CUstream handles passed as void*.
 *   - The caller owns every device buffer, host blob and stream.  The library owns
 *     only nnv_plan_t (host memory, plus CUDA events, recorded graphs and one
 *     side stream created lazily) and nnv_cache_t (an open model file), and allocates
 *     NO device memory; nnv_cold_run and nnv_profile sub-allocate from the arena
 *     the caller passes.
 *   - Device pointers must be 256-byte aligned unless stated otherwise.
 *   - Every call returns nnv_status_t and never throws, aborts or exits.
 *     Argument and shape errors are found on the host before any launch.
 *     nnv_last_error() gives a thread-local message for the last failing call.
 *   - nnv_transform_weights, nnv_conv_exec, nnv_pool_exec and the layout helpers
 *     only enqueue work on the given stream; nnv_cold_run and nnv_profile
 *     synchronise before returning.
 *   - Layouts.  Raw weights: OIHW fp32, W[k][c][r][s], c over C/groups.
 *     Activations on the device: NHWC fp32, X[h][w][c], batch 1, no channel
 *     padding.  Model input/output on the host: NCHW fp32.
 *     Transformed weights:
 *       Winograd F(m x m, 3 x 3):  U[xi*alpha+nu][k][cp], alpha = m+2,
 *           cp < Cp = ceil(C/8)*8 (entries with cp >= C are +0), fp32 (TF32 math)
 *           or bf16 (BF16 math, F(2x2,3x3) only: one bf16 pass in the F(4x4) /
 *           F(6x6) domain misses the 1e-2 output tolerance, so those two exist
 *           in the TF32 accuracy class only);
 *       IM2COL / GEMM1X1:          P[k][q], q = (r*S+s)*C + c, row length
 *           Qp = ceil(R*S*C/8)*8, pad +0; each element rounded to nearest even to
 *           TF32 precision and kept as an fp32 word (TF32), or to bf16 (BF16);
 *       DIRECT / DEPTHWISE:        none -- these kernels read the raw weights.
 */
#ifndef NNV_H_
#define NNV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    NNV_OK = 0,
    NNV_ERR_INVALID_ARG = 1,          /* null / misaligned pointer, bad index, bad enum      */
    NNV_ERR_UNSUPPORTED = 2,          /* layer shape or (variant, math) pair not implemented */
    NNV_ERR_STATE = 3,                /* call order / plan state problem                     */
    NNV_ERR_WORKSPACE_TOO_SMALL = 4,  /* d_ws / d_arena smaller than the size query returns  */
    NNV_ERR_CUDA = 5,                 /* a CUDA runtime / driver call failed                 */
    NNV_ERR_TIMEOUT = 6               /* a bounded device-side wait gave up                  */
} nnv_status_t;

typedef struct nnv_plan nnv_plan_t;   /* opaque; created by nnv_plan_create */
typedef struct nnv_cache nnv_cache_t; /* opaque; an open model file, created by nnv_cache_open */

typedef enum { NNV_OP_CONV = 0, NNV_OP_MAXPOOL = 1, NNV_OP_GAVGPOOL = 2 } nnv_op_t;

/* Kernel variants of the convolution operator ("one operator, many kernels",
 * the paper's Section 3.1.1).  Enum order is the tie-break order of selection. */
typedef enum {
    NNV_VAR_DIRECT = 0,     /* fp32 FFMA, reads raw weights, no transform            */
    NNV_VAR_IM2COL = 1,     /* im2col + tensor-core GEMM on packed weights           */
    NNV_VAR_GEMM1X1 = 2,    /* 1x1 conv as a tensor-core GEMM over pixels            */
    NNV_VAR_DEPTHWISE = 3,  /* fp32 direct depthwise, reads raw weights              */
    NNV_VAR_WINO_F2 = 4,    /* Winograd F(2x2,3x3)                                   */
    NNV_VAR_WINO_F4 = 5,    /* Winograd F(4x4,3x3)                                   */
    NNV_VAR_WINO_F6 = 6     /* Winograd F(6x6,3x3)                                   */
} nnv_variant_t;
#define NNV_NUM_VARIANTS 7

typedef enum { NNV_MATH_FP32 = 0, NNV_MATH_TF32 = 1, NNV_MATH_BF16 = 2 } nnv_math_t;

typedef struct {
    int32_t op;                 /* nnv_op_t                                                      */
    int32_t C, K;               /* input / output channels (pools: K == C)                       */
    int32_t R, S;               /* filter / window height, width                                 */
    int32_t stride, pad, groups;
    int32_t H, W;               /* INPUT height, width; batch is always 1                        */
    int32_t in0;                /* producer layer index, -1 = model input; must be < own index   */
    int32_t in1;                /* residual addend's producer layer, -1 = none; < own index      */
    int32_t act;                /* 0 none, 1 ReLU, 2 ReLU6 -- applied after bias and addend      */
    int32_t has_bias;
    uint64_t w_off, b_off;      /* byte offsets of weights / bias in the host weight blob (256-B aligned) */
} nnv_layer_desc_t;

typedef struct {
    int32_t default_math;       /* nnv_math_t used where a caller passes -1; default TF32 */
    int32_t allow_cached;       /* default for selection; default 1                       */
    int32_t max_depth;          /* largest pipeline depth nnv_cold_run accepts; default 4 */
    int32_t kernel_stamps;      /* 1: the tensor-core GEMM kernels and the weight-transform kernels of every run record
                                   the device clock when their first block starts and their last block ends
                                   (two atomics per block); nnv_kernel_times reads the durations.  Default 0. */
    int32_t use_graphs;         /* 1: nnv_cold_run / nnv_resident_run record their stream work into a
                                   CUDA graph on the first call with a given argument set (choices,
                                   buffer addresses, depth) and replay it afterwards; 0: always enqueue
                                   call by call.  Calls that ask for timings never use a graph.        */
} nnv_plan_opts_t;

/* One row of the profiled cost table: the operation costs of one kernel of one
 * layer in integer nanoseconds (the paper's Table 2 has exactly these columns:
 * read raw, weights transformation, read cache, execution). */
typedef struct {
    int32_t layer, variant, math, reserved;
    uint64_t h2d_raw_ns, xform_ns, h2d_cached_ns, exec_ns;
    uint64_t zc_ns;             /* the fused preparation: the transform kernel reads the raw weights straight from pinned
                                   host memory, no copy before it (0 = not profiled / not offered) */
} nnv_cost_t;

/* One layer's kernel and how its weights are prepared.  cached: NNV_ARM_RAW = read raw weights, then
 * transform; NNV_ARM_CACHED = read cached post-transform weights (Section 3.1.2); NNV_ARM_ZERO_COPY = the
 * transform kernel reads the raw weights in place in pinned host memory and writes the transformed
 * weights to device memory (the paper bundles read and transform into one preparation operation,
 * Section 3.1.3; here they become one kernel, and the raw copy in device memory disappears). */
typedef struct { int32_t variant, math, cached; } nnv_choice_t;
#define NNV_ARM_RAW 0
#define NNV_ARM_CACHED 1
#define NNV_ARM_ZERO_COPY 2

/* Per-layer record of one cold run.  Start/end stamps are nanoseconds since the
 * run's first enqueue; 0/0 where the operation does not exist for the layer. */
typedef struct {
    uint64_t h2d_start_ns, h2d_end_ns;
    uint64_t xform_start_ns, xform_end_ns;
    uint64_t exec_start_ns, exec_end_ns;
    uint64_t h2d_bytes;         /* bytes copied host -> device for this layer              */
    uint64_t xform_bytes;       /* algorithmic bytes of the transform: raw read + written  */
    uint64_t exec_flops;        /* 2 * multiply-adds the chosen kernel performs            */
    nnv_choice_t choice;
    int32_t reserved;
} nnv_timing_t;

/* ---- plan -------------------------------------------------------------------------------- */

/* Build a plan from n layer descriptors (copied).  Validates shapes, producer
 * indices (topological order) and that every conv layer has at least one
 * eligible variant.  opts may be NULL.  The model abstraction is the paper's:
 * a list of layers, each with candidate kernels (input of its Algorithm 1). */
nnv_status_t nnv_plan_create(const nnv_layer_desc_t* layers, int32_t n,
                             const nnv_plan_opts_t* opts, nnv_plan_t** out);
/* Waits for work the plan itself still has in flight (the tail of a continuous-mode cold run:
 * reads and transforms of K_warm - K_cold), then releases events, graphs and the side stream. */
nnv_status_t nnv_plan_destroy(nnv_plan_t* plan);

/* Tuning overrides for experiments and sweeps (the paper's offline decision stage profiles
 * candidate kernels, Section 3.3; this lets a harness also profile candidate TILINGS of one
 * kernel).  Process-wide; read whenever a launch is planned; a recorded graph is tied to the
 * settings it was recorded under.  spec: "key=value;key=value", NULL or "" = all defaults.
 *   gemm_tile=BN,splits   column tile (16..128, multiple of 16) and K splits (1,2,4,8) of the GEMM
 *   gemm_ring=N           shared-memory ring depth 2..8        gemm_prefill=0|1
 *   conv3x3=off|auto|MT,BN,splits[,boxes,weight_tiles]          the halo-resident 3x3 kernel
 *   conv3x3p=off|BN,ctas_per_sm[,boxes,weight_tiles]           the persistent form of the 3x3 kernel (off unless asked for)
 *   conv3x3w=off|auto|on  the weights-stationary form of the 3x3 kernel (layers whose weight slice fits shared memory):
 *                         on = wherever it fits; auto and off = never (it measured slower than the one-tile kernel)
 *   bf16cvt=0|1           BF16-math GEMMs read the fp32 activation and round it inside the kernel (1, default) or
 *                         from an explicit bf16 im2col matrix (0)
 *   winofused=auto|0|1    F(2x2,3x3) with TF32 math as one kernel (input transform, tile GEMMs, output transform)
 *   smallp=0|1|N          the weights-on-rows kernel for layers of at most 256 pixels: off, on, on with N K splits
 *   side=0|1  merge=0|1  group=0|1   side stream for residual branches, merged reads, grouped transforms
 *   copies_first=0|1      merged reads are all put on the copy stream before the first kernel (1, default) or layer by layer
 *   chunk=first_kb,max_kb merged reads: size target of the first copy (>= 16) and the size the targets double up to
 * Every call replaces all settings (unnamed keys return to their defaults).  An item that does not
 * parse or is out of range -> NNV_ERR_INVALID_ARG and nothing changes; a setting that does not fit a
 * particular layer (more splits than K blocks, a tiling beyond shared memory) is ignored for it. */
nnv_status_t nnv_tuning_set(const char* spec);

/* Variants that can execute `layer`, ascending, written to out[0..*n_out).
 * Rules keyed on filter size, stride and grouping (the keys of the paper's
 * Figure 5 kernel tree).  cap < needed -> NNV_ERR_INVALID_ARG. */
nnv_status_t nnv_eligible(const nnv_plan_t* plan, int32_t layer,
                          int32_t* out, int32_t cap, int32_t* n_out);

/* Bytes of the transformed weights of (layer, variant, math); 0 for DIRECT /
 * DEPTHWISE.  This is also the size of the layer's cached post-transform blob
 * (the paper's Section 3.1.2: bypassing trades a larger read for no transform). */
nnv_status_t nnv_transformed_bytes(const nnv_plan_t* plan, int32_t layer,
                                   int32_t variant, int32_t math, uint64_t* bytes);

/* Scratch bytes nnv_conv_exec needs for (layer, variant, math). */
nnv_status_t nnv_exec_workspace_bytes(const nnv_plan_t* plan, int32_t layer,
                                      int32_t variant, int32_t math, uint64_t* bytes);

/* Arena bytes nnv_cold_run needs for these choices at pipeline depth `depth`. */
nnv_status_t nnv_arena_bytes(const nnv_plan_t* plan, const nnv_choice_t* choices,
                             int32_t depth, uint64_t* bytes);

/* Byte offset of every layer's transformed weights inside the cached blob that
 * nnv_cold_run reads for layers chosen with cached = 1 (0 for other layers);
 * *total = blob size.  Offsets are 256-byte aligned. */
nnv_status_t nnv_cached_layout(const nnv_plan_t* plan, const nnv_choice_t* choices,
                               uint64_t* offsets /* n layers */, uint64_t* total);

/* ---- selection (integer, exact) ------------------------------------------------------------ */

/* Candidate filter that opens the paper's Algorithm 1: of one layer's options
 * (each cost row gives a raw arm, prep = h2d_raw + xform; if the variant has a
 * transform and bit 0 of allow_cached is set a cached arm, prep = h2d_cached; if it
 * has a transform, bit 1 of allow_cached is set and zc_ns > 0 a zero-copy arm,
 * prep = zc_ns) drop every
 * option for which another is no slower in both prep and exec and faster in one;
 * of exact duplicates keep the lowest (variant, math, cached).  Survivors are
 * written in ascending (variant, math, cached) order. */
nnv_status_t nnv_filter_candidates(const nnv_plan_t* plan, int32_t layer,
                                   const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                                   nnv_choice_t* out, int32_t cap, int32_t* n_out);

/* Per conv layer pick the survivor with the least cold cost prep + exec (the
 * paper's Section 3.1.1 / 3.1.2 trade-off, its Table 2); ties go to the lowest
 * (variant, math, cached).  out has one entry per layer; pool layers get
 * {-1,-1,0}.  Rows naming a variant the layer cannot use -> NNV_ERR_INVALID_ARG;
 * a conv layer without rows -> NNV_ERR_STATE. */
nnv_status_t nnv_select_kernels(const nnv_plan_t* plan, const nnv_cost_t* costs, int32_t n_costs,
                                int32_t allow_cached, nnv_choice_t* out);

/* The warm kernel set K_warm of the paper's Section 3.5: per conv layer the
 * (variant, math) with the least exec_ns among its cost rows -- with every
 * weight already prepared only execution counts; ties go to the lowest
 * (variant, math).  out[i].cached = 1 when that kernel reads transformed weights
 * (which then stay resident), 0 when it reads raw ones; pool layers {-1,-1,0}.
 * Errors as nnv_select_kernels. */
nnv_status_t nnv_select_warm(const nnv_plan_t* plan, const nnv_cost_t* costs, int32_t n_costs,
                             nnv_choice_t* out);

/* K_warm - K_cold (Section 3.5): the layers whose warm kernel differs from the
 * cold one in (variant, math) and has a transform -- the weights that remain to
 * be prepared once the cold inference has what it needs.  Ascending layer order. */
nnv_status_t nnv_switch_set(const nnv_plan_t* plan, const nnv_choice_t* cold, const nnv_choice_t* warm,
                            int32_t* layers_out, int32_t cap, int32_t* n_out);

/* ---- scheduling (integer, exact; host only) -------------------------------------------------- */

/* Cold latency of one assignment (the paper's Eq. (1)-(2), Section 3.2): the end
 * of the last execution when queue 0 runs every execution in layer order plus the
 * preparation (read + transform, or read of cached weights) of the conv layers
 * with queue_of = 0, each directly before its execution, and queues 1..n_little
 * run the other preparations in layer order.  An execution starts when queue 0 is
 * free, its preparation has ended and the layers in0/in1 have executed.  All
 * arrays are host arrays with one entry per layer; prep entries and queue_of of
 * pool layers are ignored.  prep_big_ns is the preparation time on queue 0,
 * prep_little_ns on any other queue.  n_little in 1..NNV_MAX_QUEUES; a conv layer's queue
 * outside 0..n_little -> NNV_ERR_INVALID_ARG. */
nnv_status_t nnv_simulate(const nnv_plan_t* plan, const uint64_t* prep_little_ns, const uint64_t* prep_big_ns,
                          const uint64_t* exec_ns, const int32_t* queue_of, int32_t n_little,
                          uint64_t* t_cold_ns);

/* The body of the paper's Algorithm 1 for one kernel combination.  B starts as
 * the first conv layer.  The preparations outside B are dealt round-robin to the
 * little queues and balanced: while the longest and shortest queue differ by more
 * than eps_ns, every operation of the longest (longest first) that is shorter
 * than half the current gap moves to the shortest.  While the longest little
 * queue outlasts queue 0 (preparations of B + all executions) by more than
 * eps_ns, the first layer outside B whose big + little preparation time is below
 * that gap joins B and the little queues are dealt again.  Writes the queue of
 * every layer's preparation (-1 for pool layers) and the resulting nnv_simulate
 * value.  Same argument rules as nnv_simulate. */
nnv_status_t nnv_schedule_queues(const nnv_plan_t* plan, const uint64_t* prep_little_ns,
                                 const uint64_t* prep_big_ns, const uint64_t* exec_ns, int32_t n_little,
                                 uint64_t eps_ns, int32_t* queue_of, uint64_t* t_cold_ns);

/* The whole of Algorithm 1: over the combinations of each conv layer's
 * nnv_filter_candidates survivors, the one whose nnv_schedule_queues latency is
 * least.  An option's little-queue preparation time is its prep, its queue-0 time
 * prep * big_pct / 100 (rounded down).  pool_ns: execution time of the pool
 * layers (NULL = 0).  Up to combo_limit combinations are tried exhaustively (last
 * layer varying fastest; a tie keeps the earlier one); beyond that, coordinate
 * descent from nnv_select_kernels' choice: layer by layer, adopt the first
 * survivor in (variant, math, cached) order that strictly lowers the latency,
 * until a sweep changes nothing (at most 8 sweeps).  out / queue_of: one entry per
 * layer (pool layers {-1,-1,0} / -1).  Errors as nnv_select_kernels. */
nnv_status_t nnv_schedule(const nnv_plan_t* plan, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                          const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                          uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns);

/* The same latency for a machine on which the weights of EVERY queue arrive over one host
 * link (the paper's Eq. (1)-(2) give each queue its own processor for the whole bundled
 * preparation; on a discrete GPU all reads share the PCIe link, whatever stream issues them).
 * A preparation is two operations on its queue, a read (read_ns) and then a transform
 * (xform_little_ns, or xform_big_ns on queue 0).  The link carries one read at a time; a read
 * waits from the moment the operation before it on its queue has ended; a free link takes the
 * waiting read of the lowest layer (reads are issued in layer order).  Executions and the order
 * inside the queues are as in nnv_simulate, which this call equals when every read_ns is 0. */
nnv_status_t nnv_simulate_link(const nnv_plan_t* plan, const uint64_t* read_ns, const uint64_t* xform_little_ns,
                               const uint64_t* xform_big_ns, const uint64_t* exec_ns, const int32_t* queue_of,
                               int32_t n_little, uint64_t* t_cold_ns);

/* nnv_schedule, except that a combination's latency -- what the search minimises and what
 * *t_cold_ns returns -- is nnv_simulate_link's: read = the option's h2d_raw_ns or
 * h2d_cached_ns, transform = xform_ns (0 for a cached option; x big_pct / 100 on queue 0).
 * The queues of a combination still come from nnv_schedule_queues on the bundled times. */
nnv_status_t nnv_schedule_link(const nnv_plan_t* plan, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                               const uint64_t* pool_ns, int32_t n_little, uint64_t eps_ns, int32_t big_pct,
                               uint64_t combo_limit, nnv_choice_t* out, int32_t* queue_of, uint64_t* t_cold_ns);

/* Algorithm 1's epsilon (the listing leaves it open): eps_pct percent, rounded down, of the
 * summed execution time of nnv_select_kernels' per-layer choice. */
nnv_status_t nnv_schedule_eps(const nnv_plan_t* plan, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                              int32_t eps_pct, uint64_t* eps_ns);

/* Algorithm 1's profiling step, repeated under load (the paper's Section 3.3 notes that
 * operations running beside each other interfere): given the timings of one run of a schedule
 * (nnv_cold_run_queues with timings), rescale the isolated cost table by how much slower each
 * KIND of operation ran than it did alone.  For kind k in (read, transform, execution):
 * num_k = sum over the conv layers of the run's measured interval, den_k = sum of the chosen
 * kernels' isolated costs (read: h2d_cached_ns if the choice read cached weights, else
 * h2d_raw_ns; transform: only layers that transformed).  Every row's costs of kind k become
 * floor(cost * num_k / den_k), exactly; a kind with num_k = 0 or den_k = 0 is left alone, and
 * so is a kind whose bit in `kinds` is clear (1 read, 2 transform, 4 execution): a table meant
 * for nnv_schedule_link keeps its isolated read costs, because there the reads' waiting for one
 * another -- which a measured read interval includes -- is what the link model itself adds.
 * Scaling by kind, not by kernel, keeps options that did not run from looking cheaper than
 * those that did.  out: n_costs rows (may alias costs).  factors: NULL or 6 values
 * {num, den} x {read, transform, execution}.  A chosen kernel without a row -> NNV_ERR_STATE. */
nnv_status_t nnv_calibrate_costs(const nnv_plan_t* plan, const nnv_cost_t* costs, int32_t n_costs,
                                 const nnv_choice_t* choices, const nnv_timing_t* timings, int32_t kinds,
                                 nnv_cost_t* out, uint64_t* factors);

/* ---- single operations (asynchronous on `stream`) ------------------------------------------ */

/* Weights transformation (the paper's Section 2 stage, Figure 3): Winograd
 * filter transform U = G g G^T for WINO_F2/F4/F6, or the GEMM-ready repack for
 * IM2COL / GEMM1X1.  d_raw: the layer's raw OIHW fp32 weights.  d_out:
 * nnv_transformed_bytes() bytes.  DIRECT / DEPTHWISE -> NNV_ERR_UNSUPPORTED. */
nnv_status_t nnv_transform_weights(const nnv_plan_t* plan, int32_t layer, int32_t variant, int32_t math,
                                   const void* d_raw, void* d_out, void* stream);

/* The weights transformation of EVERY layer in one launch (the paper's decision
 * stage writes all post-transformed weights out once, its Section 3.1.2; the
 * same job builds the cached blob here).  d_weights: device copy of the weight
 * blob (raw weights at w_off).  d_out: nnv_transformed_layout() bytes; layer i's
 * transformed weights land at offsets[i] (256-byte aligned; 0 for layers without
 * a transform).  Bit-identical to calling nnv_transform_weights per layer. */
nnv_status_t nnv_transformed_layout(const nnv_plan_t* plan, const nnv_choice_t* choices,
                                    uint64_t* offsets /* n layers */, uint64_t* total);
nnv_status_t nnv_transform_all(const nnv_plan_t* plan, const nnv_choice_t* choices,
                               const void* d_weights, uint64_t w_bytes,
                               void* d_out, uint64_t out_bytes, void* stream);

/* Execute one conv layer (the paper's "execution" operation) with the given
 * kernel.  d_in: NHWC fp32 input (H x W x C).  d_addend: NHWC fp32 residual of
 * the output's shape or NULL.  d_wt: transformed weights of this (variant, math),
 * or the raw weights for DIRECT / DEPTHWISE.  d_bias: K floats or NULL.
 * d_out: NHWC fp32 (OH x OW x K).  d_ws: scratch of at least
 * nnv_exec_workspace_bytes() bytes (may be NULL when that is 0). */
nnv_status_t nnv_conv_exec(const nnv_plan_t* plan, int32_t layer, int32_t variant, int32_t math,
                           const void* d_in, const void* d_addend, const void* d_wt, const void* d_bias,
                           void* d_out, void* d_ws, uint64_t ws_bytes, void* stream);

/* The data transforms around the Winograd tile GEMM as single operations (nnv_conv_exec with a
 * WINO variant runs input transform, batched tile GEMM and output transform back to back; the
 * paper's engine does the same inside its winograd kernels, Section 2 / Figure 3 name only the
 * weight side).  Tiles of alpha x alpha input pixels at stride m, starting at -pad, zero outside
 * the image; tile t = th * TW + tw, TH = ceil(OH / m), TW = ceil(OW / m).
 *   nnv_wino_sizes: tiles T and the bytes of V and M for (layer, variant, math).
 *   nnv_wino_input_transform: d_in NHWC fp32 -> d_V[xi*alpha+nu][t][cp] = (B^T d B)[xi][nu], cp < Cp
 *       (entries with cp >= C are +0); element type fp32, or bf16 with BF16 math; for F(2x2,3x3)
 *       with TF32 math the fp32 words are rounded to TF32 precision (nearest even), since one TF32
 *       pass multiplies them.
 *   nnv_wino_output_transform: d_M[xi*alpha+nu][t][k] fp32 -> d_out NHWC fp32: each tile's
 *       A^T M A, clipped to the output grid, + bias + addend, then the layer's activation.
 * Asynchronous on `stream`; pointers 256-byte aligned. */
nnv_status_t nnv_wino_sizes(const nnv_plan_t* plan, int32_t layer, int32_t variant, int32_t math,
                            int32_t* tiles, uint64_t* v_bytes, uint64_t* m_bytes);
nnv_status_t nnv_wino_input_transform(const nnv_plan_t* plan, int32_t layer, int32_t variant, int32_t math,
                                      const void* d_in, void* d_V, void* stream);
nnv_status_t nnv_wino_output_transform(const nnv_plan_t* plan, int32_t layer, int32_t variant,
                                       const void* d_M, const void* d_addend, const void* d_bias, void* d_out, void* stream);

/* nnv_conv_exec without a scratch argument.  (The paper has no counterpart to
 * this call; it is a convenience of this library.)  It is for callers that cannot
 * hand over device scratch because they cannot allocate any: a plug-in inside an
 * application that owns all device memory, a latency-bound loop that must avoid
 * cudaMalloc's device-wide synchronisation, set-up code that runs before a memory
 * pool exists.  The scratch is a fixed array of NNV_STATIC_SCRATCH_BYTES compiled
 * into the library; every GPU that loads the library holds that much memory until
 * the process ends.  The call allocates and frees nothing.
 *   - Same arguments, layouts, alignment rules and result as nnv_conv_exec; inputs
 *     and outputs are still the caller's.
 *   - A (layer, variant, math) whose nnv_exec_workspace_bytes() exceeds
 *     NNV_STATIC_SCRATCH_BYTES is refused with NNV_ERR_WORKSPACE_TOO_SMALL before
 *     anything is launched; use nnv_conv_exec with your own buffer for those.
 *   - The first call on each device (with that device current) looks up the
 *     array's device address; make that first call before any stream capture
 *     begins on the device.  Later calls only enqueue kernels.
 *   - All calls on a device share the one array, and it keeps whatever the last
 *     call left in it.  Nothing in it has to start at zero -- every kernel of the
 *     chain fully writes what the next one reads -- so it is never cleared.  Two
 *     calls whose kernels may overlap on the GPU (different streams without an
 *     ordering between them) race on it: serialise them. */
#define NNV_STATIC_SCRATCH_BYTES (16u << 20)
nnv_status_t nnv_conv_exec_static(const nnv_plan_t* plan, int32_t layer, int32_t variant, int32_t math,
                                  const void* d_in, const void* d_addend, const void* d_wt, const void* d_bias,
                                  void* d_out, void* stream);

/* Max-pool / global-average-pool layer, NHWC fp32 in and out. */
nnv_status_t nnv_pool_exec(const nnv_plan_t* plan, int32_t layer,
                           const void* d_in, void* d_out, void* stream);

/* fp32 layout conversion between the host convention (CHW) and the device one (HWC). */
nnv_status_t nnv_chw_to_hwc(const float* d_in, float* d_out, int32_t C, int32_t H, int32_t W, void* stream);
nnv_status_t nnv_hwc_to_chw(const float* d_in, float* d_out, int32_t C, int32_t H, int32_t W, void* stream);

/* ---- whole-model cold run ------------------------------------------------------------------ */

/* One cold inference: for every conv layer copy its weights from pinned host
 * memory (stream s_copy), transform them (s_xform) and execute the layer
 * (s_exec), pipelined so that layer i+1.. are prepared while layer i executes
 * (the paper's Section 3.1.3).  Preparation of conv layer j may start only
 * after the execution of conv layer j-depth has finished (depth staging slots);
 * depth = 1 is the fully serial order read, transform, execute per layer;
 * depth = 0 lifts the limit: every layer gets its own raw and transformed buffer
 * in the arena and preparation never waits for execution (the paper's pipeline,
 * whose little cores run ahead freely).
 *   h_weights: pinned host blob holding raw weights / biases at w_off / b_off.
 *   h_cached:  pinned host blob of cached transformed weights laid out by
 *              nnv_cached_layout(); may be NULL if no choice has cached = 1.
 *   h_input / h_output: NCHW fp32 host buffers (pinned recommended); h_output
 *              receives the LAST layer's output.
 *   d_arena:   nnv_arena_bytes() bytes of device memory.
 *   timings:   NULL, or n entries filled from CUDA events (adds event records).
 * At depth 0 consecutive layers whose host and arena ranges line up are read by one
 * copy (256 KB at first, doubling up to 16 MB, the last layer by itself; the
 * per-layer timings then share that copy's interval, and the layers' weight
 * transforms are one grouped launch), and all these copies are put on s_copy,
 * in layer order, before the first kernel is enqueued, so that the host link
 * never waits for the host (nnv_tuning_set: chunk, copies_first, merge).
 * A conv layer whose output is only ever the residual addend of a later layer
 * and which needs no execution scratch runs on a fourth stream that the plan
 * creates and owns, beside the main branch; the result is the same bit for bit.
 * Synchronises the three streams before returning. */
nnv_status_t nnv_cold_run(nnv_plan_t* plan, const nnv_choice_t* choices,
                          const void* h_weights, uint64_t w_bytes,
                          const void* h_cached, uint64_t c_bytes,
                          const float* h_input, float* h_output,
                          void* d_arena, uint64_t arena_bytes,
                          void* s_copy, void* s_xform, void* s_exec,
                          int32_t depth, nnv_timing_t* timings);

/* nnv_cold_run for a caller whose activations already live on the GPU (an upstream stage
 * produced the input there, a downstream stage consumes the output there): d_input / d_output
 * are DEVICE NCHW fp32 buffers (256-byte aligned).  The weights still take the whole path of
 * the paper's Section 2 -- read from pinned host memory, transformed, executed; only the two
 * activation copies across the host link are gone.  Everything else as nnv_cold_run. */
nnv_status_t nnv_cold_run_dio(nnv_plan_t* plan, const nnv_choice_t* choices,
                              const void* h_weights, uint64_t w_bytes,
                              const void* h_cached, uint64_t c_bytes,
                              const float* d_input, float* d_output,
                              void* d_arena, uint64_t arena_bytes,
                              void* s_copy, void* s_xform, void* s_exec,
                              int32_t depth, nnv_timing_t* timings);

/* One cold inference on the queues Algorithm 1 produced.  queue_of (one entry
 * per layer, as written by nnv_schedule / nnv_schedule_queues) names the queue of
 * every conv layer's bundled preparation -- the copy of its raw (or cached)
 * weights followed by the transform, if any, on ONE stream: queue 0 is the
 * execution stream streams[0], where the preparation sits directly before the
 * layer's execution (the paper's big cores taking over preparation work); queue
 * j >= 1 is streams[j] (its little cores), which runs its preparations in layer
 * order and never waits for execution.  streams: n_little + 1 distinct CUDA
 * streams, n_little in 1..NNV_MAX_QUEUES.  The arena is the depth-0 one
 * (nnv_arena_bytes with depth 0).  Other arguments, results and errors as
 * nnv_cold_run; the output is bit-identical to nnv_cold_run's for the same
 * choices.  Synchronises every stream before returning. */
#define NNV_MAX_QUEUES 16
nnv_status_t nnv_cold_run_queues(nnv_plan_t* plan, const nnv_choice_t* choices,
                                 const int32_t* queue_of, int32_t n_little,
                                 const void* h_weights, uint64_t w_bytes,
                                 const void* h_cached, uint64_t c_bytes,
                                 const float* h_input, float* h_output,
                                 void* d_arena, uint64_t arena_bytes,
                                 void* const* streams, nnv_timing_t* timings);

/* The same pass with the read stage already done (the paper's Tables 1 and 2
 * separate reading from transformation and execution; this call measures the
 * latter two alone).  d_weights / d_cached are DEVICE copies of the two blobs
 * (256-byte aligned), d_input / d_output are DEVICE NCHW fp32 buffers; nothing
 * crosses the host link.  Transforms run on s_xform, layers on s_exec; the
 * transform of conv layer j waits for the execution of conv layer j-depth.  With
 * depth = 0 nothing orders the transforms, and they are issued as two multi-layer
 * launches (the first layers, then all the rest) instead of one per layer. */
nnv_status_t nnv_resident_run(nnv_plan_t* plan, const nnv_choice_t* choices,
                              const void* d_weights, uint64_t w_bytes,
                              const void* d_cached, uint64_t c_bytes,
                              const float* d_input, float* d_output,
                              void* d_arena, uint64_t arena_bytes,
                              void* s_xform, void* s_exec,
                              int32_t depth, nnv_timing_t* timings);

/* Continuous mode (the paper's Section 3.5: a cold inference that will be
 * followed by more).  nnv_cold_run_continuous is nnv_cold_run with depth 0 for
 * the kernels `cold`, except that what it prepares stays: raw weights and biases
 * are read into d_warm (same offsets as in the host blob), and a layer whose cold
 * kernel is also its warm kernel writes its transformed weights into d_warm's
 * transformed region (nnv_cached_layout order, after the raw copy rounded up to
 * 1 KiB).  For the layers of nnv_switch_set(cold, warm) -- and for warm kernels
 * that need raw weights the cold run did not read -- the read and the warm
 * kernel's transform are queued on s_copy / s_xform BEHIND everything the cold
 * inference needs, so they use the time those streams would idle while the last
 * layers execute.  The call returns when h_output holds the cold result; these
 * preparations may still be running.  nnv_warm_run then executes K_warm from
 * d_warm (input and output on the host, nothing else crosses the link); the
 * first call after nnv_cold_run_continuous makes each layer wait for its own
 * preparation, i.e. the rest is pipelined into the second inference; later
 * calls wait for nothing and replay a recorded graph.
 *   d_warm: nnv_warm_bytes() bytes of device memory, the caller's, kept for as
 *           long as warm runs follow.  warm[i].cached is ignored.
 *   h_weights (and h_cached) must stay valid and unchanged until the first nnv_warm_run
 *           after this call has returned (or until s_copy and s_xform have been
 *           synchronised): the queued reads still copy from them.
 *   Results are bit-identical to nnv_cold_run with the same kernels. */
nnv_status_t nnv_warm_bytes(const nnv_plan_t* plan, const nnv_choice_t* warm, uint64_t w_bytes, uint64_t* bytes);
nnv_status_t nnv_cold_run_continuous(nnv_plan_t* plan, const nnv_choice_t* cold, const nnv_choice_t* warm,
                                     const void* h_weights, uint64_t w_bytes,
                                     const void* h_cached, uint64_t c_bytes,
                                     const float* h_input, float* h_output,
                                     void* d_arena, uint64_t arena_bytes,
                                     void* d_warm, uint64_t warm_bytes,
                                     void* s_copy, void* s_xform, void* s_exec,
                                     nnv_timing_t* timings);
nnv_status_t nnv_warm_run(nnv_plan_t* plan, const nnv_choice_t* warm,
                          const void* d_warm, uint64_t warm_bytes, uint64_t w_bytes,
                          const float* h_input, float* h_output,
                          void* d_arena, uint64_t arena_bytes,
                          void* s_xform, void* s_exec, nnv_timing_t* timings);

/* ---- model file: what the decision stage leaves in storage ----------------------------------- */

/* The paper's decision stage writes a kernel scheduling plan and the
 * post-transformed weights to storage (its Sections 3 and 3.1.2; Table 4 counts
 * the storage overhead); the cold inference starts by reading weights from
 * there (Section 2, "weights reading").  The paper prints no file layout; this
 * library's is (all integers little-endian):
 *   header, 64 bytes: 8 bytes magic "NNV12WC\0", u32 version = 1, u32 n_layers,
 *       u64 w_bytes, u64 c_bytes, u64 raw_off = round_up(64 + 88 n_layers, 4096),
 *       u64 cached_off = raw_off + round_up(w_bytes, 4096), u32 n_little, u32 0,
 *       u64 FNV-1a (64 bit) of the two tables;
 *   layer table, 72 bytes per layer: nnv_layer_desc_t as declared above;
 *   plan table, 16 bytes per layer: i32 variant, math, cached, queue
 *       (-1, -1, 0, -1 for pool layers; queue -1 when no schedule is stored);
 *   zero padding; the raw weight blob at raw_off; zero padding; the cached blob
 *   (nnv_cached_layout of the stored choices) at cached_off; zero padding to a
 *   multiple of 4096.
 * nnv_cache_write creates / replaces `path` from host buffers and fsyncs it.
 * queue_of / n_little: a schedule from nnv_schedule, or NULL / 0.  h_cached may be
 * NULL when no stored choice has cached = 1.  I/O failures -> NNV_ERR_STATE. */
nnv_status_t nnv_cache_write(const char* path, const nnv_plan_t* plan, const nnv_choice_t* choices,
                             const int32_t* queue_of, int32_t n_little,
                             const void* h_weights, uint64_t w_bytes,
                             const void* h_cached, uint64_t c_bytes);

/* Open a model file and check it: magic, version, offsets against the file
 * size, table hash (anything wrong -> NNV_ERR_INVALID_ARG; cannot open / read
 * -> NNV_ERR_STATE).  The blobs are not read.  Close with nnv_cache_close. */
nnv_status_t nnv_cache_open(const char* path, nnv_cache_t** out);
nnv_status_t nnv_cache_close(nnv_cache_t* cache);
/* Sizes stored in the header; any output pointer may be NULL. */
nnv_status_t nnv_cache_info(const nnv_cache_t* cache, int32_t* n_layers, uint64_t* w_bytes, uint64_t* c_bytes,
                            int32_t* n_little, uint64_t* file_bytes);
/* The stored layer descriptors, choices and (if queue_of != NULL) queues; cap = entries per array. */
nnv_status_t nnv_cache_read_plan(const nnv_cache_t* cache, nnv_layer_desc_t* layers, nnv_choice_t* choices,
                                 int32_t* queue_of, int32_t cap);
/* Read the whole raw blob (and, if h_cached != NULL, the cached blob) into host buffers. */
nnv_status_t nnv_cache_read_blobs(const nnv_cache_t* cache, void* h_weights, uint64_t w_cap,
                                  void* h_cached, uint64_t c_cap);
/* Ask the operating system to drop the file's pages from its cache
 * (posix_fadvise DONTNEED), so that the next reads come from the device again:
 * the paper clears caches before each cold run.  Best effort. */
nnv_status_t nnv_cache_drop_pages(const nnv_cache_t* cache);

/* nnv_cold_run with the weights still in storage: a reader thread walks the
 * layers in order and reads, from the open model file into the PINNED staging
 * buffers, exactly the bytes each layer's choice consumes (its cached blob entry
 * if cached = 1, else its raw weights; its bias), and each layer's host->device
 * copy is issued as soon as its bytes have arrived -- storage -> host memory
 * becomes a fourth pipeline stage in front of copy, transform and execution.
 *   h_stage_weights: pinned, >= the file's w_bytes; h_stage_cached: pinned, >= the
 *       cached bytes these choices read, or NULL if none is cached.
 *   Layers read with cached = 1 must be stored in the file with the same kernel
 *       and at the same cached-blob offset, else NNV_ERR_INVALID_ARG.
 *   read_ns / read_bytes (nullable): wall time the reader took and bytes it read.
 * Everything else as nnv_cold_run; the result is bit-identical to it. */
nnv_status_t nnv_cold_run_file(nnv_plan_t* plan, const nnv_choice_t* choices, const nnv_cache_t* cache,
                               void* h_stage_weights, uint64_t stage_w_bytes,
                               void* h_stage_cached, uint64_t stage_c_bytes,
                               const float* h_input, float* h_output,
                               void* d_arena, uint64_t arena_bytes,
                               void* s_copy, void* s_xform, void* s_exec, int32_t depth,
                               nnv_timing_t* timings, uint64_t* read_ns, uint64_t* read_bytes);

/* Device address, inside the arena of the most recent nnv_cold_run on this
 * plan, of layer `layer`'s NHWC fp32 output (valid until the arena is reused). */
nnv_status_t nnv_layer_output(const nnv_plan_t* plan, int32_t layer, const void** d_ptr, uint64_t* bytes);

/* Host time, in nanoseconds, that the most recent run on this plan (nnv_cold_run and its
 * variants, nnv_resident_run, nnv_warm_run) spent putting its work on the streams: every API
 * call of an eager run, or the one graph launch of a replayed one.  When this exceeds the
 * device time of the run, the host and not the GPU or the link bounds the cold latency. */
nnv_status_t nnv_last_enqueue_ns(const nnv_plan_t* plan, uint64_t* ns);

/* Device time of the kernels of the most recent run on a plan created with kernel_stamps = 1,
 * per layer, in nanoseconds of the device clock: xform_ns[i] = from the first block's start to the
 * last block's end of layer i's weight-transform launch (a grouped launch is booked on the first
 * layer of its group, the others get 0), exec_ns[i] = the same for the layer's tensor-core GEMM
 * kernel (0 for layers executed by other kernels).  Unlike event pairs around a kernel, which add
 * microseconds of their own and serialise the streams, the stamps do not disturb the run they
 * measure.  Both arrays hold one entry per layer; either may be NULL.  Synchronises the device. */
nnv_status_t nnv_kernel_times(const nnv_plan_t* plan, uint64_t* xform_ns, uint64_t* exec_ns);

/* The same stamps as a timeline: xform_span[2i], xform_span[2i+1] = start and end of layer i's
 * weight-transform launch, exec_span[2i], exec_span[2i+1] = the same for its tensor-core GEMM
 * kernel, in nanoseconds of the device clock counted from the earliest stamped start of the run
 * (0, 0 where no stamped kernel ran for the layer).  A transform starts when its copy has landed,
 * so the spans show where a cold run (Section 3.1.3: read, transform and execution of different
 * layers overlapping) waits for the link and where for the kernels.  Both arrays hold two entries
 * per layer; either may be NULL.  Synchronises the device. */
nnv_status_t nnv_kernel_spans(const nnv_plan_t* plan, uint64_t* xform_span, uint64_t* exec_span);

/* Profile every eligible (variant, math) of every conv layer in isolation --
 * the per-operation profiling that feeds the paper's Algorithm 1 -- and write
 * one cost row each: median of `reps` timed repetitions, CUDA events, integer
 * nanoseconds.  Layer inputs are the activations left in the arena by running
 * the model once with DIRECT/IM2COL kernels.  d_arena: nnv_profile_arena_bytes(). */
nnv_status_t nnv_profile_arena_bytes(const nnv_plan_t* plan, uint64_t* bytes);
nnv_status_t nnv_profile(nnv_plan_t* plan, const void* h_weights, uint64_t w_bytes,
                         const float* h_input, void* d_arena, uint64_t arena_bytes,
                         void* stream, int32_t reps,
                         nnv_cost_t* out, int32_t cap, int32_t* n_out);

/* ---- diagnostics --------------------------------------------------------------------------- */

/* Read and clear the device-side status word that kernels with bounded waits
 * set when a wait gives up.  Synchronises the device.  *code = 0 when clean. */
nnv_status_t nnv_device_status(int32_t* code);

const char* nnv_last_error(void);   /* valid until the next failing call on this thread */
int32_t nnv_version(void);

#ifdef __cplusplus
}
#endif
#endif /* NNV_H_ */
