// Batched tensor-core GEMM for sm_100a:  D[b][M][N] = A[b][M][Kd] * B[b][N][Kd]^T.
//
// Both operands are K-major (row-major with the reduction index innermost), which is how the
// Winograd tile GEMM (V[xi,nu][T][C] x U[xi,nu][K][C]), the im2col GEMM (Xcol[P][Q] x P[K][Q])
// and the 1x1 GEMM (X[P][C] x W[K][C]) all present themselves.  Pixels / tiles sit on the MMA's
// M dimension (128 TMEM lanes), output channels on N.
//
// Structure of one CTA (one 128 x BN output tile, 192 threads):
//   warp 0   TMA producer: cp.async.bulk.tensor loads of 128-byte-wide K slices of A and B into a
//            ring of shared-memory stages (128B swizzle), completion on "full" mbarriers
//   warp 1   allocates TMEM, issues tcgen05.mma (one lane) from shared-memory descriptors into
//            the fp32 accumulator in TMEM, releases stages with tcgen05.commit on "empty" mbarriers
//   warps 2-5  epilogue: tcgen05.ld the accumulator (each warp its own 32 TMEM lanes), apply
//            bias / residual / activation, store fp32 rows
// Every mbarrier wait is bounded; a wait that gives up records NNV_ERR_TIMEOUT in a device status
// word and the CTA drains and exits instead of hanging.
#include <cuda.h>
#include <cudaTypedefs.h>
#include <cuda_bf16.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <mutex>

#include "nnv_internal.h"

namespace nnv {

__device__ int g_device_status = 0;

nnv_status_t read_device_status(int32_t* code) {
    NNV_CUDA(cudaDeviceSynchronize());
    int v = 0;
    NNV_CUDA(cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)));
    if (v != 0) {
        int zero = 0;
        NNV_CUDA(cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)));
    }
    *code = v;
    return NNV_OK;
}

__device__ unsigned long long g_stamps[2 * STAMP_SLOTS_PER_LAYER * STAMP_MAX_LAYERS];

unsigned long long*& next_stamp() {
    static thread_local unsigned long long* p = nullptr;
    return p;
}

nnv_status_t stamps_device_base(unsigned long long** base) {
    void* ptr = nullptr;
    NNV_CUDA(cudaGetSymbolAddress(&ptr, g_stamps));
    *base = static_cast<unsigned long long*>(ptr);
    return NNV_OK;
}

nnv_status_t enqueue_status_read(int* h_pinned, cudaStream_t st) {
    NNV_CUDA(cudaMemcpyFromSymbolAsync(h_pinned, g_device_status, sizeof(int), 0, cudaMemcpyDeviceToHost, st));
    return NNV_OK;
}

namespace {

constexpr int BM = 128;                 // rows of A per tile = TMEM lanes
constexpr int BK_BYTES = 128;           // bytes of K per stage row = one 128B swizzle atom
constexpr int A_STAGE_BYTES = BM * BK_BYTES;
constexpr int GEMM_THREADS = 192;
constexpr uint32_t WAIT_LIMIT = 1u << 20;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false when the limit ran out (the caller records a timeout and bails out).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < WAIT_LIMIT; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}

// im2col-mode load: `pixelsPerColumn` consecutive output pixels starting at the filter window whose
// top-left input coordinate is (w, h), each shifted by the tap offset (off_w, off_h); channels
// [c, c + channelsPerPixel).  Positions outside the image read as zero.
__device__ __forceinline__ void tma_load_im2col_4d(uint32_t dst, const CUtensorMap* map, int c, int w, int h, int n,
                                                   uint16_t off_w, uint16_t off_h, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.im2col.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6], {%7, %8};"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c), "r"(w), "r"(h), "r"(n), "r"(bar), "h"(off_w), "h"(off_h)
        : "memory");
}

// Tile store shared -> global through the tensor map (rows / columns outside the tensor are clipped).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
                 ::"l"(reinterpret_cast<uint64_t>(map)), "r"(src), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}
__device__ __forceinline__ void tma_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// All of this thread's tile stores have finished READING shared memory (the global writes complete with the grid).
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }

// Barrier over every thread of every CTA in the cluster (release / acquire).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows 128 bytes apart,
// 8-row groups 1024 bytes apart (stride byte offset), descriptor version 1.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;                     // leading byte offset (unused for swizzled K-major)
    d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset
    d |= (uint64_t)1 << 46;                     // version
    d |= (uint64_t)2 << 61;                     // SWIZZLE_128B
    return d;
}

template <bool BF16>
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if constexpr (BF16) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}

__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

struct GemmDev {
    unsigned long long* stamp;        // device-clock stamps of this launch, or null
    float* D;
    const float* bias;
    const float* addend;
    long long ldd, strideD;
    int M, N, Kd, BN, act, tmem_cols, splits, stages, prefill;
    int tma_out;                      // 0: plain stores; else the column width (16 or 32) of the staged tiles stored by TMA
    uint32_t stage_off;               // byte offset (from the aligned base) of the dedicated staging tile; 0 = the idle ring
    // implicit im2col (A is the NHWC activation itself): 0 = off
    int ic_on, ic_C, ic_cblk, ic_S, ic_OW, ic_stride, ic_pad;
};

__device__ __forceinline__ float act_fn(float v, int act) {
    if (act == 1) return fmaxf(v, 0.f);
    if (act == 2) return fminf(fmaxf(v, 0.f), 6.f);
    return v;
}

// Descriptor for the un-swizzled K-major layout used by the converted bf16 tiles: 8x16-byte core
// matrices, `lbo` bytes between core matrices adjacent in K, `sbo` bytes between 8-row groups.
__device__ __forceinline__ uint64_t make_smem_desc_plain(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;                     // version; layout type 0 = no swizzle
    return d;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Split eight fp32 values into bf16 hi = rn(x) and lo = rn(x - hi), packed as two 16-byte chunks.
__device__ __forceinline__ void split8(const float4& a, const float4& b, uint4& hi, uint4& lo) {
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint32_t h[4], l[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const __nv_bfloat16 h0 = __float2bfloat16_rn(x[2 * i]), h1 = __float2bfloat16_rn(x[2 * i + 1]);
        const __nv_bfloat16 l0 = __float2bfloat16_rn(x[2 * i] - __bfloat162float(h0));
        const __nv_bfloat16 l1 = __float2bfloat16_rn(x[2 * i + 1] - __bfloat162float(h1));
        h[i] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
        l[i] = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
    }
    hi = make_uint4(h[0], h[1], h[2], h[3]);
    lo = make_uint4(l[0], l[1], l[2], l[3]);
}

// Converts one row (32 fp32 = 128 bytes, stored by TMA with the 128-byte swizzle) of a staged tile
// into the hi and lo bf16 tiles (un-swizzled core-matrix layout, `rows` rows tall).
__device__ __forceinline__ void convert_row(uint32_t src_tile, uint32_t hi_tile, uint32_t lo_tile, int r, int rows) {
    const uint32_t src = src_tile + (uint32_t)r * 128u;
    const uint32_t lbo = (uint32_t)rows * 16u;
#pragma unroll
    for (int c = 0; c < 4; ++c) {                              // 4 chunks of 8 K-elements
        float4 v0, v1;
        const uint32_t a0 = src + ((uint32_t)((2 * c) ^ (r & 7)) << 4), a1 = src + ((uint32_t)((2 * c + 1) ^ (r & 7)) << 4);
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v0.x), "=f"(v0.y), "=f"(v0.z), "=f"(v0.w) : "r"(a0));
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v1.x), "=f"(v1.y), "=f"(v1.z), "=f"(v1.w) : "r"(a1));
        uint4 hi, lo;
        split8(v0, v1, hi, lo);
        const uint32_t off = (uint32_t)c * lbo + (uint32_t)r * 16u;
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(hi_tile + off), "r"(hi.x), "r"(hi.y), "r"(hi.z), "r"(hi.w) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(lo_tile + off), "r"(lo.x), "r"(lo.y), "r"(lo.z), "r"(lo.w) : "memory");
    }
}

// Converts one row (32 fp32, stored by TMA with the 128-byte swizzle) of a staged tile into ONE bf16 tile (round to
// nearest even; un-swizzled core-matrix layout, `rows` rows tall).
__device__ __forceinline__ void convert_row_bf16(uint32_t src_tile, uint32_t dst_tile, int r, int rows) {
    const uint32_t src = src_tile + (uint32_t)r * 128u;
    const uint32_t lbo = (uint32_t)rows * 16u;
#pragma unroll
    for (int c = 0; c < 4; ++c) {                              // 4 chunks of 8 K-elements
        float4 v0, v1;
        const uint32_t a0 = src + ((uint32_t)((2 * c) ^ (r & 7)) << 4), a1 = src + ((uint32_t)((2 * c + 1) ^ (r & 7)) << 4);
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v0.x), "=f"(v0.y), "=f"(v0.z), "=f"(v0.w) : "r"(a0));
        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v1.x), "=f"(v1.y), "=f"(v1.z), "=f"(v1.w) : "r"(a1));
        const __nv_bfloat162 p0 = __floats2bfloat162_rn(v0.x, v0.y), p1 = __floats2bfloat162_rn(v0.z, v0.w);
        const __nv_bfloat162 p2 = __floats2bfloat162_rn(v1.x, v1.y), p3 = __floats2bfloat162_rn(v1.z, v1.w);
        const uint32_t off = (uint32_t)c * lbo + (uint32_t)r * 16u;
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(dst_tile + off), "r"(*reinterpret_cast<const uint32_t*>(&p0)),
                     "r"(*reinterpret_cast<const uint32_t*>(&p1)), "r"(*reinterpret_cast<const uint32_t*>(&p2)),
                     "r"(*reinterpret_cast<const uint32_t*>(&p3)) : "memory");
    }
}

// MODE 3: A is fp32 (the activation itself, direct or through the TMA's im2col mode) and is rounded to bf16 by the
// epilogue warps on its way through shared memory; B is the bf16 packed weight, fetched straight into the
// un-swizzled core-matrix layout by ONE TMA box per stage over the rows seen as {8 elements, N rows, chunks}.
// MODE 0: TF32 operands (fp32 words), 1: BF16 operands, 2: fp32 operands multiplied as
// hi*hi + lo*hi + hi*lo of their bf16 splits (error-compensated, fp32-class accuracy).
template <int MODE> struct ModeTraits {
    static constexpr int BKE = (MODE == 1) ? 64 : 32;          // K elements per stage
};

template <int MODE>
__host__ __device__ constexpr uint32_t stage_bytes_of(int BN) {
    // staged TMA tiles (A: 128 rows x 128 B, B: BN rows x 128 B); mode 2 adds hi and lo bf16 tiles
    if (MODE == 3) return (uint32_t)(A_STAGE_BYTES + A_STAGE_BYTES / 2 + BN * 64);   // fp32 A, bf16 A, bf16 B (32 elements per row)
    return (uint32_t)(A_STAGE_BYTES + BN * BK_BYTES) * (MODE == 2 ? 2u : 1u);
}

template <int MODE>
__global__ void __launch_bounds__(GEMM_THREADS)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmD, const __grid_constant__ CUtensorMap tmAdd, const GemmDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const int STAGES = g.stages;                              // depth of the shared-memory ring (2..8)
    constexpr int MAXS = 8;
    constexpr int BKE = ModeTraits<MODE>::BKE;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int BN = g.BN;
    const uint32_t b_stage_bytes = (uint32_t)BN * BK_BYTES;
    const uint32_t tma_bytes = A_STAGE_BYTES + (MODE == 3 ? (uint32_t)BN * 64u : b_stage_bytes);
    const uint32_t stage_bytes = stage_bytes_of<MODE>(BN);
    const uint32_t bars = sbase + STAGES * stage_bytes;       // full[S], empty[S], conv[S], tmem_full, holder
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (MAXS + s); };
    auto conv_bar = [&](int s) { return bars + 8u * (2 * MAXS + s); };
    const uint32_t tmem_full_bar = bars + 8u * (3 * MAXS);
    const uint32_t holder = bars + 8u * (3 * MAXS + 1);
    const uint32_t addend_bar = bars + 8u * (3 * MAXS + 2);
    // Write-out through shared memory (g.tma_out): the tile is staged as [column chunk][warp quarter] sub-tiles of
    // 32 rows x CW columns in the swizzled layout of the output tensor map and stored by TMA.  With a residual
    // addend the sub-tiles live in their own region and the addend is loaded INTO them while the K loop runs, so
    // the epilogue adds in place; without one they reuse the ring, which is idle by then.
    const int CW = g.tma_out;
    const uint32_t chunk_bytes = 32u * (uint32_t)CW * 4u;
    const uint32_t stg0 = sbase + g.stage_off;
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // blockIdx.z = batch * splits + split; the `splits` CTAs of one output tile form a thread-block
    // cluster, each reducing its own contiguous range of K blocks.
    const int splits = g.splits;
    const int sp = (int)blockIdx.z % splits, b = (int)blockIdx.z / splits;
    const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
    const int nkb_all = g.ic_on ? g.Kd : (g.Kd + BKE - 1) / BKE;  // implicit mode: Kd already counts K blocks
    const int kb0 = (nkb_all * sp) / splits;                  // K blocks number a few thousand at most: 32-bit is enough
    const int nkb = (nkb_all * (sp + 1)) / splits - kb0;

    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
            mbar_init(conv_bar(s), 128);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(addend_bar, 1);
        if (CW) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmD)) : "memory");
            if (g.addend) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmAdd)) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // One K block: operand tiles of iteration `it` into ring slot `s` (= it mod STAGES; the loops carry
    // slot and phase along instead of dividing: STAGES is a run-time value and these single-thread
    // loops are latency-bound, every instruction in them is on the critical path).
    // Implicit mode: K runs over (filter tap, channel block).  The tile's first output pixel and the K
    // position of the next block are kept as running values: the producer issues blocks in order, and a
    // division per block would sit on the latency path of the very first loads.
    int ic_w0 = 0, ic_h0 = 0, ic_cb = 0, ic_fs = 0, ic_fr = 0, ic_tap = 0;
    if (g.ic_on) {
        const int p0 = m0 / g.ic_OW, q0 = m0 - p0 * g.ic_OW;
        ic_w0 = q0 * g.ic_stride - g.ic_pad;
        ic_h0 = p0 * g.ic_stride - g.ic_pad;
        ic_tap = kb0 / g.ic_cblk;
        ic_cb = kb0 - ic_tap * g.ic_cblk;
        ic_fr = ic_tap / g.ic_S;
        ic_fs = ic_tap - ic_fr * g.ic_S;
    }
    auto issue_stage = [&](int it, int s) {
        const int kb = kb0 + it;
        mbar_expect_tx(full_bar(s), tma_bytes);
        const uint32_t a_dst = sbase + s * stage_bytes;
        if (g.ic_on) {
            // A comes straight from the activation: block `kb` is channel block ic_cb of tap (ic_fr, ic_fs)
            tma_load_im2col_4d(a_dst, &tmA, ic_cb * BKE, ic_w0, ic_h0, 0, (uint16_t)ic_fs, (uint16_t)ic_fr, full_bar(s));
            if constexpr (MODE == 3) {   // B: one box of four 8-element chunks x BN rows, staged after the fp32 and the bf16 A tile
                tma_load_3d(a_dst + A_STAGE_BYTES + A_STAGE_BYTES / 2, &tmB, 0, n0, (ic_tap * g.ic_C + ic_cb * BKE) >> 3, full_bar(s));
            } else {
                tma_load_3d(a_dst + A_STAGE_BYTES, &tmB, ic_tap * g.ic_C + ic_cb * BKE, n0, b, full_bar(s));
            }
            if (++ic_cb == g.ic_cblk) {
                ic_cb = 0; ++ic_tap;
                if (++ic_fs == g.ic_S) { ic_fs = 0; ++ic_fr; }
            }
        } else {
            tma_load_3d(a_dst, &tmA, kb * BKE, m0, b, full_bar(s));
            if constexpr (MODE == 3) {
                tma_load_3d(a_dst + A_STAGE_BYTES + A_STAGE_BYTES / 2, &tmB, 0, n0, (kb * BKE) >> 3, full_bar(s));
            } else {
                tma_load_3d(a_dst + A_STAGE_BYTES, &tmB, kb * BKE, n0, b, full_bar(s));
            }
        }
    };
    // The producer fills the whole ring before the CTA-wide barrier: the first loads fly while
    // TMEM is being allocated.  It only needs its own barrier initialisation and the previous
    // kernel's results (pdl_wait).
    const int prefill = g.prefill ? (nkb < STAGES ? nkb : STAGES) : 0;
    if (warp == 0 && lane == 0) {
        pdl_wait();
        for (int it = 0; it < prefill; ++it) issue_stage(it, it);
        if (CW && g.addend) {                                 // the residual tile, straight into the staging sub-tiles
            const int nch = BN / CW;
            mbar_expect_tx(addend_bar, (uint32_t)nch * 4u * chunk_bytes);
            for (int j = 0; j < nch; ++j)
                for (int q = 0; q < 4; ++q)
                    tma_load_3d(stg0 + (uint32_t)(j * 4 + q) * chunk_bytes, &tmAdd, n0 + j * CW, m0 + q * 32, 0, addend_bar);
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *holder_ptr;
    pdl_wait();                                               // set-up above overlaps the previous kernel's tail
    if (threadIdx.x == 32) stamp_start(g.stamp);

    bool epi_ok = false;
    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int s = prefill == STAGES ? 0 : prefill;
            uint32_t ph = prefill == STAGES ? 1u : 0u;
            for (int it = prefill; it < nkb && ok; ++it) {
                ok = mbar_wait(empty_bar(s), ph ^ 1u);
                if (!ok) break;
                issue_stage(it, s);
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulate, A/B format, both K-major, N, M = 128
            const uint32_t fmt = (MODE == 0) ? 2u : 1u;
            const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < nkb; ++it, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                ok = mbar_wait((MODE == 2 || MODE == 3) ? conv_bar(s) : full_bar(s), ph);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = sbase + s * stage_bytes;
                if constexpr (MODE == 2) {
                    // converted tiles follow the staged ones: A_hi, A_lo (8 KB each), B_hi, B_lo
                    const uint32_t a_hi = a_src + tma_bytes, a_lo = a_hi + A_STAGE_BYTES / 2;
                    const uint32_t b_hi = a_lo + A_STAGE_BYTES / 2, b_lo = b_hi + b_stage_bytes / 2;
                    const uint32_t lbo_a = BM * 16u, lbo_b = (uint32_t)BN * 16u;
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk) {            // 2 K-steps of 16 bf16 = 2 core matrices each
                        const uint64_t ah = make_smem_desc_plain(a_hi + kk * 2 * lbo_a, lbo_a, 128);
                        const uint64_t al = make_smem_desc_plain(a_lo + kk * 2 * lbo_a, lbo_a, 128);
                        const uint64_t bh = make_smem_desc_plain(b_hi + kk * 2 * lbo_b, lbo_b, 128);
                        const uint64_t bl = make_smem_desc_plain(b_lo + kk * 2 * lbo_b, lbo_b, 128);
                        umma<true>(tmem_base, al, bh, idesc, (it | kk) ? 1u : 0u);   // small terms first
                        umma<true>(tmem_base, ah, bl, idesc, 1u);
                        umma<true>(tmem_base, ah, bh, idesc, 1u);
                    }
                } else if constexpr (MODE == 3) {
                    const uint32_t a_bf = a_src + A_STAGE_BYTES, b_bf = a_bf + A_STAGE_BYTES / 2;
                    const uint32_t lbo_a = BM * 16u, lbo_b = (uint32_t)BN * 16u;
#pragma unroll
                    for (int kk = 0; kk < 2; ++kk)             // 2 K-steps of 16 bf16 = 2 core matrices each
                        umma<true>(tmem_base, make_smem_desc_plain(a_bf + kk * 2 * lbo_a, lbo_a, 128),
                                   make_smem_desc_plain(b_bf + kk * 2 * lbo_b, lbo_b, 128), idesc, (it | kk) ? 1u : 0u);
                } else {
                    const uint64_t adesc = make_smem_desc(a_src);
                    const uint64_t bdesc = make_smem_desc(a_src + A_STAGE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)             // 4 MMAs of 32 bytes of K each
                        umma<MODE == 1>(tmem_base, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (it | kk) ? 1u : 0u);
                }
                umma_commit(empty_bar(s));
            }
            if (ok) umma_commit(tmem_full_bar);
            else atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        bool ok = true;
        if constexpr (MODE == 3) {
            // warps 2-5 first round every staged fp32 A tile to bf16 (the weights arrive as bf16)
            const int idx = (int)threadIdx.x - 64;              // 0..127: one row of A each
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < nkb; ++it, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                ok = mbar_wait(full_bar(s), ph);
                if (!ok) break;
                const uint32_t a_src = sbase + s * stage_bytes;
                convert_row_bf16(a_src, a_src + A_STAGE_BYTES, idx, BM);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
                mbar_arrive(conv_bar(s));
            }
        }
        if constexpr (MODE == 2) {
            // warps 2-5 first convert every staged fp32 tile into its bf16 hi / lo tiles
            const int idx = (int)threadIdx.x - 64;              // 0..127: one row of A (and of B) each
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < nkb; ++it, s = (s + 1 == STAGES ? 0 : s + 1), ph ^= (s == 0 ? 1u : 0u)) {
                ok = mbar_wait(full_bar(s), ph);
                if (!ok) break;
                const uint32_t a_src = sbase + s * stage_bytes;
                const uint32_t a_hi = a_src + tma_bytes, a_lo = a_hi + A_STAGE_BYTES / 2;
                const uint32_t b_hi = a_lo + A_STAGE_BYTES / 2, b_lo = b_hi + b_stage_bytes / 2;
                convert_row(a_src, a_hi, a_lo, idx, BM);
                if (idx < BN) convert_row(a_src + A_STAGE_BYTES, b_hi, b_lo, idx, BN);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
                mbar_arrive(conv_bar(s));
            }
        }
        ok = ok && mbar_wait(tmem_full_bar, 0);
        tc_fence_after();
        if (!ok) {
            if (lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        } else if (splits == 1 && CW) {
            // lane = one accumulator row; per column chunk: TMEM -> registers -> (+ bias, + addend from the staging
            // sub-tile, activation) -> staging sub-tile -> one TMA store per warp and chunk
            const int quarter = warp & 3;
            const int nch = BN / CW;
            bool aok = true;
            if (g.addend) aok = mbar_wait(addend_bar, 0);
            if (!aok) {
                if (lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
            } else {
                const bool row_live = m0 + quarter * 32 < g.M;
                for (int j = 0; j < nch; ++j) {
                    const uint32_t buf = stg0 + (uint32_t)(j * 4 + quarter) * chunk_bytes;
                    const uint32_t rowa = buf + (uint32_t)lane * (uint32_t)CW * 4u;
                    const int nbase = n0 + j * CW;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h * 16 >= CW) break;
                        uint32_t r[16];
                        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(j * CW + h * 16), r);
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) {
                            const int c = h * 4 + c4;                       // 16-byte chunk of the row
                            const int n = nbase + c * 4;
                            const uint32_t sw = (CW == 32) ? (uint32_t)(c ^ (lane & 7)) : (uint32_t)(c ^ ((lane >> 1) & 3));
                            const uint32_t addr = rowa + sw * 16u;
                            float4 v = make_float4(__uint_as_float(r[c4 * 4]), __uint_as_float(r[c4 * 4 + 1]),
                                                   __uint_as_float(r[c4 * 4 + 2]), __uint_as_float(r[c4 * 4 + 3]));
                            if (g.bias && n < g.N) {
                                const float4 bb = __ldg(reinterpret_cast<const float4*>(g.bias + n));
                                v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                            }
                            if (g.addend) {
                                float4 aa;
                                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(aa.x), "=f"(aa.y), "=f"(aa.z), "=f"(aa.w) : "r"(addr));
                                v.x += aa.x; v.y += aa.y; v.z += aa.z; v.w += aa.w;
                            }
                            v.x = act_fn(v.x, g.act); v.y = act_fn(v.y, g.act); v.z = act_fn(v.z, g.act); v.w = act_fn(v.w, g.act);
                            asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
                        }
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the TMA's reads
                    __syncwarp();
                    if (lane == 0 && row_live && nbase < g.N) {
                        tma_store_3d(&tmD, buf, nbase, m0 + quarter * 32, b);
                        tma_store_commit();
                    }
                }
                if (lane == 0) tma_store_wait_read();
            }
        } else if (splits == 1) {
            const int quarter = warp & 3;                     // TMEM lanes this warp may read
            const int m = m0 + quarter * 32 + lane;
            float* drow = g.D + (long long)b * g.strideD + (long long)m * g.ldd;
            const float* arow = g.addend ? g.addend + (long long)m * g.ldd : nullptr;
            const bool vec = ((g.ldd & 3) == 0) && ((g.N & 3) == 0) && ((reinterpret_cast<uintptr_t>(g.D) & 15) == 0) &&
                             (!g.addend || (reinterpret_cast<uintptr_t>(g.addend) & 15) == 0) &&
                             (!g.bias || (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0);
            for (int c0 = 0; c0 < BN; c0 += 16) {
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
                if (m >= g.M) continue;
                const int n = n0 + c0;
                if (vec) {
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        if (n + j >= g.N) break;
                        float4 v = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]), __uint_as_float(r[j + 2]),
                                               __uint_as_float(r[j + 3]));
                        if (g.bias) {
                            const float4 bb = __ldg(reinterpret_cast<const float4*>(g.bias + n + j));
                            v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                        }
                        if (arow) {
                            const float4 aa = __ldg(reinterpret_cast<const float4*>(arow + n + j));
                            v.x += aa.x; v.y += aa.y; v.z += aa.z; v.w += aa.w;
                        }
                        v.x = act_fn(v.x, g.act); v.y = act_fn(v.y, g.act); v.z = act_fn(v.z, g.act); v.w = act_fn(v.w, g.act);
                        *reinterpret_cast<float4*>(drow + n + j) = v;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        if (n + j < g.N) {
                            float v = __uint_as_float(r[j]);
                            if (g.bias) v += __ldg(g.bias + n + j);
                            if (arow) v += __ldg(arow + n + j);
                            drow[n + j] = act_fn(v, g.act);
                        }
                    }
                }
            }
        } else {
            epi_ok = true;
            // park this CTA's (partial) tile in its own shared memory (the stage ring is idle by now):
            // P[row][col], row pitch BN + 4 words
            const int quarter = warp & 3;
            const int row = quarter * 32 + lane;
            const uint32_t prow = sbase + (uint32_t)row * (uint32_t)(BN + 4) * 4u;
            for (int c0 = 0; c0 < BN; c0 += 16) {
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
#pragma unroll
                for (int j = 0; j < 16; j += 4)
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(prow + (uint32_t)(c0 + j) * 4u), "r"(r[j]),
                                 "r"(r[j + 1]), "r"(r[j + 2]), "r"(r[j + 3]) : "memory");
            }
        }
    }
    __syncwarp();
    {
        // Split-K write-out.  Every CTA of the cluster has parked its partial tile in shared memory;
        // CTA `sp` sums rows [sp*128/splits, (sp+1)*128/splits) over the cluster through distributed
        // shared memory in rank order (a fixed order: the result does not depend on timing), then
        // applies bias / residual / activation and stores row-contiguous 128-bit words.  The
        // cluster barriers are reached by every thread on every path.
        if (splits > 1) cluster_sync_all();
        if (splits > 1 && warp >= 2 && g_device_status == 0) {
            const int t = (int)threadIdx.x - 64;
            // only the rows of the tile that exist are reduced, shared evenly by the cluster's CTAs
            const int live = min(BM, g.M - m0);
            const int rows_per = (live + splits - 1) / splits, r0 = sp * rows_per;
            const int c4n = BN / 4;
            const bool vec = ((g.ldd & 3) == 0) && ((g.N & 3) == 0) && ((reinterpret_cast<uintptr_t>(g.D) & 15) == 0) &&
                             (!g.addend || (reinterpret_cast<uintptr_t>(g.addend) & 15) == 0) &&
                             (!g.bias || (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0);
            // Thread t walks the (row, 4-column group) grid in steps of 128 without divisions.  The loop
            // is kept small on purpose (no unrolling): each CTA runs it once, and instruction fetch of
            // cold code costs more here than the arithmetic.
            const int total = max(0, min(rows_per, live - r0)) * c4n;
            const int qstep = 128 / c4n, rstep = 128 - qstep * c4n;
            int row = r0 + t / c4n, col4 = t % c4n;
            float* const dbase = g.D + (long long)b * g.strideD;
#pragma unroll 1
            for (int idx = t; idx < total; idx += 128) {
                const int rr = row, cc = col4 * 4;
                row += qstep; col4 += rstep;
                if (col4 >= c4n) { col4 -= c4n; ++row; }
                const uint32_t local = sbase + ((uint32_t)rr * (uint32_t)(BN + 4) + (uint32_t)cc) * 4u;
                // all remote loads are issued before the first is consumed, so their latencies overlap
                float4 v[8];
#pragma unroll
                for (int rk = 0; rk < 8; ++rk) {
                    if (rk < splits) {
                        uint32_t remote;
                        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rk));
                        asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v[rk].x), "=f"(v[rk].y), "=f"(v[rk].z), "=f"(v[rk].w) : "r"(remote));
                    }
                }
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int rk = 0; rk < 8; ++rk)
                    if (rk < splits) { acc.x += v[rk].x; acc.y += v[rk].y; acc.z += v[rk].z; acc.w += v[rk].w; }
                const int m = m0 + rr, n = n0 + cc;
                if (m >= g.M || n >= g.N) continue;
                float* drow = dbase + (long long)m * g.ldd;
                const float* arow = g.addend ? g.addend + (long long)m * g.ldd : nullptr;
                float vv[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (vec || n + j < g.N) {
                        if (g.bias) vv[j] += __ldg(g.bias + n + j);
                        if (arow) vv[j] += __ldg(arow + n + j);
                        vv[j] = act_fn(vv[j], g.act);
                    }
                }
                if (vec) {
                    *reinterpret_cast<float4*>(drow + n) = make_float4(vv[0], vv[1], vv[2], vv[3]);
                } else {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (n + j < g.N) drow[n + j] = vv[j];
                }
            }
        }
        if (splits > 1) cluster_sync_all();                   // nobody leaves while its tile may still be read
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

#include "conv3x3_tc.cuh"
#include "gemm_sp.cuh"
#include "wino_fused.cuh"

// ---- host side --------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;
PFN_cuTensorMapEncodeIm2col_v12000 g_encode_im2col = nullptr;
std::once_flag g_encode_once;
cudaError_t g_encode_err = cudaSuccess;

nnv_status_t get_encoder() {
    std::call_once(g_encode_once, [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        g_encode_err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (g_encode_err == cudaSuccess && q == cudaDriverEntryPointSuccess) g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
        void* fn2 = nullptr;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeIm2col", &fn2, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            g_encode_im2col = (PFN_cuTensorMapEncodeIm2col_v12000)fn2;
    });
    NNV_REQUIRE(g_encode != nullptr, NNV_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    return NNV_OK;
}

// 3-D map over a K-major operand: dims {Kd, rows, batch}, box {128 bytes of K, box_rows, 1}.
nnv_status_t encode_operand(CUtensorMap* map, const void* base, bool bf16, int Kd, int rows, int batch, int64_t ld,
                            int64_t batch_stride, int box_rows) {
    const uint64_t es = bf16 ? 2 : 4;
    NNV_REQUIRE((reinterpret_cast<uintptr_t>(base) & 15) == 0, NNV_ERR_INVALID_ARG, "GEMM operand is not 16-byte aligned");
    NNV_REQUIRE((ld * es) % 16 == 0 && (batch_stride * es) % 16 == 0, NNV_ERR_INVALID_ARG,
                "GEMM operand strides must be multiples of 16 bytes");
    cuuint64_t dims[3] = {(cuuint64_t)Kd, (cuuint64_t)rows, (cuuint64_t)batch};
    cuuint64_t strides[2] = {(cuuint64_t)(ld * es), (cuuint64_t)(batch_stride * es)};
    cuuint32_t box[3] = {(cuuint32_t)(BK_BYTES / es), (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
                          const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    return NNV_OK;
}

// 3-D map over the fp32 output (or the residual addend, same geometry): dims {N, M, batch}, boxes of
// `cw` columns (32 with the 128-byte swizzle, 16 with the 64-byte one) x 32 rows.
nnv_status_t encode_output(CUtensorMap* map, const void* base, int N, int M, int batch, int64_t ld, int64_t batch_stride, int cw) {
    cuuint64_t dims[3] = {(cuuint64_t)N, (cuuint64_t)M, (cuuint64_t)batch};
    cuuint64_t strides[2] = {(cuuint64_t)(ld * 4), (cuuint64_t)(batch_stride * 4)};
    cuuint32_t box[3] = {(cuuint32_t)cw, 32, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, cw == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled (output tiles) failed with code %d", (int)r);
    return NNV_OK;
}

// 4-D im2col map over an NHWC fp32 activation {C, W, H, 1}: 32 channels x 128 output pixels per load.
nnv_status_t encode_im2col_operand(CUtensorMap* map, const void* base, int C, int H, int W, int R, int S, int stride,
                                   int pad) {
    NNV_REQUIRE(g_encode_im2col != nullptr, NNV_ERR_CUDA, "cuTensorMapEncodeIm2col is not available from this driver");
    NNV_REQUIRE((reinterpret_cast<uintptr_t>(base) & 15) == 0 && (C % 4) == 0, NNV_ERR_INVALID_ARG,
                "implicit-GEMM activation must be 16-byte aligned with C a multiple of 4");
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, 1};
    cuuint64_t strides[3] = {(cuuint64_t)C * 4, (cuuint64_t)W * C * 4, (cuuint64_t)H * W * C * 4};
    int lower[2] = {-pad, -pad};
    int upper[2] = {pad - (S - 1), pad - (R - 1)};
    cuuint32_t estr[4] = {1, (cuuint32_t)stride, (cuuint32_t)stride, 1};
    CUresult r = g_encode_im2col(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, const_cast<void*>(base), dims, strides, lower,
                                 upper, 32, BM, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeIm2col failed with code %d", (int)r);
    return NNV_OK;
}

// 3-D tiled map over an NHWC fp32 activation {C, W, H}: boxes of 32 channels x 8 pixels x `box_h`
// rows (the halo boxes of conv3x3_tc_kernel); coordinates outside the image read as zero.
nnv_status_t encode_halo_operand(CUtensorMap* map, const void* base, int C, int H, int W, int box_h) {
    NNV_REQUIRE((reinterpret_cast<uintptr_t>(base) & 15) == 0 && (C % 4) == 0, NNV_ERR_INVALID_ARG,
                "activation must be 16-byte aligned with C a multiple of 4");
    cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H};
    cuuint64_t strides[2] = {(cuuint64_t)C * 4, (cuuint64_t)W * C * 4};
    cuuint32_t box[3] = {32, 8, (cuuint32_t)box_h};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled (halo boxes) failed with code %d", (int)r);
    return NNV_OK;
}

// Tiling of conv3x3_tc_kernel for one layer.
struct ConvTiling { int MT, BN, splits, na, nb, tmem_cols, bf16; size_t smem; };

// Bytes of one halo-box slot and one weight-tile slot: with BF16 math a box slot also holds the box rounded to bf16
// (half its size) and a weight tile is bf16.
size_t conv_a_slot(int MT, int bf16) { return (size_t)(16 * MT + 2) * 1024 * (bf16 ? 3 : 2) / 2; }
size_t conv_b_slot(int BN, int bf16) { return (size_t)BN * (bf16 ? 64 : BK_BYTES); }

size_t conv_smem_bytes(int MT, int BN, int na, int nb, int bf16) {
    return (size_t)1024 + (size_t)na * conv_a_slot(MT, bf16) + (size_t)nb * conv_b_slot(BN, bf16) + 8 * (3 * CONV_MAX_NA + 2 * CONV_MAX_NB + 2);
}

// Fills in ring depths (unless given), shared-memory size and TMEM columns; false if the tiling does
// not fit (shared memory, or room to park the partial tiles of a K split).
bool finish_conv_tiling(ConvTiling* t) {
    const size_t park = t->splits > 1 ? (size_t)t->MT * BM * (t->BN + 4) * 4 : 0;
    auto rings = [&] { return (size_t)t->na * conv_a_slot(t->MT, t->bf16) + (size_t)t->nb * conv_b_slot(t->BN, t->bf16); };
    if (t->na <= 0 || t->nb <= 0) {
        t->na = 2; t->nb = 3;
        while (rings() < park && t->nb < CONV_MAX_NB) ++t->nb;      // deeper rings only to make room for the parked tiles
        while (rings() < park && t->na < CONV_MAX_NA) ++t->na;
    }
    t->smem = conv_smem_bytes(t->MT, t->BN, t->na, t->nb, t->bf16);
    t->tmem_cols = 32;
    while (t->tmem_cols < t->MT * t->BN) t->tmem_cols *= 2;
    return t->smem <= 200u * 1024u && rings() >= park;
}

// Measured on B200 (sweeps over tilings, ring depths and K splits at the 3x3 shapes of the VGG / ResNet
// configurations, L2 flushed before each launch): the kernel runs best with one MMA tile per CTA,
// channel tiles of 128, shallow rings (two or three CTAs then share an SM, and one CTA's fill and
// write-out overlap another's MMAs) and enough K splits for ~1.5 CTAs per SM; all CTAs should be
// resident at once (a second, mostly empty wave costs as much as the first), so the box ring drops
// to one slot when that makes them fit.  Layers with fewer than four channel blocks and fewer than
// two patches per SM, and layers too small to give every SM a CTA even with 8 splits, stay on the
// plain implicit GEMM, which is faster there.
bool pick_conv_tiling(int C, int H, int W, int N, int bf16, ConvTiling* out) {
    const int cblk = ceil_div(C, 32);
    ConvTiling t{};
    t.MT = 1;
    t.bf16 = bf16;
    t.BN = std::min(128, ceil_div(N, 16) * 16);
    const long long tiles = (long long)ceil_div(H, 16) * ceil_div(W, 8) * ceil_div(N, t.BN);
    int max_sp = 1;
    while (max_sp * 2 <= std::min(8, cblk)) max_sp *= 2;
    if (tiles * max_sp < 148 || (cblk < 4 && tiles < 296)) return false;
    // Against the implicit GEMM with its refit tiling model (kernel stamps, L2 flushed; halo kernel / implicit GEMM, us):
    // 64 -> 64 @224 13.4 / 18.0 and 256 -> 256 @56 18.8 / 24.0, but 128 -> 128 @112 17.7 / 14.9, 128 -> 256 @56 14.7 / 12.8,
    // 256 -> 512 @28 14.7 / 12.9, 512 -> 512 @28 19.0 / 18.6: the halo kernel keeps the layers with two or more patches per SM
    // and the deep ones (eight or more channel blocks) that still have ~50 tiles.
    if (tiles < 296 && !(cblk >= 8 && tiles >= 48)) return false;
    t.splits = 1;
    while (t.splits < max_sp && tiles * t.splits < 224) t.splits *= 2;
    const long long ctas = tiles * t.splits;
    bool found = false;
    const int rings[2][2] = {{2, 3}, {1, 3}};
    for (int i = 0; i < 2 && !found; ++i) {
        ConvTiling c = t;
        c.na = rings[i][0]; c.nb = rings[i][1];
        if (!finish_conv_tiling(&c)) continue;
        const int occ = std::max(1, std::min((int)(227u * 1024u / (c.smem + 1024)), 512 / c.tmem_cols));
        if (ctas <= 148ll * occ) { t = c; found = true; }
    }
    if (!found) { t.na = 0; t.nb = 0; found = finish_conv_tiling(&t); }
    if (found) *out = t;
    return found;
}

std::once_flag g_attr_once;

}  // namespace

nnv_status_t gemm_tc_init() {
    NNV_TRY(get_encoder());
    std::call_once(g_attr_once, [] {
        cudaFuncSetAttribute(gemm_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(gemm_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(gemm_tc_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(gemm_tc_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(conv3x3_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(gemm_sp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(conv3x3_tc_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(wino_f2_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024);
        cudaFuncSetAttribute(conv3x3_tc_ws_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
    });
    return NNV_OK;
}

// bf16 packed weights [N][ld]: boxes of 8 elements (16 bytes) x BN rows, no swizzle -- four of them make the
// un-swizzled core-matrix layout of a 32-element K block.
static nnv_status_t encode_bf16_weight_chunks(CUtensorMap* map, const void* base, int64_t ld, int N, int BN) {
    NNV_REQUIRE((ld % 8) == 0 && (reinterpret_cast<uintptr_t>(base) & 15) == 0, NNV_ERR_INVALID_ARG, "bf16 weight rows must be 16-byte multiples");
    // the rows seen as {8 elements, N rows, ld / 8 chunks}: one box of {8, BN, 4} lands as [chunk][row][16 bytes], i.e. a whole
    // 32-element K block of BN rows in the core-matrix layout with ONE load (a fill costs ~150 cycles whatever its size)
    cuuint64_t dims[3] = {8, (cuuint64_t)N, (cuuint64_t)(ld / 8)};
    cuuint64_t strides[2] = {(cuuint64_t)ld * 2, 16};
    cuuint32_t box[3] = {8, (cuuint32_t)BN, 4};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled (bf16 weight chunks) failed with code %d", (int)r);
    return NNV_OK;
}

// 3-D tiled map over the NHWC fp32 output {K, W, H}: boxes of `cw` channels x 8 pixels x 4 rows (what one warp of the
// 3x3 kernel holds), in the swizzled layout the epilogue writes.
static nnv_status_t encode_conv_output(CUtensorMap* map, const void* base, int K, int H, int W, int cw) {
    cuuint64_t dims[3] = {(cuuint64_t)K, (cuuint64_t)W, (cuuint64_t)H};
    cuuint64_t strides[2] = {(cuuint64_t)K * 4, (cuuint64_t)W * K * 4};
    cuuint32_t box[3] = {(cuuint32_t)cw, 8, 4};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, cw == 32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled (3x3 output boxes) failed with code %d", (int)r);
    return NNV_OK;
}

static nnv_status_t launch_conv3x3_tc(const GemmArgs& a, const ConvTiling& ct, cudaStream_t st) {
    CUtensorMap tmA, tmB, tmD;
    NNV_TRY(encode_halo_operand(&tmA, a.A, a.ic.C, a.ic.H, a.ic.W, 16 * ct.MT + 2));
    if (ct.bf16) NNV_TRY(encode_bf16_weight_chunks(&tmB, a.B, a.ldb, a.N, ct.BN));
    else NNV_TRY(encode_operand(&tmB, a.B, false, a.Kd, a.N, 1, a.ldb, a.strideB, ct.BN));
    ConvDev g;
    g.stamp = next_stamp();
    next_stamp() = nullptr;
    g.D = a.D; g.bias = a.bias; g.addend = a.addend;
    g.C = a.ic.C; g.H = a.ic.H; g.W = a.ic.W; g.K = a.N;
    g.BN = ct.BN; g.MT = ct.MT; g.act = a.act; g.tmem_cols = ct.tmem_cols; g.splits = ct.splits; g.na = ct.na; g.nb = ct.nb;
    g.cblk = ceil_div(a.ic.C, 32); g.tiles_w = ceil_div(a.ic.W, 8);
    g.bf16 = ct.bf16;
    NNV_REQUIRE(a.ldd == a.N, NNV_ERR_INVALID_ARG, "the 3x3 kernel writes a dense NHWC output");
    // Write-out by TMA when nothing is added after the K loop but the bias, the output rows are 16-byte multiples and
    // the staged tile fits into the (then idle) rings; else plain stores.
    g.tma_out = 0;
    const size_t rings = (size_t)ct.na * conv_a_slot(ct.MT, ct.bf16) + (size_t)ct.nb * conv_b_slot(ct.BN, ct.bf16);
    if (ct.splits == 1 && !a.addend && (a.N % 4) == 0 && (reinterpret_cast<uintptr_t>(a.D) & 15) == 0 &&
        (!a.bias || (reinterpret_cast<uintptr_t>(a.bias) & 15) == 0) && (size_t)ct.MT * BM * ct.BN * 4 <= rings) {
        g.tma_out = (ct.BN % 32) == 0 ? 32 : 16;
        NNV_TRY(encode_conv_output(&tmD, a.D, a.N, a.ic.H, a.ic.W, g.tma_out));
    } else {
        tmD = tmA;                                               // unused by the kernel, but a kernel parameter must hold a valid object
    }
    dim3 grid(ceil_div(a.ic.H, 16 * ct.MT) * g.tiles_w, ceil_div(a.N, ct.BN), ct.splits);
    NNV_REQUIRE(grid.y <= 65535, NNV_ERR_UNSUPPORTED, "convolution grid too large");
    (void)launch_pdl_cluster(conv3x3_tc_kernel, grid, dim3(GEMM_THREADS), ct.smem, st, ct.splits, tmA, tmB, tmD, g);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// 3-D tiled map over an NHWC fp32 activation {C, W, H} whose box is 32 channels of the WHOLE image.
static nnv_status_t encode_image_operand(CUtensorMap* map, const void* base, int C, int H, int W) {
    NNV_REQUIRE((reinterpret_cast<uintptr_t>(base) & 15) == 0 && (C % 4) == 0 && W <= 256 && H <= 256, NNV_ERR_INVALID_ARG,
                "activation must be 16-byte aligned with C a multiple of 4 and at most 256 pixels a side");
    cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H};
    cuuint64_t strides[2] = {(cuuint64_t)C * 4, (cuuint64_t)W * C * 4};
    cuuint32_t box[3] = {32, (cuuint32_t)W, (cuuint32_t)H};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = g_encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled (whole-image boxes) failed with code %d", (int)r);
    return NNV_OK;
}

nnv_status_t launch_gemm_sp(const nnv_layer_desc_t& L, const LayerGeom& geo, const SmallPPlan& sp, const float* x, const float* wt,
                            const float* bias, const float* addend, float* y, void* ws, cudaStream_t st) {
    NNV_TRY(gemm_tc_init());
    NNV_REQUIRE(sp.splits == 1 || ws, NNV_ERR_INVALID_ARG, "the K split needs its scratch");
    CUtensorMap tmW, tmX;
    NNV_TRY(encode_operand(&tmW, wt, false, geo.Qp, L.K, 1, geo.Qp, (int64_t)L.K * geo.Qp, BM));
    NNV_TRY(encode_image_operand(&tmX, x, L.C, L.H, L.W));
    SpDev g;
    g.stamp = next_stamp();
    next_stamp() = nullptr;
    g.D = y; g.part = (float*)ws; g.bias = bias; g.addend = addend;
    g.P = geo.P; g.K = L.K; g.C = L.C; g.S = L.S; g.pad = L.pad; g.Npad = sp.Npad; g.act = L.act;
    g.tmem_cols = 32;
    while (g.tmem_cols < sp.Npad) g.tmem_cols *= 2;
    g.splits = sp.splits; g.stages = sp.stages; g.cblk = L.C / 32; g.nkb_all = sp.nkb;
    g.b_slot_bytes = sp.b_slot_bytes; g.b_tx_bytes = (uint32_t)(L.H * L.W) * 128u;
    const size_t smem = (size_t)1024 + (size_t)sp.stages * (A_STAGE_BYTES + sp.b_slot_bytes) + 8 * (2 * SP_MAX_STAGES + 2);
    dim3 grid(ceil_div(L.K, BM), sp.splits);
    (void)launch_pdl(gemm_sp_kernel, grid, dim3(GEMM_THREADS), smem, st, tmW, tmX, g);
    NNV_CUDA(cudaGetLastError());
    if (sp.splits > 1) {
        const long long n4 = (long long)geo.P * L.K / 4;
        const unsigned blocks = (unsigned)((n4 + 31) / 32);
        (void)launch_pdl(splitk_reduce_kernel, dim3(blocks), dim3(256), 0, st, (const float*)ws, y, bias, addend, geo.P, L.K, sp.splits,
                         L.act, g.stamp);
        NNV_CUDA(cudaGetLastError());
    }
    return NNV_OK;
}

nnv_status_t launch_wino_f2_fused(const nnv_layer_desc_t& L, const LayerGeom& geo, const float* x, const float* U, const float* bias,
                                  const float* addend, float* y, cudaStream_t st) {
    NNV_TRY(gemm_tc_init());
    NNV_REQUIRE((reinterpret_cast<uintptr_t>(x) & 15) == 0 && (reinterpret_cast<uintptr_t>(U) & 15) == 0 &&
                    (reinterpret_cast<uintptr_t>(y) & 15) == 0 && (!bias || (reinterpret_cast<uintptr_t>(bias) & 15) == 0) &&
                    (!addend || (reinterpret_cast<uintptr_t>(addend) & 15) == 0),
                NNV_ERR_INVALID_ARG, "the fused Winograd kernel needs 16-byte aligned buffers");
    WfDev g;
    g.stamp = next_stamp();
    next_stamp() = nullptr;
    g.x = x; g.y = y; g.bias = bias; g.addend = addend;
    g.C = L.C; g.H = L.H; g.W = L.W; g.K = L.K; g.pad = L.pad; g.OH = geo.OH; g.OW = geo.OW;
    g.TW = ceil_div(geo.OW, 2);
    g.T = ceil_div(geo.OH, 2) * g.TW;
    g.act = L.act;
    // 32 output channels per CTA (all 512 TMEM columns) when that still gives every other SM a CTA, else 16
    const int row_tiles = ceil_div(g.T, BM);
    g.BN = ((L.K % 32) == 0 && (long long)row_tiles * (L.K / 32) >= 74) ? 32 : 16;
    g.tmem_cols = 16 * g.BN;
    g.nsteps = L.C / 8;
    g.stages = std::min(WF_MAX_STAGES, std::max(1, g.nsteps));
    const uint32_t b_stage = 2u * 16u * (uint32_t)g.BN * 16u;
    while (g.stages > 1 && (size_t)1024 + (size_t)g.stages * (WF_A_STAGE + b_stage) + 8 * (3 * WF_MAX_STAGES + 2) > 220u * 1024u) --g.stages;
    const size_t smem = (size_t)1024 + (size_t)g.stages * (WF_A_STAGE + b_stage) + 8 * (3 * WF_MAX_STAGES + 2);
    CUtensorMap tmU;
    {
        cuuint64_t dims[3] = {(cuuint64_t)geo.Cp, (cuuint64_t)L.K, 16};
        cuuint64_t strides[2] = {(cuuint64_t)geo.Cp * 4, (cuuint64_t)L.K * geo.Cp * 4};
        cuuint32_t box[3] = {4, (cuuint32_t)g.BN, 16};
        cuuint32_t estr[3] = {1, 1, 1};
        CUresult r = g_encode(&tmU, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float*>(U), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        NNV_REQUIRE(r == CUDA_SUCCESS, NNV_ERR_CUDA, "cuTensorMapEncodeTiled (transformed filters) failed with code %d", (int)r);
    }
    dim3 grid(row_tiles, ceil_div(L.K, g.BN));
    (void)launch_pdl(wino_f2_fused_kernel, grid, dim3(GEMM_THREADS), smem, st, tmU, g);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// The weights-stationary form; `fits` tells whether the layer's weight slice and the kernel's other buffers fit.
static size_t convw_smem_bytes(int cblk, int BN) {
    return (size_t)1024 + (size_t)9 * cblk * BN * BK_BYTES + (size_t)CONVW_NA * 18 * 1024 + 4 * 4096 + 8 * (CONVW_MAX_WT + 2 * CONVW_NA + 5);
}
static bool convw_fits(const GemmArgs& a, int* BN_out) {
    const int cblk = ceil_div(a.ic.C, 32);
    const int BN = std::min(128, ceil_div(a.N, 16) * 16);
    if (9 * cblk > CONVW_MAX_WT || (BN % 16) != 0 || a.addend || (a.N % 4) != 0 || a.ldd != a.N) return false;
    if ((reinterpret_cast<uintptr_t>(a.D) & 15) != 0 || (a.bias && (reinterpret_cast<uintptr_t>(a.bias) & 15) != 0)) return false;
    // the widest channel tile (a multiple of 16, at most 128) whose weight slice fits
    for (int bn = BN; bn >= 16; bn -= 16) {
        if (convw_smem_bytes(cblk, bn) <= 226u * 1024u) { *BN_out = bn; return true; }
    }
    return false;
}
static nnv_status_t launch_conv3x3_ws(const GemmArgs& a, int BN, cudaStream_t st) {
    CUtensorMap tmA, tmB, tmD;
    NNV_TRY(encode_halo_operand(&tmA, a.A, a.ic.C, a.ic.H, a.ic.W, 18));
    NNV_TRY(encode_operand(&tmB, a.B, false, a.Kd, a.N, 1, a.ldb, a.strideB, BN));
    ConvWDev g;
    g.stamp = next_stamp();
    next_stamp() = nullptr;
    g.bias = a.bias;
    g.C = a.ic.C; g.H = a.ic.H; g.W = a.ic.W; g.K = a.N;
    g.BN = BN; g.act = a.act;
    g.cblk = ceil_div(a.ic.C, 32); g.tiles_w = ceil_div(a.ic.W, 8);
    g.patches = ceil_div(a.ic.H, 16) * g.tiles_w;
    g.cw = (BN % 32) == 0 ? 32 : 16;
    g.tmem_cols = 32;
    while (g.tmem_cols < 2 * BN) g.tmem_cols *= 2;
    NNV_TRY(encode_conv_output(&tmD, a.D, a.N, a.ic.H, a.ic.W, g.cw));
    const int n_tiles = ceil_div(a.N, BN);
    const int ctas_x = std::max(1, std::min(g.patches, 148 / n_tiles));
    const size_t smem = convw_smem_bytes(g.cblk, BN);
    (void)launch_pdl(conv3x3_tc_ws_kernel, dim3(ctas_x, n_tiles), dim3(GEMM_THREADS), smem, st, tmA, tmB, tmD, g);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// The persistent form: BN channels per tile, `per_sm` CTAs per SM, ring depths na / nb.
static nnv_status_t launch_conv3x3_persistent(const GemmArgs& a, int BN, int per_sm, int na, int nb, cudaStream_t st) {
    CUtensorMap tmA, tmB;
    NNV_TRY(encode_halo_operand(&tmA, a.A, a.ic.C, a.ic.H, a.ic.W, 18));
    NNV_TRY(encode_operand(&tmB, a.B, false, a.Kd, a.N, 1, a.ldb, a.strideB, BN));
    ConvPDev g;
    g.stamp = next_stamp();
    next_stamp() = nullptr;
    g.D = a.D; g.bias = a.bias; g.addend = a.addend;
    g.C = a.ic.C; g.H = a.ic.H; g.W = a.ic.W; g.K = a.N;
    g.BN = BN; g.act = a.act; g.na = na; g.nb = nb;
    g.cblk = ceil_div(a.ic.C, 32); g.tiles_w = ceil_div(a.ic.W, 8);
    g.n_tiles = ceil_div(a.N, BN);
    g.tiles_total = ceil_div(a.ic.H, 16) * g.tiles_w * g.n_tiles;
    g.tmem_cols = 32;
    while (g.tmem_cols < 2 * BN) g.tmem_cols *= 2;
    NNV_REQUIRE(a.ldd == a.N, NNV_ERR_INVALID_ARG, "the 3x3 kernel writes a dense NHWC output");
    const size_t smem = (size_t)1024 + (size_t)na * 18 * 1024 + (size_t)nb * BN * BK_BYTES + 4 * 32 * 36 * 4 +
                        8 * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB + 5);
    NNV_REQUIRE(smem <= 220u * 1024u, NNV_ERR_UNSUPPORTED, "persistent 3x3 tiling does not fit shared memory");
    const int ctas = std::min(g.tiles_total, 148 * per_sm);
    (void)launch_pdl(conv3x3_tc_persistent_kernel, dim3(ctas), dim3(GEMM_THREADS), smem, st, tmA, tmB, g);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

nnv_status_t launch_gemm_tc(const GemmArgs& a, cudaStream_t st) {
    NNV_REQUIRE(a.M > 0 && a.N > 0 && a.Kd > 0 && a.batch > 0, NNV_ERR_INVALID_ARG, "empty GEMM");
    NNV_TRY(gemm_tc_init());
    // Tiling.  These layers are small for 148 SMs, and one CTA can pull operand tiles out of L2 only
    // so fast (~90 GB/s measured), so the column tile BN and the number of K splits (a thread-block
    // cluster of up to 8 CTAs reducing through shared memory) are picked by a small cost model:
    // waves x (fixed cost + K blocks per CTA x bytes per K block / per-SM bandwidth).
    const int bke = (a.mode == GEMM_BF16) ? 64 : 32;
    const int nkb_all = a.ic.on ? a.ic.R * a.ic.S * ceil_div(a.ic.C, 32) : ceil_div(a.Kd, bke);
    const int m_tiles = ceil_div(a.M, BM);
    // Ring depth: 8 stages when every CTA has an SM to itself (a lone CTA needs that many loads in flight to keep
    // the SM's ~100 GB/s of shared-memory fill busy on weights that come cold from HBM), 4 when several share one.
    auto ring_for = [&](int bn, long long ctas) {
        const uint32_t stage = (a.mode == GEMM_X3) ? stage_bytes_of<2>(bn) : (a.mode == GEMM_BF16_CVT) ? stage_bytes_of<3>(bn) : stage_bytes_of<0>(bn);
        if (a.mode == GEMM_X3) return 3;
        return (ctas <= 148 && (size_t)8 * stage <= 200u * 1024u) ? 8 : 4;
    };
    int BN = 0, splits = 1;
    double best = 1e30;
    for (int nt = ceil_div(a.N, 128); nt <= ceil_div(a.N, 16); nt *= 2) {
        const int bn = ceil_div(ceil_div(a.N, nt), 16) * 16;
        const int n_tiles = ceil_div(a.N, bn);
        const double kb_bytes = (double)(A_STAGE_BYTES + bn * BK_BYTES);
        for (int sp = 1; sp <= 8 && sp <= nkb_all; sp *= 2) {
            const long long ctas = (long long)m_tiles * n_tiles * a.batch * sp;
            const int stages = ring_for(bn, ctas);
            const double smem = 1024.0 + stages * kb_bytes * (a.mode == GEMM_X3 ? 2 : 1);
            const int occ = std::max(1, std::min(4, (int)(220.0 * 1024.0 / smem)));
            double waves = std::ceil((double)ctas / (148.0 * occ));
            // whole clusters must find free SMs in one GPC (16 - 20 SMs): measured in one wave are 14 clusters of 8
            // (128 -> 128 3x3 @28 at BN = 64: 6.3 us against 8.3) and 32 clusters of 4 (1024 -> 2048 1x1 / 2 @14 at BN = 64: 6.8 against 9.0)
            if (sp > 1 && occ == 1 && ctas > (sp == 8 ? 112 : sp == 4 ? 128 : 144)) waves = std::max(waves, 2.0);
            const int resident = (int)std::min<long long>(occ, (ctas + 147) / 148);   // CTAs that really share an SM
            // refit on a sweep of every (BN, splits) over the GEMM layer shapes of the ResNet-shaped configurations (kernel
            // stamps, L2 flushed): a K block costs a CTA at least 0.25 us however narrow its tile (an unsplit BN = 16 launch of
            // 512 -> 128 @28 took 6.5 us where 5.3 was predicted, 64 x 8 splits 6.0), a split 2.5 us
            const double per_kb_us = std::max(kb_bytes * resident / 100e3, 0.25) * (stages >= 8 ? 1.0 : 1.3);
            const double t = waves * (2.0 + (sp > 1 ? 2.5 : 0.0) + std::ceil((double)nkb_all / sp) * per_kb_us + 0.3 + bn * 0.004);
            if (t < best - 1e-9) { best = t; BN = bn; splits = sp; }
        }
        if (bn <= 16) break;
    }
    const Tuning tn = tuning();
    if (tn.gemm_bn && tn.gemm_splits <= nkb_all) { BN = tn.gemm_bn; splits = tn.gemm_splits; }   // override (nnv_tuning_set)
    // A 3x3 / stride 1 / pad 1 layer large enough to fill the GPU runs on the halo-resident kernel,
    // which moves fewer operand bytes through L2 and shared memory.
    if (a.ic.on && (a.mode == GEMM_TF32 || a.mode == GEMM_BF16_CVT) && a.batch == 1 && a.ic.R == 3 && a.ic.S == 3 && a.ic.stride == 1 &&
        a.ic.pad == 1 && (a.ic.C % 32) == 0) {
        const int cbf = a.mode == GEMM_BF16_CVT ? 1 : 0;
        ConvTiling ct;
        bool use = pick_conv_tiling(a.ic.C, a.ic.H, a.ic.W, a.N, cbf, &ct);
        // BF16 math: every box passes through the conversion warps before its MMAs, which a CTA with a single channel
        // block (three boxes) cannot hide -- measured on 128 -> 128 @112: 29.7 us against 18.2 for the converting implicit
        // GEMM; with two or more blocks per CTA the halo kernel is ahead (64 -> 64 @224: 19.6 against 29.3 us,
        // 256 -> 256 @56: 20.4 against 26.2, 512 -> 512 @28: 20.7 against 26.9).
        if (use && cbf && ceil_div(a.ic.C, 32) / ct.splits < 2) use = false;
        if (tn.conv3x3 == 1) {
            use = false;
        } else if (tn.conv3x3 == 2) {
            ConvTiling f{};
            f.MT = tn.conv_mt; f.BN = tn.conv_bn; f.splits = tn.conv_splits; f.na = tn.conv_na; f.nb = tn.conv_nb;
            f.bf16 = cbf;
            if (f.splits <= ceil_div(a.ic.C, 32) && finish_conv_tiling(&f)) {
                ct = f;
                use = true;
            }
        }
        // The persistent form runs only on request.  Measured on B200 (VGG-shaped layers, L2 flushed): one resident
        // CTA per SM reaches 154 TFLOP/s on 64 -> 64 @ 224 and two reach 206, against 260 for two or three
        // one-tile CTAs per SM: inside one CTA the single MMA-issuing thread (about 82 cycles per tcgen05.mma
        // against 32 cycles of execution at N = 64) bounds the tile rate, and independent CTAs, each with its own
        // issuing thread, lift that bound where a second accumulator does not.
        // The weights-stationary form runs only on request.  Measured on B200 (64 -> 64, L2 flushed or not): 20.4 us on
        // a 224 x 224 image against 12.8 for the one-tile kernel, and 5.4 us for every further patch of a CTA.  One thread
        // issues one tcgen05.mma per ~82 cycles whatever N is, so the 72 MMAs (N = 64) of a patch take 3 us of issue time
        // alone where the tensor pipe needs 1.2; three one-tile CTAs per SM issue from three threads, and the resident
        // weights leave room for only three halo boxes in flight.
        int wbn = 0;
        if (!cbf && tn.convw == 2 && convw_fits(a, &wbn)) return launch_conv3x3_ws(a, wbn, st);
        if (!cbf && tn.convp == 2 && (size_t)tn.convp_bn <= (size_t)ceil_div(a.N, 16) * 16)
            return launch_conv3x3_persistent(a, tn.convp_bn, tn.convp_per_sm, tn.convp_na ? tn.convp_na : 2, tn.convp_nb ? tn.convp_nb : 4, st);
        if (use) return launch_conv3x3_tc(a, ct, st);
    }
    int tmem_cols = 32;
    while (tmem_cols < BN) tmem_cols *= 2;
    const uint32_t sb = (a.mode == GEMM_X3) ? stage_bytes_of<2>(BN) : (a.mode == GEMM_BF16_CVT) ? stage_bytes_of<3>(BN) : stage_bytes_of<0>(BN);
    int ring = ring_for(BN, (long long)m_tiles * ceil_div(a.N, BN) * a.batch * splits);
    if (tn.gemm_ring && (size_t)tn.gemm_ring * sb <= 210u * 1024u) ring = tn.gemm_ring;
    while (splits > 1 && ring < 8 && (uint32_t)ring * sb < (uint32_t)BM * (BN + 4) * 4u) ++ring;   // room to park the partial tile

    const bool bf16 = a.mode == GEMM_BF16;
    CUtensorMap tmA, tmB, tmD, tmAdd;
    GemmDev g;
    g.stamp = next_stamp();
    next_stamp() = nullptr;
    g.D = a.D; g.bias = a.bias; g.addend = a.addend;
    g.ldd = a.ldd; g.strideD = a.strideD;
    g.M = a.M; g.N = a.N; g.Kd = a.Kd; g.BN = BN; g.act = a.act; g.tmem_cols = tmem_cols; g.splits = splits; g.stages = ring; g.prefill = tn.gemm_prefill;
    g.ic_on = 0; g.ic_C = g.ic_cblk = g.ic_S = g.ic_OW = g.ic_stride = g.ic_pad = 0;
    if (a.ic.on) {
        NNV_REQUIRE((a.mode == GEMM_TF32 || a.mode == GEMM_BF16_CVT) && a.batch == 1, NNV_ERR_INVALID_ARG,
                    "implicit im2col needs fp32 activations (TF32 or converting BF16 mode) and one batch");
        NNV_TRY(encode_im2col_operand(&tmA, a.A, a.ic.C, a.ic.H, a.ic.W, a.ic.R, a.ic.S, a.ic.stride, a.ic.pad));
        g.ic_on = 1; g.ic_C = a.ic.C; g.ic_cblk = ceil_div(a.ic.C, 32); g.ic_S = a.ic.S; g.ic_OW = a.ic.OW;
        g.ic_stride = a.ic.stride; g.ic_pad = a.ic.pad;
        g.Kd = a.ic.R * a.ic.S * g.ic_cblk;                       // number of K blocks
    } else {
        NNV_TRY(encode_operand(&tmA, a.A, bf16, a.Kd, a.M, a.batch, a.lda, a.strideA, BM));
    }
    if (a.mode == GEMM_BF16_CVT) {
        NNV_REQUIRE(a.batch == 1, NNV_ERR_INVALID_ARG, "the converting BF16 mode needs one batch");
        NNV_TRY(encode_bf16_weight_chunks(&tmB, a.B, a.ldb, a.N, BN));
    } else {
        NNV_TRY(encode_operand(&tmB, a.B, bf16, a.Kd, a.N, a.batch, a.ldb, a.strideB, BN));
    }

    // Write-out by TMA through swizzled staging tiles when the output rows are 16-byte multiples (else plain stores).
    // A residual addend needs a staging tile of its own beside the ring: the ring gives up stages for it.
    if (a.addend && splits == 1)
        while (ring > 4 && (size_t)2048 + (size_t)ring * sb + 8 * (3 * 8 + 3) + (size_t)BM * BN * 4 > 220u * 1024u) --ring;
    g.stages = ring;
    const size_t ring_and_bars = (size_t)ring * sb + 8 * (3 * 8 + 3);
    size_t smem_bytes = (size_t)1024 + ring_and_bars;
    g.tma_out = 0;
    g.stage_off = 0;
    const bool out_ok = splits == 1 && (a.N % 4) == 0 && (a.ldd % 4) == 0 && (a.strideD % 4) == 0 &&
                        (reinterpret_cast<uintptr_t>(a.D) & 15) == 0 && (!a.addend || (reinterpret_cast<uintptr_t>(a.addend) & 15) == 0) &&
                        (!a.bias || (reinterpret_cast<uintptr_t>(a.bias) & 15) == 0) && (!a.addend || a.batch == 1);
    if (out_ok) {
        const int cw = (BN % 32) == 0 ? 32 : 16;
        size_t need = smem_bytes;
        uint32_t off = 0;
        if (a.addend) {                                          // the staging tile cannot share the ring: it is filled while the ring works
            off = (uint32_t)align_up(ring_and_bars, 1024);
            need = (size_t)1024 + off + (size_t)BM * BN * 4;
        }
        if (need <= 220u * 1024u) {
            g.tma_out = cw;
            g.stage_off = off;
            smem_bytes = need;
            NNV_TRY(encode_output(&tmD, a.D, a.N, a.M, a.batch, a.ldd, a.batch > 1 ? a.strideD : (int64_t)a.M * a.ldd, cw));
            if (a.addend) NNV_TRY(encode_output(&tmAdd, a.addend, a.N, a.M, 1, a.ldd, (int64_t)a.M * a.ldd, cw));
        }
    }
    if (!g.tma_out) tmD = tmA;                                   // unused by the kernel, but a kernel parameter must hold a valid object
    if (!g.tma_out || !a.addend) tmAdd = tmA;

    dim3 grid(m_tiles, ceil_div(a.N, BN), a.batch * splits);
    NNV_REQUIRE(grid.y <= 65535 && grid.z <= 65535, NNV_ERR_UNSUPPORTED, "GEMM grid too large");
    if (a.mode == GEMM_TF32)
        (void)launch_pdl_cluster(gemm_tc_kernel<0>, grid, dim3(GEMM_THREADS), smem_bytes, st, splits, tmA, tmB, tmD, tmAdd, g);
    else if (a.mode == GEMM_BF16)
        (void)launch_pdl_cluster(gemm_tc_kernel<1>, grid, dim3(GEMM_THREADS), smem_bytes, st, splits, tmA, tmB, tmD, tmAdd, g);
    else if (a.mode == GEMM_BF16_CVT)
        (void)launch_pdl_cluster(gemm_tc_kernel<3>, grid, dim3(GEMM_THREADS), smem_bytes, st, splits, tmA, tmB, tmD, tmAdd, g);
    else if (a.mode == GEMM_X3)
        (void)launch_pdl_cluster(gemm_tc_kernel<2>, grid, dim3(GEMM_THREADS), smem_bytes, st, splits, tmA, tmB, tmD, tmAdd, g);
    else
        return fail(NNV_ERR_INVALID_ARG, "unknown GEMM mode %d", a.mode);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

}  // namespace nnv
