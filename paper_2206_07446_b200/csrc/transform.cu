// Weight-transformation kernels (memory-bound): Winograd filter transform U = G g G^T for
// F(2x2,3x3), F(4x4,3x3), F(6x6,3x3), and the GEMM-ready repack.  This is the paper's "weights
// transformation" stage (its Section 2 and Figure 3), run on the device.
#include <cuda_bf16.h>

#include "nnv_internal.h"

namespace nnv {

// G matrices of the Cook-Toom construction with points {0, +-1, +-2, +-1/2, inf} (the published
// F(m,3) minimal-filtering matrices); row j belongs to point j, the last row to infinity.
template <int M_> struct WinoG;
template <> struct WinoG<2> {
    static constexpr int A = 4;
    __host__ __device__ static constexpr float g(int r, int c) {
        constexpr float t[4][3] = {{1.f, 0.f, 0.f}, {.5f, .5f, .5f}, {.5f, -.5f, .5f}, {0.f, 0.f, 1.f}};
        return t[r][c];
    }
};
template <> struct WinoG<4> {
    static constexpr int A = 6;
    __host__ __device__ static constexpr float g(int r, int c) {
        constexpr float t[6][3] = {{1.f / 4.f, 0.f, 0.f},
                                   {-1.f / 6.f, -1.f / 6.f, -1.f / 6.f},
                                   {-1.f / 6.f, 1.f / 6.f, -1.f / 6.f},
                                   {1.f / 24.f, 1.f / 12.f, 1.f / 6.f},
                                   {1.f / 24.f, -1.f / 12.f, 1.f / 6.f},
                                   {0.f, 0.f, 1.f}};
        return t[r][c];
    }
};
template <> struct WinoG<6> {
    static constexpr int A = 8;
    __host__ __device__ static constexpr float g(int r, int c) {
        constexpr float t[8][3] = {{1.f, 0.f, 0.f},
                                   {-2.f / 9.f, -2.f / 9.f, -2.f / 9.f},
                                   {-2.f / 9.f, 2.f / 9.f, -2.f / 9.f},
                                   {1.f / 90.f, 1.f / 45.f, 2.f / 45.f},
                                   {1.f / 90.f, -1.f / 45.f, 2.f / 45.f},
                                   {32.f / 45.f, 16.f / 45.f, 8.f / 45.f},
                                   {32.f / 45.f, -16.f / 45.f, 8.f / 45.f},
                                   {0.f, 0.f, 1.f}};
        return t[r][c];
    }
};

template <typename OutT, int NF> struct VecStore;
template <> struct VecStore<float, 1> {
    __device__ static void st(float* p, const float* v) { *p = v[0]; }
};
template <> struct VecStore<float, 2> {
    __device__ static void st(float* p, const float* v) { *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]); }
};
template <> struct VecStore<float, 4> {
    __device__ static void st(float* p, const float* v) {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct VecStore<__nv_bfloat16, 2> {
    __device__ static void st(__nv_bfloat16* p, const float* v) {
        *reinterpret_cast<__nv_bfloat162*>(p) = __floats2bfloat162_rn(v[0], v[1]);
    }
};
template <> struct VecStore<__nv_bfloat16, 4> {
    __device__ static void st(__nv_bfloat16* p, const float* v) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
        __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
        uint2 u;
        u.x = *reinterpret_cast<uint32_t*>(&a);
        u.y = *reinterpret_cast<uint32_t*>(&b);
        *reinterpret_cast<uint2*>(p) = u;
    }
};

template <> struct VecStore<__nv_bfloat16, 8> {
    __device__ static void st(__nv_bfloat16* p, const float* v) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
        __nv_bfloat162 c = __floats2bfloat162_rn(v[4], v[5]), d = __floats2bfloat162_rn(v[6], v[7]);
        uint4 u;
        u.x = *reinterpret_cast<uint32_t*>(&a);
        u.y = *reinterpret_cast<uint32_t*>(&b);
        u.z = *reinterpret_cast<uint32_t*>(&c);
        u.w = *reinterpret_cast<uint32_t*>(&d);
        *reinterpret_cast<uint4*>(p) = u;
    }
};

constexpr int FT_THREADS = 256;
constexpr int FT_FILTERS = 1024;                                // most filters (padded (k, c) pairs) a block takes
// Filters of one block: every thread busy, at most FT_FILTERS (which the shared staging buffer holds).
__host__ __device__ constexpr int ft_filters(int nf) { return FT_THREADS * nf > FT_FILTERS ? FT_FILTERS : FT_THREADS * nf; }
// Filters per thread.  F(2x2,3x3): as many as make every store of a thread 16 bytes wide (4 fp32 or 8 bf16
// values).  F(4x4,3x3) and F(6x6,3x3) keep 2 -- four filters' intermediates need 128 registers and halve the
// resident warps (measured: 1024^2 filters 47 us against 41) -- and reach 16-byte stores by exchanging halves
// between neighbouring lanes: of every pair of planes the even lane stores one plane for both lanes' filters
// and the odd lane the other.
template <int M_, typename OutT> struct FtNF { static constexpr int value = (M_ == 2) ? 4 : 2; };
template <int M_> struct FtNF<M_, __nv_bfloat16> { static constexpr int value = (M_ == 2) ? 8 : 2; };

// One thread transforms NF filters that are adjacent in the padded channel index, so that each of the alpha^2
// output planes receives one NF-wide (16-byte) vector store per thread and a warp writes 32*NF consecutive
// elements of the plane.  A block covers FT_FILTERS filters with FT_FILTERS / NF of its threads.  With C == Cp
// the block's raw filters are one contiguous range, staged through shared memory with 128-bit loads by all
// threads and read back with 128-bit loads (a thread's NF * 9 floats start on a 16-byte boundary; the eight
// threads of a quarter warp then touch all 32 banks once).
template <int M_, typename OutT, int NF>
__device__ __forceinline__ void filter_transform_block(const float* __restrict__ g, OutT* __restrict__ U, int K, int C,
                                                       int Cp, unsigned block, float* sg, bool late_wait) {
    constexpr int A = WinoG<M_>::A;
    constexpr int FPB = ft_filters(NF);                          // filters of this block
    constexpr int ACTIVE = FPB / NF;                              // threads that transform
    const long long F = (long long)K * Cp;                      // padded filter count = plane size
    const long long f_block = (long long)block * FPB;
    const long long f0 = f_block + (long long)threadIdx.x * NF;
    const bool contiguous = (C == Cp);

    if (contiguous) {
        const long long total = (long long)K * C * 9;             // multiple of 4 because C % 8 == 0
        const long long base = f_block * 9;
        const float4* src = reinterpret_cast<const float4*>(g + base);
        float4* dst = reinterpret_cast<float4*>(sg);
        constexpr int NV = FPB * 9 / 4;
        for (int i = threadIdx.x; i < NV; i += FT_THREADS) {
            if (base + 4ll * i < total) dst[i] = __ldg(src + i);
        }
        __syncthreads();
    }
    // Weights read in place from host memory do not depend on the previous kernel of the stream: those loads were
    // issued above, before this wait (which then only orders the stores below).
    if (late_wait) pdl_wait();
    if ((int)threadIdx.x >= ACTIVE || f0 >= F) return;

    float w[NF][9];
    bool pad[NF];
    if (contiguous) {
        float flat[NF * 9];
        if constexpr ((NF * 9) % 4 == 0) {
            const float4* s4 = reinterpret_cast<const float4*>(sg + (size_t)threadIdx.x * NF * 9);
#pragma unroll
            for (int i = 0; i < NF * 9 / 4; ++i) {
                const float4 v = s4[i];
                flat[4 * i] = v.x; flat[4 * i + 1] = v.y; flat[4 * i + 2] = v.z; flat[4 * i + 3] = v.w;
            }
        } else {                                                  // NF = 2: 18 floats on an 8-byte boundary, conflict-free as 64-bit loads
            const float2* s2 = reinterpret_cast<const float2*>(sg + (size_t)threadIdx.x * NF * 9);
#pragma unroll
            for (int i = 0; i < NF * 9 / 2; ++i) {
                const float2 v = s2[i];
                flat[2 * i] = v.x; flat[2 * i + 1] = v.y;
            }
        }
#pragma unroll
        for (int j = 0; j < NF; ++j) {
            pad[j] = false;
#pragma unroll
            for (int i = 0; i < 9; ++i) w[j][i] = flat[j * 9 + i];
        }
    } else {
#pragma unroll
        for (int j = 0; j < NF; ++j) {
            const long long f = f0 + j;
            const int k = (int)(f / Cp), c = (int)(f % Cp);
            pad[j] = c >= C;
#pragma unroll
            for (int i = 0; i < 9; ++i) w[j][i] = (c < C) ? __ldg(g + ((long long)k * C + c) * 9 + i) : 0.f;
        }
    }

    // t[i][nu] = sum_j g[i][j] * G[nu][j]
    float t[NF][3][A];
#pragma unroll
    for (int j = 0; j < NF; ++j)
#pragma unroll
        for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int nu = 0; nu < A; ++nu)
                t[j][i][nu] = w[j][i * 3 + 0] * WinoG<M_>::g(nu, 0) + w[j][i * 3 + 1] * WinoG<M_>::g(nu, 1) +
                              w[j][i * 3 + 2] * WinoG<M_>::g(nu, 2);

    // U[xi][nu] = sum_i G[xi][i] * t[i][nu]; plane xi*A+nu, element f0..f0+NF-1
    OutT* out = U + f0;
    auto plane_values = [&](int xi, int nu, float* v) {
#pragma unroll
        for (int j = 0; j < NF; ++j) {
            v[j] = WinoG<M_>::g(xi, 0) * t[j][0][nu] + WinoG<M_>::g(xi, 1) * t[j][1][nu] + WinoG<M_>::g(xi, 2) * t[j][2][nu];
            if (pad[j]) v[j] = 0.f;                              // padded channels hold +0, never -0
        }
    };
    if constexpr (NF == 2 && sizeof(OutT) == 4) {
        // pairs of planes (A is even): lanes 2i and 2i+1 hold four adjacent filters between them (the plane size is a
        // multiple of 8, so both are live or neither); each sends the partner its two values of the plane the partner stores
        const unsigned live = __activemask();
        const bool odd = (threadIdx.x & 1) != 0;
#pragma unroll
        for (int xi = 0; xi < A; ++xi) {
#pragma unroll
            for (int nu = 0; nu < A; nu += 2) {
                float vp[2], vq[2];
                plane_values(xi, nu, vp);
                plane_values(xi, nu + 1, vq);
                const float s0 = __shfl_xor_sync(live, odd ? vp[0] : vq[0], 1);
                const float s1 = __shfl_xor_sync(live, odd ? vp[1] : vq[1], 1);
                float v4[4];
                if (!odd) { v4[0] = vp[0]; v4[1] = vp[1]; v4[2] = s0; v4[3] = s1; }
                else { v4[0] = s0; v4[1] = s1; v4[2] = vq[0]; v4[3] = vq[1]; }
                OutT* dst = out + (long long)(xi * A + nu + (odd ? 1 : 0)) * F - (odd ? 2 : 0);
                VecStore<OutT, 4>::st(dst, v4);
            }
        }
    } else {
#pragma unroll
        for (int xi = 0; xi < A; ++xi) {
#pragma unroll
            for (int nu = 0; nu < A; ++nu) {
                float v[NF];
                plane_values(xi, nu, v);
                VecStore<OutT, NF>::st(out + (long long)(xi * A + nu) * F, v);
            }
        }
    }
}

constexpr int XF_SMEM_FLOATS = FT_FILTERS * 9;                   // 36 KB staging buffer shared by all transform kernels

template <int M_, typename OutT, int NF>
__global__ void __launch_bounds__(FT_THREADS)
filter_transform_kernel(const float* __restrict__ g, OutT* __restrict__ U, int K, int C, int Cp, unsigned long long* stamp,
                        int host_src) {
    pdl_trigger();
    if (!host_src) pdl_wait();
    if (threadIdx.x == 0) stamp_start(stamp);
    __shared__ __align__(16) float sg[XF_SMEM_FLOATS];
    filter_transform_block<M_, OutT, NF>(g, U, K, C, Cp, blockIdx.x, sg, host_src != 0);
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(stamp);
}

template <int M_, typename OutT>
static nnv_status_t launch_ft(const float* g, void* U, int K, int C, int Cp, cudaStream_t st, bool host_src) {
    constexpr int NF = FtNF<M_, OutT>::value;
    const long long F = (long long)K * Cp;
    const unsigned grid = (unsigned)((F + ft_filters(NF) - 1) / ft_filters(NF));
    unsigned long long* stamp = next_stamp();
    next_stamp() = nullptr;
    NNV_LAUNCH((filter_transform_kernel<M_, OutT, NF>), grid, FT_THREADS, 0, st, g, reinterpret_cast<OutT*>(U), K, C, Cp, stamp,
               host_src ? 1 : 0);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

nnv_status_t launch_filter_transform(int m, bool bf16, const float* g, void* U, int K, int C, int Cp,
                                     cudaStream_t st, bool host_src) {
    switch (m) {
        case 2: return bf16 ? launch_ft<2, __nv_bfloat16>(g, U, K, C, Cp, st, host_src) : launch_ft<2, float>(g, U, K, C, Cp, st, host_src);
        // F(4,3) and F(6,3) exist with fp32 U only: their tile GEMM multiplies fp32 operands (one bf16 pass in
        // those domains misses the output tolerance of the bf16 class)
        case 4: NNV_REQUIRE(!bf16, NNV_ERR_UNSUPPORTED, "F(4x4,3x3) has no bf16 filter transform"); return launch_ft<4, float>(g, U, K, C, Cp, st, host_src);
        case 6: NNV_REQUIRE(!bf16, NNV_ERR_UNSUPPORTED, "F(6x6,3x3) has no bf16 filter transform"); return launch_ft<6, float>(g, U, K, C, Cp, st, host_src);
        default: return fail(NNV_ERR_INVALID_ARG, "no Winograd tile size %d", m);
    }
}

// ---- GEMM-ready repack ----------------------------------------------------------------------
// Elements are rounded to the precision the tensor core will use: TF32 (stored as fp32 words) or
// bf16, round to nearest even, so the hardware never truncates the weights.
// fp32 -> TF32 precision (10 explicit mantissa bits), round to nearest even, by integer arithmetic;
// the result is an fp32 word whose low 13 mantissa bits are zero.
__device__ __forceinline__ float round_tf32(float v) {
    uint32_t b = __float_as_uint(v);
    b += 0xFFFu + ((b >> 13) & 1u);
    return __uint_as_float(b & 0xFFFFE000u);
}
template <typename OutT> __device__ inline OutT cvt_out(float v);
template <> __device__ inline float cvt_out<float>(float v) { return round_tf32(v); }
template <> __device__ inline __nv_bfloat16 cvt_out<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

constexpr int PACK_THREADS = 256;
constexpr int PACK_SMEM_FLOATS = XF_SMEM_FLOATS;
constexpr int PACK1X1_PER_BLOCK = PACK_THREADS * 16;            // elements of P one block of pack1x1 writes

template <typename OutT> __device__ __forceinline__ void store4(OutT* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(round_tf32(a), round_tf32(b), round_tf32(c), round_tf32(d));
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
    __nv_bfloat162 x = __floats2bfloat162_rn(a, b), y = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&x);
    u.y = *reinterpret_cast<uint32_t*>(&y);
    *reinterpret_cast<uint2*>(p) = u;
}

// Repack of R*S > 1 filters.  Work unit = (output channel k, chunk of CH input channels): CH*RS
// contiguous raw floats in, RS segments of CH consecutive elements out -- a transpose of the
// (c, rs) index pair.  One WARP owns a unit and stages it in its private slice of shared memory
// (only __syncwarp between its coalesced loads and its coalesced stores), so the eight warps of
// a block stream independently and many loads stay in flight.  CH = 32 (128-byte store segments)
// while 32*RS floats fit the slice, else 8.  The pad q in [R*S*C, Qp) is written as +0 by the
// unit of the row's last chunk.
constexpr int PACK_WARPS = PACK_THREADS / 32;
constexpr int PACK_SLICE = PACK_SMEM_FLOATS / PACK_WARPS;        // floats of shared memory per warp

__host__ __device__ inline int pack_ch(int RS) { return 32 * RS <= PACK_SLICE ? 32 : 8; }
__host__ __device__ inline int pack_units_per_row(int C, int RS) { return (C + pack_ch(RS) - 1) / pack_ch(RS); }

// Fast repack for the common case C % 64 == 0 (then R*S*C needs no padding): a block stages a
// contiguous range of PACK_NF filters (k, c pairs; PACK_NF * RS floats) with 128-bit loads, as the
// filter transform does, and writes the transposed (rs, c) order with 128-bit stores -- consecutive
// threads write consecutive 16-byte words of one (k, rs) segment.
constexpr int PACK_NF = 512;
__host__ __device__ inline bool pack_fast(int C, int RS) {
    return RS > 1 && (C % 64) == 0 && PACK_NF * RS <= PACK_SMEM_FLOATS && (C >= PACK_NF ? C % PACK_NF == 0 : PACK_NF % C == 0);
}

template <typename OutT>
__device__ __forceinline__ void pack_fast_block(const float* __restrict__ w, OutT* __restrict__ P, int K, int C, int RS,
                                                int Qp, unsigned block, float* sg, bool late_wait) {
    const long long F = (long long)K * C;
    const long long f_block = (long long)block * PACK_NF;
    const int nf = (int)min((long long)PACK_NF, F - f_block);    // multiple of 64
    const float4* src = reinterpret_cast<const float4*>(w + f_block * RS);
    float4* dst = reinterpret_cast<float4*>(sg);
    const int nv = nf * RS / 4;
    for (int i = threadIdx.x; i < nv; i += PACK_THREADS) dst[i] = __ldg(src + i);
    __syncthreads();
    if (late_wait) pdl_wait();                                    // host weights were loaded above; only the stores wait
    const int Cb = min(C, PACK_NF);                               // channels of one k row inside this block
    const int k0 = (int)(f_block / C), cbase = (int)(f_block - (long long)k0 * C);
    // Write-out.  A row is one (k, rs) pair: Cb consecutive output elements.  A warp takes four
    // consecutive rows x 32 channels: lane = 8 * (row in the group) + (16-byte word of the chunk).
    // Each lane gathers its four channels from the staged (c, rs) order; the 32 addresses of one
    // such gather differ by 36 words along the chunk and by 1 word along the rows, i.e. they fall
    // in 32 different banks.  Each group of eight lanes stores 128 contiguous bytes.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nch = Cb >> 5;                                      // 32-channel chunks per row (a power of two)
    const int rows = (nf / Cb) * RS;
    const int items = ((rows + 3) >> 2) * nch;
    const int sub = lane >> 3, c = (lane & 7) * 4;
    const int nch_log = __ffs(nch) - 1;
    for (int item = warp; item < items; item += PACK_WARPS) {
        const int g = item >> nch_log, ch = item & (nch - 1);
        const int row = 4 * g + sub;
        if (row >= rows) continue;
        const int kl = row / RS, rs = row - kl * RS;
        const int cc = ch * 32 + c;
        const float* s = sg + ((kl * Cb + cc) * RS + rs);
        store4<OutT>(P + (long long)(k0 + kl) * Qp + (long long)rs * C + cbase + cc, s[0], s[RS], s[2 * RS], s[3 * RS]);
    }
}

template <typename OutT>
__device__ __forceinline__ void pack_block(const float* __restrict__ w, OutT* __restrict__ P, int K, int C, int RS, int Qp,
                                           unsigned block, float* smem, bool late_wait) {
    if (pack_fast(C, RS)) {
        pack_fast_block<OutT>(w, P, K, C, RS, Qp, block, smem, late_wait);
        return;
    }
    if (late_wait) pdl_wait();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int CH = pack_ch(RS), upr = pack_units_per_row(C, RS);
    const long long unit = (long long)block * PACK_WARPS + warp;
    if (unit >= (long long)K * upr) return;
    const int k = (int)(unit / upr), c0 = (int)(unit - (long long)k * upr) * CH;
    const int cc = min(CH, C - c0), n = cc * RS;
    float* sw = smem + warp * PACK_SLICE;
    const float* src = w + ((long long)k * C + c0) * RS;
    OutT* dst = P + (long long)k * Qp;
    for (int i = lane; i < n; i += 32) sw[i] = __ldg(src + i);
    __syncwarp();
    if (CH == 32) {
        for (int rs = 0; rs < RS; ++rs)
            if (lane < cc) dst[(long long)rs * C + c0 + lane] = cvt_out<OutT>(sw[lane * RS + rs]);
    } else {
        for (int i = lane; i < n; i += 32) {
            const int rs = i / cc, c = i - rs * cc;
            dst[(long long)rs * C + c0 + c] = cvt_out<OutT>(sw[c * RS + rs]);
        }
    }
    if (c0 + cc == C)
        for (int q = C * RS + lane; q < Qp; q += 32) dst[q] = cvt_out<OutT>(0.f);
}

// 1x1 filters: the repack is a row-padded copy (and conversion); one block writes
// PACK1X1_PER_BLOCK consecutive elements of P.
template <typename OutT>
__device__ __forceinline__ void pack1x1_block(const float* __restrict__ w, OutT* __restrict__ P, int K, int C, int Qp,
                                              unsigned block, bool late_wait) {
    const long long n = (long long)K * Qp;
    const long long base = (long long)block * PACK1X1_PER_BLOCK;
    if (C == Qp) {                                              // no padding: a straight conversion copy, 4 at a time
        float4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {                             // all loads first: four 16-byte requests in flight per thread
            const long long i = base + ((long long)u * PACK_THREADS + threadIdx.x) * 4;
            if (i < n) v[u] = __ldg(reinterpret_cast<const float4*>(w + i));
        }
        if (late_wait) pdl_wait();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const long long i = base + ((long long)u * PACK_THREADS + threadIdx.x) * 4;
            if (i < n) store4<OutT>(P + i, v[u].x, v[u].y, v[u].z, v[u].w);
        }
    } else {
        if (late_wait) pdl_wait();
#pragma unroll
        for (int u = 0; u < 16; ++u) {
            const long long i = base + (long long)u * PACK_THREADS + threadIdx.x;
            if (i < n) {
                const int k = (int)(i / Qp), q = (int)(i - (long long)k * Qp);
                P[i] = cvt_out<OutT>(q < C ? __ldg(w + (long long)k * C + q) : 0.f);
            }
        }
    }
}

template <typename OutT>
__global__ void __launch_bounds__(PACK_THREADS)
pack_kernel(const float* __restrict__ w, OutT* __restrict__ P, int K, int C, int RS, int Qp, unsigned long long* stamp, int host_src) {
    pdl_trigger();
    if (!host_src) pdl_wait();
    if (threadIdx.x == 0) stamp_start(stamp);
    __shared__ __align__(16) float sw[PACK_SMEM_FLOATS];
    pack_block<OutT>(w, P, K, C, RS, Qp, blockIdx.x, sw, host_src != 0);
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(stamp);
}

template <typename OutT>
__global__ void __launch_bounds__(PACK_THREADS)
pack1x1_kernel(const float* __restrict__ w, OutT* __restrict__ P, int K, int C, int Qp, unsigned long long* stamp, int host_src) {
    pdl_trigger();
    if (!host_src) pdl_wait();
    if (threadIdx.x == 0) stamp_start(stamp);
    pack1x1_block<OutT>(w, P, K, C, Qp, blockIdx.x, host_src != 0);
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(stamp);
}

// ---- many layers in one launch ----------------------------------------------------------------
// Block b belongs to the descriptor whose [block0, block0 + blocks) range holds it and does there
// exactly what the single-layer kernels do.  A batch of small layers then costs one launch and
// presents the memory system with one large stream of work.  The kernel is instantiated per group
// of transform kinds (repacks / F(2,3) and F(4,3) / F(6,3)) so that the register allocation, and with
// it the number of resident warps, is that of the group's own code and not of the largest transform.
enum { XG_PACK = 0, XG_WINO_SMALL = 1, XG_WINO6 = 2, XG_COUNT = 3 };
__host__ __device__ inline int xform_group(int kind) {
    return kind == XF_WINO6 ? XG_WINO6 : (kind == XF_WINO2 || kind == XF_WINO4) ? XG_WINO_SMALL : XG_PACK;
}

template <int GROUP>
__global__ void __launch_bounds__(FT_THREADS)
multi_transform_kernel(const __grid_constant__ XformBatch batch) {
    pdl_trigger();
    const bool late = batch.host_src != 0;                      // sources in host memory: load first, wait before the stores
    if (!late) pdl_wait();
    if (threadIdx.x == 0) stamp_start(batch.stamp);
    __shared__ __align__(16) float smem[XF_SMEM_FLOATS];
    const unsigned vb = blockIdx.x;
    int di = 0;
    for (int i = 1; i < batch.n; ++i)
        if (vb >= (unsigned)batch.d[i].block0) di = i;
    const XformDesc& d = batch.d[di];
    const unsigned lb = vb - (unsigned)d.block0;
    const float* src = static_cast<const float*>(d.src);
    if constexpr (GROUP == XG_PACK) {
        switch (d.kind * 2 + d.bf16) {
            case XF_PACK * 2: pack_block<float>(src, (float*)d.dst, d.K, d.C, d.RS, d.Qp, lb, smem, late); break;
            case XF_PACK * 2 + 1: pack_block<__nv_bfloat16>(src, (__nv_bfloat16*)d.dst, d.K, d.C, d.RS, d.Qp, lb, smem, late); break;
            case XF_PACK1X1 * 2: pack1x1_block<float>(src, (float*)d.dst, d.K, d.C, d.Qp, lb, late); break;
            case XF_PACK1X1 * 2 + 1: pack1x1_block<__nv_bfloat16>(src, (__nv_bfloat16*)d.dst, d.K, d.C, d.Qp, lb, late); break;
            default: break;
        }
    } else if constexpr (GROUP == XG_WINO_SMALL) {
        switch (d.kind * 2 + d.bf16) {
            case XF_WINO2 * 2: filter_transform_block<2, float, 4>(src, (float*)d.dst, d.K, d.C, d.Cp, lb, smem, late); break;
            case XF_WINO2 * 2 + 1: filter_transform_block<2, __nv_bfloat16, 8>(src, (__nv_bfloat16*)d.dst, d.K, d.C, d.Cp, lb, smem, late); break;
            case XF_WINO4 * 2: filter_transform_block<4, float, 2>(src, (float*)d.dst, d.K, d.C, d.Cp, lb, smem, late); break;
            default: break;
        }
    } else {
        if (d.kind == XF_WINO6 && !d.bf16) filter_transform_block<6, float, 2>(src, (float*)d.dst, d.K, d.C, d.Cp, lb, smem, late);
    }
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(batch.stamp);
}

static long long pack_blocks(int K, int C, int RS) {
    if (pack_fast(C, RS)) return ((long long)K * C + PACK_NF - 1) / PACK_NF;
    return ((long long)K * pack_units_per_row(C, RS) + PACK_WARPS - 1) / PACK_WARPS;
}

int xform_blocks(const XformDesc& d) {
    switch (d.kind) {
        case XF_PACK: return (int)pack_blocks(d.K, d.C, d.RS);
        case XF_PACK1X1: return (int)(((long long)d.K * d.Qp + PACK1X1_PER_BLOCK - 1) / PACK1X1_PER_BLOCK);
        default: {                                              // the block size of the kind's instantiation in multi_transform_kernel
            const int fpb = d.kind == XF_WINO2 ? ft_filters(d.bf16 ? 8 : 4) : ft_filters(2);
            return (int)(((long long)d.K * d.Cp + fpb - 1) / fpb);
        }
    }
}

nnv_status_t launch_transform_batch(XformDesc* descs, int n, cudaStream_t st) {
    unsigned long long* stamp = next_stamp();                  // every launch of the batch stamps the same slot
    next_stamp() = nullptr;
    for (int grp = 0; grp < XG_COUNT; ++grp) {
        XformBatch b;
        b.stamp = stamp;
        b.host_src = (n > 0 && descs[0].host_src) ? 1 : 0;      // a batch is all device or all host sources
        b.n = 0;
        int blocks = 0;
        auto flush = [&]() -> nnv_status_t {
            if (b.n == 0) return NNV_OK;
            b.total_blocks = blocks;
            if (grp == XG_PACK) NNV_LAUNCH((multi_transform_kernel<XG_PACK>), blocks, FT_THREADS, 0, st, b);
            else if (grp == XG_WINO_SMALL) NNV_LAUNCH((multi_transform_kernel<XG_WINO_SMALL>), blocks, FT_THREADS, 0, st, b);
            else NNV_LAUNCH((multi_transform_kernel<XG_WINO6>), blocks, FT_THREADS, 0, st, b);
            NNV_CUDA(cudaGetLastError());
            b.n = 0;
            blocks = 0;
            return NNV_OK;
        };
        for (int i = 0; i < n; ++i) {
            if (xform_group(descs[i].kind) != grp) continue;
            XformDesc d = descs[i];
            NNV_REQUIRE(d.kind != XF_PACK || 8 * d.RS <= PACK_SLICE, NNV_ERR_UNSUPPORTED,
                        "filter window of %d taps is too large to repack", d.RS);
            d.block0 = blocks;
            blocks += xform_blocks(d);
            b.d[b.n++] = d;
            if (b.n == XF_BATCH_MAX) NNV_TRY(flush());
        }
        NNV_TRY(flush());
    }
    return NNV_OK;
}

nnv_status_t launch_pack(bool bf16, const float* w, void* P, int K, int C, int RS, int Qp, cudaStream_t st, bool host_src) {
    const int hs = host_src ? 1 : 0;
    unsigned long long* stamp = next_stamp();
    next_stamp() = nullptr;
    if (RS == 1) {
        const long long n = (long long)K * Qp;
        const unsigned grid = (unsigned)((n + PACK1X1_PER_BLOCK - 1) / PACK1X1_PER_BLOCK);
        if (bf16) NNV_LAUNCH((pack1x1_kernel<__nv_bfloat16>), grid, PACK_THREADS, 0, st, w, (__nv_bfloat16*)P, K, C, Qp, stamp, hs);
        else NNV_LAUNCH((pack1x1_kernel<float>), grid, PACK_THREADS, 0, st, w, (float*)P, K, C, Qp, stamp, hs);
    } else {
        NNV_REQUIRE(8 * RS <= PACK_SLICE, NNV_ERR_UNSUPPORTED, "filter window of %d taps is too large to repack", RS);
        const unsigned grid = (unsigned)pack_blocks(K, C, RS);
        if (bf16) NNV_LAUNCH((pack_kernel<__nv_bfloat16>), grid, PACK_THREADS, 0, st, w, (__nv_bfloat16*)P, K, C, RS, Qp, stamp, hs);
        else NNV_LAUNCH((pack_kernel<float>), grid, PACK_THREADS, 0, st, w, (float*)P, K, C, RS, Qp, stamp, hs);
    }
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

}  // namespace nnv
