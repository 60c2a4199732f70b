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

constexpr int FT_THREADS = 256;

// One thread transforms NF filters that are adjacent in the padded channel index, so that each
// of the alpha^2 output planes receives one NF-wide vector store per thread and a warp writes
// 32*NF consecutive elements of the plane.  With C == Cp the block's raw filters are one
// contiguous range, staged through shared memory with 128-bit loads.
template <int M_, typename OutT, int NF>
__global__ void __launch_bounds__(FT_THREADS)
filter_transform_kernel(const float* __restrict__ g, OutT* __restrict__ U, int K, int C, int Cp) {
    pdl_enter();
    constexpr int A = WinoG<M_>::A;
    __shared__ __align__(16) float sg[FT_THREADS * NF * 9];
    const long long F = (long long)K * Cp;                      // padded filter count = plane size
    const long long f_block = (long long)blockIdx.x * (FT_THREADS * NF);
    const long long f0 = f_block + (long long)threadIdx.x * NF;
    const bool contiguous = (C == Cp);

    if (contiguous) {
        const long long total = (long long)K * C * 9;             // multiple of 4 because C % 8 == 0
        const long long base = f_block * 9;
        const float4* src = reinterpret_cast<const float4*>(g + base);
        float4* dst = reinterpret_cast<float4*>(sg);
        constexpr int NV = FT_THREADS * NF * 9 / 4;
        for (int i = threadIdx.x; i < NV; i += FT_THREADS) {
            if (base + 4ll * i < total) dst[i] = __ldg(src + i);
        }
        __syncthreads();
    }
    if (f0 >= F) return;

    float w[NF][9];
    bool pad[NF];
#pragma unroll
    for (int j = 0; j < NF; ++j) {
        pad[j] = false;
        if (contiguous) {
#pragma unroll
            for (int i = 0; i < 9; ++i) w[j][i] = sg[(threadIdx.x * NF + j) * 9 + i];
        } else {
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
#pragma unroll
    for (int xi = 0; xi < A; ++xi) {
#pragma unroll
        for (int nu = 0; nu < A; ++nu) {
            float v[NF];
#pragma unroll
            for (int j = 0; j < NF; ++j)
                v[j] = WinoG<M_>::g(xi, 0) * t[j][0][nu] + WinoG<M_>::g(xi, 1) * t[j][1][nu] +
                       WinoG<M_>::g(xi, 2) * t[j][2][nu];
#pragma unroll
            for (int j = 0; j < NF; ++j)
                if (pad[j]) v[j] = 0.f;                          // padded channels hold +0, never -0
            VecStore<OutT, NF>::st(out + (long long)(xi * A + nu) * F, v);
        }
    }
}

template <int M_, typename OutT>
static nnv_status_t launch_ft(const float* g, void* U, int K, int C, int Cp, cudaStream_t st) {
    constexpr int NF = 2;
    const long long F = (long long)K * Cp;
    const long long per_block = (long long)FT_THREADS * NF;
    const unsigned grid = (unsigned)((F + per_block - 1) / per_block);
    NNV_LAUNCH((filter_transform_kernel<M_, OutT, NF>), grid, FT_THREADS, 0, st, g, reinterpret_cast<OutT*>(U), K, C, Cp);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

nnv_status_t launch_filter_transform(int m, bool bf16, const float* g, void* U, int K, int C, int Cp,
                                     cudaStream_t st) {
    switch (m) {
        case 2: return bf16 ? launch_ft<2, __nv_bfloat16>(g, U, K, C, Cp, st) : launch_ft<2, float>(g, U, K, C, Cp, st);
        case 4: return bf16 ? launch_ft<4, __nv_bfloat16>(g, U, K, C, Cp, st) : launch_ft<4, float>(g, U, K, C, Cp, st);
        case 6: return bf16 ? launch_ft<6, __nv_bfloat16>(g, U, K, C, Cp, st) : launch_ft<6, float>(g, U, K, C, Cp, st);
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
constexpr int PACK_SMEM_FLOATS = 8192;

// One block per output channel k.  The row W[k][c][rs] (contiguous) is staged through shared
// memory in channel chunks and written back as P[k][rs*C + c]: a transpose of the (c, rs)
// index pair, coalesced on both sides; the pad q in [R*S*C, Qp) is written as +0.
template <typename OutT>
__global__ void __launch_bounds__(PACK_THREADS)
pack_kernel(const float* __restrict__ w, OutT* __restrict__ P, int C, int RS, int Qp) {
    pdl_enter();
    __shared__ float sw[PACK_SMEM_FLOATS];
    const int k = blockIdx.x;
    const long long Q = (long long)C * RS;
    const float* src = w + (long long)k * Q;
    OutT* dst = P + (long long)k * Qp;
    const int CC = PACK_SMEM_FLOATS / RS;                      // channels per chunk
    for (int c0 = 0; c0 < C; c0 += CC) {
        const int cc = min(CC, C - c0);
        const int n = cc * RS;
        for (int i = threadIdx.x; i < n; i += PACK_THREADS) sw[i] = __ldg(src + (long long)c0 * RS + i);
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += PACK_THREADS) {
            const int rs = i / cc, c = i - rs * cc;
            dst[(long long)rs * C + c0 + c] = cvt_out<OutT>(sw[c * RS + rs]);
        }
        __syncthreads();
    }
    for (int q = (int)Q + threadIdx.x; q < Qp; q += PACK_THREADS) dst[q] = cvt_out<OutT>(0.f);
}

// 1x1 filters: the repack is a row-padded copy (and conversion).
template <typename OutT>
__global__ void __launch_bounds__(PACK_THREADS)
pack1x1_kernel(const float* __restrict__ w, OutT* __restrict__ P, int K, int C, int Qp) {
    pdl_enter();
    const long long n = (long long)K * Qp;
    for (long long i = (long long)blockIdx.x * PACK_THREADS + threadIdx.x; i < n; i += (long long)gridDim.x * PACK_THREADS) {
        const int k = (int)(i / Qp), q = (int)(i - (long long)k * Qp);
        P[i] = cvt_out<OutT>(q < C ? __ldg(w + (long long)k * C + q) : 0.f);
    }
}

nnv_status_t launch_pack(bool bf16, const float* w, void* P, int K, int C, int RS, int Qp, cudaStream_t st) {
    if (RS == 1) {
        const long long n = (long long)K * Qp;
        const unsigned grid = (unsigned)std::min<long long>((n + PACK_THREADS - 1) / PACK_THREADS, 148 * 16);
        if (bf16) NNV_LAUNCH((pack1x1_kernel<__nv_bfloat16>), grid, PACK_THREADS, 0, st, w, (__nv_bfloat16*)P, K, C, Qp);
        else NNV_LAUNCH((pack1x1_kernel<float>), grid, PACK_THREADS, 0, st, w, (float*)P, K, C, Qp);
    } else {
        NNV_REQUIRE(RS <= PACK_SMEM_FLOATS, NNV_ERR_UNSUPPORTED, "filter window of %d taps is too large to repack", RS);
        if (bf16) NNV_LAUNCH((pack_kernel<__nv_bfloat16>), K, PACK_THREADS, 0, st, w, (__nv_bfloat16*)P, C, RS, Qp);
        else NNV_LAUNCH((pack_kernel<float>), K, PACK_THREADS, 0, st, w, (float*)P, C, RS, Qp);
    }
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

}  // namespace nnv
