// Execution-side kernels that are not tensor-core contractions: im2col, the Winograd input and
// output transforms, fp32 direct and depthwise convolution, pooling and layout conversion.
// Activations are NHWC fp32 (batch 1).
#include <cuda_bf16.h>

#include "nnv_internal.h"

namespace nnv {

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == 1) return fmaxf(v, 0.f);
    if (act == 2) return fminf(fmaxf(v, 0.f), 6.f);
    return v;
}

// fp32 -> TF32 precision, round to nearest even (the tensor core would otherwise truncate).
__device__ __forceinline__ float round_tf32(float v) {
    uint32_t b = __float_as_uint(v);
    b += 0xFFFu + ((b >> 13) & 1u);
    return __uint_as_float(b & 0xFFFFE000u);
}
template <typename OutT> __device__ inline OutT to_out(float v);
template <> __device__ inline float to_out<float>(float v) { return v; }
template <> __device__ inline __nv_bfloat16 to_out<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// ---- im2col ---------------------------------------------------------------------------------
// Xcol[p][q], q = (r*S+s)*C + c; zero outside the image and for q >= R*S*C.
template <typename OutT>
__global__ void __launch_bounds__(256)
im2col_kernel(const float* __restrict__ x, OutT* __restrict__ col, int C, int H, int W, int R, int S, int stride,
              int pad, int OH, int OW, int Qp) {
    pdl_enter();
    const long long n = (long long)OH * OW * Qp;
    const int Q = R * S * C;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int p = (int)(i / Qp), q = (int)(i - (long long)p * Qp);
        float v = 0.f;
        if (q < Q) {
            const int rs = q / C, c = q - rs * C;
            const int r = rs / S, s = rs - r * S;
            const int oh = p / OW, ow = p - oh * OW;
            const int ih = oh * stride + r - pad, iw = ow * stride + s - pad;
            if (ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(x + ((long long)ih * W + iw) * C + c);
        }
        col[i] = to_out<OutT>(sizeof(OutT) == 4 ? round_tf32(v) : v);
    }
}

// The same matrix for small reductions (R*S*C up to IM2COL_TABLE entries: network stems with C = 3).  The
// (r, s, c) of every column q is worked out once per block into a shared-memory table; a warp then writes one
// pixel's row at a time, lane = q, so the inner loop has no division and the stores are contiguous.
constexpr int IM2COL_TABLE = 1024;
template <typename OutT>
__global__ void __launch_bounds__(256)
im2col_table_kernel(const float* __restrict__ x, OutT* __restrict__ col, int C, int H, int W, int R, int S, int stride,
                    int pad, int OH, int OW, int Qp) {
    pdl_enter();
    __shared__ int tab[IM2COL_TABLE];                           // (r << 20) | (s << 10) | c, or -1 for the zero padding q >= Q
    const int Q = R * S * C;
    for (int q = threadIdx.x; q < Qp; q += 256) {
        const int rs = q / C, c = q - rs * C;
        const int r = rs / S, sx = rs - r * S;
        tab[q] = q < Q ? ((r << 20) | (sx << 10) | c) : -1;
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int P = OH * OW;
    for (int p = blockIdx.x * 8 + warp; p < P; p += gridDim.x * 8) {
        const int oh = p / OW, ow = p - oh * OW;
        const int ih0 = oh * stride - pad, iw0 = ow * stride - pad;
        OutT* dst = col + (long long)p * Qp;
        for (int q = lane; q < Qp; q += 32) {
            const int e = tab[q];
            float v = 0.f;
            if (e >= 0) {
                const int ih = ih0 + (e >> 20), iw = iw0 + ((e >> 10) & 1023);
                if (ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(x + ((long long)ih * W + iw) * C + (e & 1023));
            }
            dst[q] = to_out<OutT>(sizeof(OutT) == 4 ? round_tf32(v) : v);
        }
    }
}

// Four consecutive q per thread; valid when C % 4 == 0 (a quad never straddles a filter tap).
template <typename OutT>
__global__ void __launch_bounds__(256)
im2col_vec4_kernel(const float* __restrict__ x, OutT* __restrict__ col, int C, int H, int W, int R, int S, int stride,
                   int pad, int OH, int OW, int Qp) {
    pdl_enter();
    const int Qv = Qp / 4;
    const long long n = (long long)OH * OW * Qv;
    const int Q = R * S * C;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int p = (int)(i / Qv), q = 4 * (int)(i - (long long)p * Qv);
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (q < Q) {
            const int rs = q / C, c = q - rs * C;
            const int r = rs / S, s = rs - r * S;
            const int oh = p / OW, ow = p - oh * OW;
            const int ih = oh * stride + r - pad, iw = ow * stride + s - pad;
            if (ih >= 0 && ih < H && iw >= 0 && iw < W)
                v = __ldg(reinterpret_cast<const float4*>(x + ((long long)ih * W + iw) * C + c));
        }
        OutT* dst = col + (long long)p * Qp + q;
        if constexpr (sizeof(OutT) == 4) {
            *reinterpret_cast<float4*>(dst) = make_float4(round_tf32(v.x), round_tf32(v.y), round_tf32(v.z), round_tf32(v.w));
        } else {
            __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
            uint2 u;
            u.x = *reinterpret_cast<uint32_t*>(&a);
            u.y = *reinterpret_cast<uint32_t*>(&b);
            *reinterpret_cast<uint2*>(dst) = u;
        }
    }
}

nnv_status_t launch_im2col(bool bf16, const float* x, void* col, int C, int H, int W, int R, int S, int stride,
                           int pad, int OH, int OW, int Qp, cudaStream_t st) {
    const bool vec = (C % 4) == 0;
    const long long n = (long long)OH * OW * (vec ? Qp / 4 : Qp);
    const unsigned grid = (unsigned)std::min<long long>((n + 255) / 256, 148ll * 32);
    if (vec) {
        if (bf16) NNV_LAUNCH((im2col_vec4_kernel<__nv_bfloat16>), grid, 256, 0, st, x, (__nv_bfloat16*)col, C, H, W, R, S, stride, pad, OH, OW, Qp);
        else NNV_LAUNCH((im2col_vec4_kernel<float>), grid, 256, 0, st, x, (float*)col, C, H, W, R, S, stride, pad, OH, OW, Qp);
    } else if (Qp <= IM2COL_TABLE && C < 1024 && R < 1024 && S < 1024) {
        const unsigned g2 = (unsigned)std::min<long long>(((long long)OH * OW + 7) / 8, 148ll * 16);
        if (bf16) NNV_LAUNCH((im2col_table_kernel<__nv_bfloat16>), g2, 256, 0, st, x, (__nv_bfloat16*)col, C, H, W, R, S, stride, pad, OH, OW, Qp);
        else NNV_LAUNCH((im2col_table_kernel<float>), g2, 256, 0, st, x, (float*)col, C, H, W, R, S, stride, pad, OH, OW, Qp);
    } else {
        if (bf16) NNV_LAUNCH((im2col_kernel<__nv_bfloat16>), grid, 256, 0, st, x, (__nv_bfloat16*)col, C, H, W, R, S, stride, pad, OH, OW, Qp);
        else NNV_LAUNCH((im2col_kernel<float>), grid, 256, 0, st, x, (float*)col, C, H, W, R, S, stride, pad, OH, OW, Qp);
    }
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// ---- Winograd data transforms ---------------------------------------------------------------
// B^T (alpha x alpha) and A^T (m x alpha) of the same Cook-Toom construction as the filter
// transform's G: finite points {0, 1, -1, 2, -2, 1/2, -1/2} in that order, then infinity.
template <int M_> struct WinoBA;
template <> struct WinoBA<2> {
    static constexpr int A = 4;
    __host__ __device__ static constexpr float bt(int r, int c) {
        constexpr float t[4][4] = {{1, 0, -1, 0}, {0, 1, 1, 0}, {0, -1, 1, 0}, {0, -1, 0, 1}};
        return t[r][c];
    }
    __host__ __device__ static constexpr float at(int r, int c) {
        constexpr float t[2][4] = {{1, 1, 1, 0}, {0, 1, -1, 1}};
        return t[r][c];
    }
};
template <> struct WinoBA<4> {
    static constexpr int A = 6;
    __host__ __device__ static constexpr float bt(int r, int c) {
        constexpr float t[6][6] = {{4, 0, -5, 0, 1, 0},  {0, -4, -4, 1, 1, 0}, {0, 4, -4, -1, 1, 0},
                                   {0, -2, -1, 2, 1, 0}, {0, 2, -1, -2, 1, 0}, {0, 4, 0, -5, 0, 1}};
        return t[r][c];
    }
    __host__ __device__ static constexpr float at(int r, int c) {
        constexpr float t[4][6] = {{1, 1, 1, 1, 1, 0}, {0, 1, -1, 2, -2, 0}, {0, 1, 1, 4, 4, 0}, {0, 1, -1, 8, -8, 1}};
        return t[r][c];
    }
};
template <> struct WinoBA<6> {
    static constexpr int A = 8;
    __host__ __device__ static constexpr float bt(int r, int c) {
        constexpr float t[8][8] = {{1, 0, -5.25f, 0, 5.25f, 0, -1, 0},
                                   {0, 1, 1, -4.25f, -4.25f, 1, 1, 0},
                                   {0, -1, 1, 4.25f, -4.25f, -1, 1, 0},
                                   {0, .5f, .25f, -2.5f, -1.25f, 2, 1, 0},
                                   {0, -.5f, .25f, 2.5f, -1.25f, -2, 1, 0},
                                   {0, 2, 4, -2.5f, -5, .5f, 1, 0},
                                   {0, -2, 4, 2.5f, -5, -.5f, 1, 0},
                                   {0, -1, 0, 5.25f, 0, -5.25f, 0, 1}};
        return t[r][c];
    }
    __host__ __device__ static constexpr float at(int r, int c) {
        constexpr float t[6][8] = {{1, 1, 1, 1, 1, 1, 1, 0},
                                   {0, 1, -1, 2, -2, .5f, -.5f, 0},
                                   {0, 1, 1, 4, 4, .25f, .25f, 0},
                                   {0, 1, -1, 8, -8, .125f, -.125f, 0},
                                   {0, 1, 1, 16, 16, .0625f, .0625f, 0},
                                   {0, 1, -1, 32, -32, .03125f, -.03125f, 1}};
        return t[r][c];
    }
};

// One thread per (tile, padded channel); channel is the fastest index so that every load and
// store of a warp covers 32 consecutive channels.  V[(xi*A+nu)][t][cp].
template <int M_, typename OutT>
__global__ void __launch_bounds__(128)
wino_input_kernel(const float* __restrict__ x, OutT* __restrict__ V, int C, int Cp, int H, int W, int pad, int TH,
                  int TW) {
    pdl_enter();
    constexpr int A = WinoBA<M_>::A;
    const long long T = (long long)TH * TW;
    const long long idx = (long long)blockIdx.x * 128 + threadIdx.x;
    if (idx >= T * Cp) return;
    const int t = (int)(idx / Cp), c = (int)(idx - (long long)t * Cp);
    const int th = t / TW, tw = t - th * TW;
    const int h0 = th * M_ - pad, w0 = tw * M_ - pad;
    float d[A][A];
#pragma unroll
    for (int i = 0; i < A; ++i) {
        const int h = h0 + i;
#pragma unroll
        for (int j = 0; j < A; ++j) {
            const int w = w0 + j;
            d[i][j] = (c < C && h >= 0 && h < H && w >= 0 && w < W) ? __ldg(x + ((long long)h * W + w) * C + c) : 0.f;
        }
    }
    float tmp[A][A];                                             // tmp = B^T d
#pragma unroll
    for (int i = 0; i < A; ++i)
#pragma unroll
        for (int j = 0; j < A; ++j) {
            float s = 0.f;
#pragma unroll
            for (int l = 0; l < A; ++l)
                if (WinoBA<M_>::bt(i, l) != 0.f) s += WinoBA<M_>::bt(i, l) * d[l][j];
            tmp[i][j] = s;
        }
    OutT* out = V + (long long)t * Cp + c;
#pragma unroll
    for (int i = 0; i < A; ++i)
#pragma unroll
        for (int j = 0; j < A; ++j) {                            // V = tmp B
            float s = 0.f;
#pragma unroll
            for (int l = 0; l < A; ++l)
                if (WinoBA<M_>::bt(j, l) != 0.f) s += tmp[i][l] * WinoBA<M_>::bt(j, l);
            out[(long long)(i * A + j) * T * Cp] = to_out<OutT>((sizeof(OutT) == 4 && M_ == 2) ? round_tf32(s) : s);
        }
}

nnv_status_t launch_wino_input(int m, bool bf16, const float* x, void* V, int C, int Cp, int H, int W, int pad,
                               int TH, int TW, cudaStream_t st) {
    const long long n = (long long)TH * TW * Cp;
    const unsigned grid = (unsigned)((n + 127) / 128);
#define NNV_WI(MM)                                                                                              \
    if (bf16) NNV_LAUNCH((wino_input_kernel<MM, __nv_bfloat16>), grid, 128, 0, st, x, (__nv_bfloat16*)V, C, Cp, H, W, pad, TH, TW); \
    else NNV_LAUNCH((wino_input_kernel<MM, float>), grid, 128, 0, st, x, (float*)V, C, Cp, H, W, pad, TH, TW);
    if (m == 2) { NNV_WI(2) } else if (m == 4) { NNV_WI(4) } else if (m == 6) { NNV_WI(6) }
    else return fail(NNV_ERR_INVALID_ARG, "no Winograd tile size %d", m);
#undef NNV_WI
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// One thread per (tile, output channel), channel fastest.  Y tile = A^T M A, then bias, residual
// addend and activation; pixels beyond the output grid are clipped.
template <int M_>
__global__ void __launch_bounds__(128)
wino_output_kernel(const float* __restrict__ Mt, float* __restrict__ y, const float* __restrict__ bias,
                   const float* __restrict__ add, int act, int K, int OH, int OW, int TH, int TW) {
    pdl_enter();
    constexpr int A = WinoBA<M_>::A;
    const long long T = (long long)TH * TW;
    const long long idx = (long long)blockIdx.x * 128 + threadIdx.x;
    if (idx >= T * K) return;
    const int t = (int)(idx / K), k = (int)(idx - (long long)t * K);
    const int th = t / TW, tw = t - th * TW;
    const float* src = Mt + (long long)t * K + k;
    float tmp[M_][A];                                            // tmp = A^T M, built one M row at a time
#pragma unroll
    for (int i = 0; i < M_; ++i)
#pragma unroll
        for (int j = 0; j < A; ++j) tmp[i][j] = 0.f;
#pragma unroll
    for (int l = 0; l < A; ++l) {
        float row[A];
#pragma unroll
        for (int j = 0; j < A; ++j) row[j] = __ldg(src + (long long)(l * A + j) * T * K);
#pragma unroll
        for (int i = 0; i < M_; ++i)
            if (WinoBA<M_>::at(i, l) != 0.f) {
#pragma unroll
                for (int j = 0; j < A; ++j) tmp[i][j] += WinoBA<M_>::at(i, l) * row[j];
            }
    }
    const float b = bias ? __ldg(bias + k) : 0.f;
#pragma unroll
    for (int i = 0; i < M_; ++i) {
        const int oh = th * M_ + i;
#pragma unroll
        for (int j = 0; j < M_; ++j) {
            const int ow = tw * M_ + j;
            float s = 0.f;
#pragma unroll
            for (int l = 0; l < A; ++l)
                if (WinoBA<M_>::at(j, l) != 0.f) s += tmp[i][l] * WinoBA<M_>::at(j, l);
            if (oh < OH && ow < OW) {
                const long long o = ((long long)oh * OW + ow) * K + k;
                s += b;
                if (add) s += __ldg(add + o);
                y[o] = apply_act(s, act);
            }
        }
    }
}

nnv_status_t launch_wino_output(int m, const float* Mt, float* y, const float* bias, const float* add, int act,
                                int K, int OH, int OW, int TH, int TW, cudaStream_t st) {
    const long long n = (long long)TH * TW * K;
    const unsigned grid = (unsigned)((n + 127) / 128);
    if (m == 2) NNV_LAUNCH((wino_output_kernel<2>), grid, 128, 0, st, Mt, y, bias, add, act, K, OH, OW, TH, TW);
    else if (m == 4) NNV_LAUNCH((wino_output_kernel<4>), grid, 128, 0, st, Mt, y, bias, add, act, K, OH, OW, TH, TW);
    else if (m == 6) NNV_LAUNCH((wino_output_kernel<6>), grid, 128, 0, st, Mt, y, bias, add, act, K, OH, OW, TH, TW);
    else return fail(NNV_ERR_INVALID_ARG, "no Winograd tile size %d", m);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// ---- fp32 direct convolution ----------------------------------------------------------------
// Implicit GEMM on the FP32 pipes straight from the raw OIHW weights: the reduction index is
// q = c*R*S + r*S + s, which is exactly the raw row W[k][:], so no weight transform is needed.
// Tile: 64 pixels x 64 output channels per block, 16 reduction steps per stage, 4x4 per thread.
constexpr int DC_BM = 64, DC_BN = 64, DC_BK = 16;
__global__ void __launch_bounds__(256)
direct_conv_kernel(const float* __restrict__ x, const float* __restrict__ w, const float* __restrict__ bias,
                   const float* __restrict__ add, float* __restrict__ y, int act, int C, int H, int W, int K, int R,
                   int S, int stride, int pad, int OH, int OW) {
    pdl_enter();
    __shared__ float As[DC_BK][DC_BM + 4];
    __shared__ float Bs[DC_BK][DC_BN + 4];
    const int P = OH * OW, RS = R * S, Q = C * RS;
    const int p0 = blockIdx.x * DC_BM, k0 = blockIdx.y * DC_BN;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;      // tx -> channels, ty -> pixels
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int q0 = 0; q0 < Q; q0 += DC_BK) {
#pragma unroll
        for (int it = 0; it < 4; ++it) {                          // A: 64 x 16 gathered input
            const int e = threadIdx.x + it * 256;
            const int pm = e % DC_BM, kk = e / DC_BM;
            const int p = p0 + pm, q = q0 + kk;
            float v = 0.f;
            if (p < P && q < Q) {
                const int c = q / RS, rs = q - c * RS;
                const int r = rs / S, s = rs - r * S;
                const int oh = p / OW, ow = p - oh * OW;
                const int ih = oh * stride + r - pad, iw = ow * stride + s - pad;
                if (ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(x + ((long long)ih * W + iw) * C + c);
            }
            As[kk][pm] = v;
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {                          // B: 64 x 16 raw weights
            const int e = threadIdx.x + it * 256;
            const int kk = e % DC_BK, n = e / DC_BK;
            const int k = k0 + n, q = q0 + kk;
            Bs[kk][n] = (k < K && q < Q) ? __ldg(w + (long long)k * Q + q) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < DC_BK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int p = p0 + ty * 4 + i;
        if (p >= P) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = k0 + tx * 4 + j;
            if (k >= K) continue;
            const long long o = (long long)p * K + k;
            float v = acc[i][j];
            if (bias) v += __ldg(bias + k);
            if (add) v += __ldg(add + o);
            y[o] = apply_act(v, act);
        }
    }
}

nnv_status_t launch_direct(const float* x, const float* w, const float* bias, const float* add, float* y, int act,
                           int C, int H, int W, int K, int R, int S, int stride, int pad, int OH, int OW,
                           cudaStream_t st) {
    dim3 grid(ceil_div(OH * OW, DC_BM), ceil_div(K, DC_BN));
    NNV_LAUNCH((direct_conv_kernel), grid, 256, 0, st, x, w, bias, add, y, act, C, H, W, K, R, S, stride, pad, OH, OW);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// ---- fp32 depthwise convolution -------------------------------------------------------------
// One thread per (output pixel, channel), channel fastest; raw weights W[c][r][s] are read as is.
__global__ void __launch_bounds__(256)
depthwise_kernel(const float* __restrict__ x, const float* __restrict__ w, const float* __restrict__ bias,
                 const float* __restrict__ add, float* __restrict__ y, int act, int C, int H, int W, int R, int S,
                 int stride, int pad, int OH, int OW) {
    pdl_enter();
    const long long n = (long long)OH * OW * C;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int p = (int)(i / C), c = (int)(i - (long long)p * C);
        const int oh = p / OW, ow = p - oh * OW;
        float acc = bias ? __ldg(bias + c) : 0.f;
        for (int r = 0; r < R; ++r) {
            const int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < S; ++s) {
                const int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                acc = fmaf(__ldg(x + ((long long)ih * W + iw) * C + c), __ldg(w + ((long long)c * R + r) * S + s), acc);
            }
        }
        if (add) acc += __ldg(add + i);
        y[i] = apply_act(acc, act);
    }
}

// 3x3 depthwise, stride 1 or 2, C % 4 == 0: one thread = four channels x four neighbouring output pixels of a row.
// Every access is 16 bytes and a warp's accesses are 512 contiguous bytes (channel groups are the fastest index); the
// (3 STRIDE + 3) x 3 input window is loaded once for the four outputs (18 loads instead of 36 at stride 1), and the
// thread's 36 weights are nine 16-byte loads of the raw W[c][r][s] rows, rearranged in registers.
template <int STRIDE>
__global__ void __launch_bounds__(256)
depthwise3x3_v4_kernel(const float* __restrict__ x, const float* __restrict__ w, const float* __restrict__ bias,
                       const float* __restrict__ add, float* __restrict__ y, int act, int C, int H, int W, int pad, int OH, int OW) {
    pdl_enter();
    constexpr int NCOL = 3 * STRIDE + 3;
    const int C4 = C >> 2, OW4 = (OW + 3) >> 2;
    const long long n = (long long)OH * OW4 * C4;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int c4 = (int)(i % C4);
        const long long pq = i / C4;
        const int oq = (int)(pq % OW4), oh = (int)(pq / OW4);
        const int c = c4 * 4, ow0 = oq * 4;
        float wv[36];                                         // [channel 0..3][tap 0..8]
#pragma unroll
        for (int j = 0; j < 9; ++j) {
            const float4 t = __ldg(reinterpret_cast<const float4*>(w + (long long)c * 9) + j);
            wv[4 * j] = t.x; wv[4 * j + 1] = t.y; wv[4 * j + 2] = t.z; wv[4 * j + 3] = t.w;
        }
        float4 acc[4];
        const float4 b4 = bias ? __ldg(reinterpret_cast<const float4*>(bias + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[p] = b4;
        const int iw0 = ow0 * STRIDE - pad;
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const int ih = oh * STRIDE + r - pad;
            if (ih < 0 || ih >= H) continue;
            const float* row = x + ((long long)ih * W) * C + c;
#pragma unroll
            for (int col = 0; col < NCOL; ++col) {
                const int iw = iw0 + col;
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                if (iw >= 0 && iw < W) v = __ldg(reinterpret_cast<const float4*>(row + (long long)iw * C));
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const int sft = col - p * STRIDE;         // the tap column this input column is for output p
                    if (sft >= 0 && sft < 3) {
                        const int t = r * 3 + sft;
                        acc[p].x = fmaf(v.x, wv[t], acc[p].x);
                        acc[p].y = fmaf(v.y, wv[9 + t], acc[p].y);
                        acc[p].z = fmaf(v.z, wv[18 + t], acc[p].z);
                        acc[p].w = fmaf(v.w, wv[27 + t], acc[p].w);
                    }
                }
            }
        }
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const int ow = ow0 + p;
            if (ow >= OW) break;
            const long long o = ((long long)oh * OW + ow) * C + c;
            float4 v = acc[p];
            if (add) {
                const float4 a4 = __ldg(reinterpret_cast<const float4*>(add + o));
                v.x += a4.x; v.y += a4.y; v.z += a4.z; v.w += a4.w;
            }
            v.x = apply_act(v.x, act); v.y = apply_act(v.y, act); v.z = apply_act(v.z, act); v.w = apply_act(v.w, act);
            *reinterpret_cast<float4*>(y + o) = v;
        }
    }
}

nnv_status_t launch_depthwise(const float* x, const float* w, const float* bias, const float* add, float* y,
                              int act, int C, int H, int W, int R, int S, int stride, int pad, int OH, int OW,
                              cudaStream_t st) {
    const bool al16 = ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(y) |
                        reinterpret_cast<uintptr_t>(bias) | reinterpret_cast<uintptr_t>(add)) & 15) == 0;
    if (R == 3 && S == 3 && (stride == 1 || stride == 2) && (C % 4) == 0 && al16) {
        const long long n4 = (long long)OH * ((OW + 3) / 4) * (C / 4);
        const unsigned grid4 = (unsigned)std::min<long long>((n4 + 255) / 256, 148ll * 32);
        if (stride == 1) NNV_LAUNCH((depthwise3x3_v4_kernel<1>), grid4, 256, 0, st, x, w, bias, add, y, act, C, H, W, pad, OH, OW);
        else NNV_LAUNCH((depthwise3x3_v4_kernel<2>), grid4, 256, 0, st, x, w, bias, add, y, act, C, H, W, pad, OH, OW);
        NNV_CUDA(cudaGetLastError());
        return NNV_OK;
    }
    const long long n = (long long)OH * OW * C;
    const unsigned grid = (unsigned)std::min<long long>((n + 255) / 256, 148ll * 32);
    NNV_LAUNCH((depthwise_kernel), grid, 256, 0, st, x, w, bias, add, y, act, C, H, W, R, S, stride, pad, OH, OW);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

// ---- pooling and layout ---------------------------------------------------------------------
__global__ void __launch_bounds__(256)
maxpool_kernel(const float* __restrict__ x, float* __restrict__ y, int C, int H, int W, int R, int stride, int pad,
               int OH, int OW) {
    pdl_enter();
    const long long n = (long long)OH * OW * C;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int p = (int)(i / C), c = (int)(i - (long long)p * C);
        const int oh = p / OW, ow = p - oh * OW;
        float m = -INFINITY;
        for (int r = 0; r < R; ++r) {
            const int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < R; ++s) {
                const int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                m = fmaxf(m, __ldg(x + ((long long)ih * W + iw) * C + c));
            }
        }
        y[i] = m;
    }
}

__global__ void __launch_bounds__(256)
gavgpool_kernel(const float* __restrict__ x, float* __restrict__ y, int C, int HW) {
    pdl_enter();
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c >= C) return;
    float s = 0.f;
    for (int p = 0; p < HW; ++p) s += __ldg(x + (long long)p * C + c);
    y[c] = s / (float)HW;
}

__global__ void __launch_bounds__(256)
chw_to_hwc_kernel(const float* __restrict__ in, float* __restrict__ out, int C, int HW) {
    pdl_enter();
    const long long n = (long long)C * HW;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int p = (int)(i / C), c = (int)(i - (long long)p * C);
        out[i] = __ldg(in + (long long)c * HW + p);
    }
}

__global__ void __launch_bounds__(256)
hwc_to_chw_kernel(const float* __restrict__ in, float* __restrict__ out, int C, int HW) {
    pdl_enter();
    const long long n = (long long)C * HW;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n; i += (long long)gridDim.x * 256) {
        const int c = (int)(i / HW), p = (int)(i - (long long)c * HW);
        out[i] = __ldg(in + (long long)p * C + c);
    }
}

static inline unsigned grid_for(long long n) { return (unsigned)std::min<long long>((n + 255) / 256, 148ll * 32); }

nnv_status_t launch_maxpool(const float* x, float* y, int C, int H, int W, int R, int stride, int pad, int OH,
                            int OW, cudaStream_t st) {
    NNV_LAUNCH((maxpool_kernel), grid_for((long long)OH * OW * C), 256, 0, st, x, y, C, H, W, R, stride, pad, OH, OW);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}
nnv_status_t launch_gavgpool(const float* x, float* y, int C, int H, int W, cudaStream_t st) {
    NNV_LAUNCH((gavgpool_kernel), ceil_div(C, 256), 256, 0, st, x, y, C, H * W);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}
nnv_status_t launch_chw_to_hwc(const float* in, float* out, int C, int H, int W, cudaStream_t st) {
    NNV_LAUNCH((chw_to_hwc_kernel), grid_for((long long)C * H * W), 256, 0, st, in, out, C, H * W);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}
nnv_status_t launch_hwc_to_chw(const float* in, float* out, int C, int H, int W, cudaStream_t st) {
    NNV_LAUNCH((hwc_to_chw_kernel), grid_for((long long)C * H * W), 256, 0, st, in, out, C, H * W);
    NNV_CUDA(cudaGetLastError());
    return NNV_OK;
}

}  // namespace nnv
