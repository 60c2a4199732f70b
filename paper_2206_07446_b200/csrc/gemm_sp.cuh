// Tensor-core convolution for layers with few output pixels (H * W <= 256, stride 1, "same" padding):
// the weights, not the pixels, sit on the MMA's 128-row dimension.  Included by gemm_tc.cu.
//
// On 14 x 14 and 7 x 7 grids a layer is bound by streaming its packed weights (1 - 9 MB) once; with
// pixels on the 128 MMA rows there are one or two row tiles, most of each operand tile is zero padding,
// and a cluster of 8 CTAs is all the K split can use.  Here D^T[k][p] = W[k][q] * Xcol[p][q]^T:
//   A operand  128 output channels x 32 reduction elements of the packed weights (all of it useful),
//   B operand  all P = H * W pixels x 32 channels of ONE filter tap, fetched by a single tiled TMA box
//              {32 channels, W, H} that starts at pixel (s - pad, r - pad): positions outside the image are
//              zero-filled, and the box lands in shared memory in pixel order, i.e. already as the im2col tile,
//   D^T        128 channels (TMEM lanes) x Npad = ceil(P / 16) * 16 pixels (TMEM columns).
// The reduction (taps x channel blocks) is split over grid.y CTAs so that every SM streams a share of the
// weights.  With more than one split each CTA writes its partial tile to scratch as part[split][p][k] and
// splitk_reduce_kernel adds the splits in index order (the result does not depend on timing) and applies
// bias / residual / activation; with one split the epilogue does that itself.  Either way a warp stores 32
// consecutive channels of one pixel per instruction: whole 128-byte lines.
#pragma once

struct SpDev {
    unsigned long long* stamp;
    float* D;                       // NHWC output [P][K]
    float* part;                    // scratch [splits][P][K] (splits > 1)
    const float* bias;
    const float* addend;
    int P, K, C, S, pad, Npad, act, tmem_cols, splits, stages, cblk, nkb_all;
    uint32_t b_slot_bytes, b_tx_bytes;
};

constexpr int SP_MAX_STAGES = 8;

__global__ void __launch_bounds__(GEMM_THREADS)
gemm_sp_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX, const SpDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const int STAGES = g.stages;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t stage_bytes = A_STAGE_BYTES + g.b_slot_bytes;
    const uint32_t bars = sbase + STAGES * stage_bytes;
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (SP_MAX_STAGES + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * SP_MAX_STAGES);
    const uint32_t holder = tmem_full_bar + 8u;
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * BM, sp = blockIdx.y, splits = g.splits;
    const int kb0 = (g.nkb_all * sp) / splits;
    const int nkb = (g.nkb_all * (sp + 1)) / splits - kb0;

    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmW)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmX)) : "memory");
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // K block `kb` = channel block cb of filter tap (fr, fs); the position is carried along (no division in the loop)
    int tap = kb0 / g.cblk, cb = kb0 - tap * g.cblk;
    int fr = tap / g.S, fs = tap - fr * g.S;
    auto issue_stage = [&](int s) {
        const uint32_t a_dst = sbase + s * stage_bytes;
        mbar_expect_tx(full_bar(s), A_STAGE_BYTES + g.b_tx_bytes);
        tma_load_3d(a_dst, &tmW, tap * g.C + cb * 32, m0, 0, full_bar(s));
        tma_load_3d(a_dst + A_STAGE_BYTES, &tmX, cb * 32, fs - g.pad, fr - g.pad, full_bar(s));
        if (++cb == g.cblk) {
            cb = 0; ++tap;
            if (++fs == g.S) { fs = 0; ++fr; }
        }
    };
    // The weights do not depend on the previous kernel, but the activation does: wait, then fill the ring.
    const int prefill = nkb < STAGES ? nkb : STAGES;
    if (warp == 0 && lane == 0) {
        pdl_wait();
        for (int it = 0; it < prefill; ++it) issue_stage(it);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *holder_ptr;
    pdl_wait();
    if (threadIdx.x == 32) stamp_start(g.stamp);

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int s = prefill == STAGES ? 0 : prefill;
            uint32_t ph = prefill == STAGES ? 1u : 0u;
            for (int it = prefill; it < nkb && ok; ++it) {
                ok = mbar_wait(empty_bar(s), ph ^ 1u);
                if (!ok) break;
                issue_stage(s);
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulate, TF32 operands, both K-major, N = Npad, M = 128
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(g.Npad >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < nkb; ++it) {
                ok = mbar_wait(full_bar(s), ph);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = sbase + s * stage_bytes;
                const uint64_t adesc = make_smem_desc(a_src);
                const uint64_t bdesc = make_smem_desc(a_src + A_STAGE_BYTES);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)                 // 4 MMAs of 32 bytes of K each
                    umma<false>(tmem_base, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (it | kk) ? 1u : 0u);
                umma_commit(empty_bar(s));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(tmem_full_bar);
            else atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        const bool ok = mbar_wait(tmem_full_bar, 0);
        tc_fence_after();
        if (!ok) {
            if (lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        } else {
            const int quarter = warp & 3;                     // TMEM lanes this warp may read
            const int k = m0 + quarter * 32 + lane;           // this lane's output channel
            const bool k_ok = k < g.K;
            const bool final_out = splits == 1;
            const float bias = (final_out && g.bias && k_ok) ? __ldg(g.bias + k) : 0.f;
            float* dst = final_out ? g.D : g.part + (long long)sp * g.P * g.K;
            for (int c0 = 0; c0 < g.Npad; c0 += 16) {
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0, r);
                float add[16];
                if (final_out && g.addend) {                  // all loads of the chunk first
#pragma unroll
                    for (int j = 0; j < 16; ++j) add[j] = (k_ok && c0 + j < g.P) ? __ldg(g.addend + (long long)(c0 + j) * g.K + k) : 0.f;
                }
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int p = c0 + j;
                    if (!k_ok || p >= g.P) continue;
                    float v = __uint_as_float(r[j]);
                    if (final_out) {
                        v += bias;
                        if (g.addend) v += add[j];
                        v = act_fn(v, g.act);
                    }
                    dst[(long long)p * g.K + k] = v;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && g.splits == 1) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

// out[p][k] = act(sum over the splits of part[s][p][k] + bias[k] + addend[p][k]); K % 4 == 0.  A block of eight
// warps owns 32 consecutive 16-byte words of the output: warp w adds the splits w, w + 8, w + 16, ... in
// ascending order (four loads in flight at a time), then warp 0 adds the eight sums in warp order.  The order
// of every addition is fixed by the indices alone, so the result is the same bits on every run.
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const float* __restrict__ part, float* __restrict__ D, const float* __restrict__ bias,
                     const float* __restrict__ addend, int P, int K, int splits, int act, unsigned long long* stamp) {
    pdl_enter();
    __shared__ float4 sm[8][32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long n4 = (long long)P * K / 4;
    const long long slab4 = n4;                                 // 16-byte words per split
    const long long i = (long long)blockIdx.x * 32 + lane;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < n4) {
        const float4* src = reinterpret_cast<const float4*>(part) + i;
        int s = warp;
        for (; s + 24 < splits; s += 32) {                       // four splits of this warp at a time
            const float4 v0 = __ldcg(src + (long long)s * slab4), v1 = __ldcg(src + (long long)(s + 8) * slab4);
            const float4 v2 = __ldcg(src + (long long)(s + 16) * slab4), v3 = __ldcg(src + (long long)(s + 24) * slab4);
            acc.x += v0.x; acc.y += v0.y; acc.z += v0.z; acc.w += v0.w;
            acc.x += v1.x; acc.y += v1.y; acc.z += v1.z; acc.w += v1.w;
            acc.x += v2.x; acc.y += v2.y; acc.z += v2.z; acc.w += v2.w;
            acc.x += v3.x; acc.y += v3.y; acc.z += v3.z; acc.w += v3.w;
        }
        for (; s < splits; s += 8) {
            const float4 v = __ldcg(src + (long long)s * slab4);
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
    }
    sm[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && i < n4) {
        float4 r = sm[0][lane];
#pragma unroll
        for (int w = 1; w < 8; ++w) {
            if (w < splits) { const float4 v = sm[w][lane]; r.x += v.x; r.y += v.y; r.z += v.z; r.w += v.w; }
        }
        const int k = (int)((i * 4) % K);
        if (bias) {
            const float4 b = __ldg(reinterpret_cast<const float4*>(bias + k));
            r.x += b.x; r.y += b.y; r.z += b.z; r.w += b.w;
        }
        if (addend) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(addend) + i);
            r.x += a.x; r.y += a.y; r.z += a.z; r.w += a.w;
        }
        r.x = act_fn(r.x, act); r.y = act_fn(r.y, act); r.z = act_fn(r.z, act); r.w = act_fn(r.w, act);
        reinterpret_cast<float4*>(D)[i] = r;
    }
    if (threadIdx.x == 0) stamp_end(stamp);
}
