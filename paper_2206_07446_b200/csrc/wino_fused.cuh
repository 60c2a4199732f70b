// Winograd F(2x2,3x3) in ONE kernel: input transform -> 16 tile GEMMs on the tensor cores -> output
// transform, with the 16 accumulators in TMEM.  Included by gemm_tc.cu.
//
// The three-kernel path writes V (16 planes of tiles x channels) and M (16 planes of tiles x output channels)
// to global memory and reads them back; here neither exists.  A CTA owns 128 Winograd tiles (the MMA's rows)
// and BN output channels:
//   warps 2-5  (a thread per tile) load the tile's 4 x 4 input patch for 8 channels at a time, form
//              V = B^T d B in registers, round it to TF32 and store it as the A operands of the 16 planes
//              (un-swizzled core-matrix layout: 8 rows x 16 bytes), stage by stage of a shared-memory ring;
//   warp 0     fetches the matching 8 channels of U for all 16 planes with two TMA boxes per stage;
//   warp 1     issues 16 MMAs per stage, plane p into accumulator p (TMEM columns p * BN ...);
//   warps 2-5  then read the 16 accumulators 8 channels at a time, form Y = A^T M A per tile and channel,
//              add bias / residual, apply the activation and write the 2 x 2 output pixels.
// Same arithmetic as wino_input_kernel + the TF32 tile GEMM + wino_output_kernel: V rounded to TF32
// (nearest even), U as the filter transform left it, channels accumulated in ascending groups of 8.
#pragma once

struct WfDev {
    unsigned long long* stamp;
    const float* x;                 // NHWC input
    float* y;                       // NHWC output
    const float* bias;
    const float* addend;
    int C, H, W, K, pad, OH, OW, TW, T, act, BN, stages, tmem_cols, nsteps;
};

constexpr int WF_MAX_STAGES = 3;
constexpr uint32_t WF_A_STAGE = 16u * 2u * 2048u;               // 16 planes x 2 k-chunks x (128 rows x 16 bytes)

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&r)[8]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ float wf_round_tf32(float v) {
    uint32_t b = __float_as_uint(v);
    b += 0xFFFu + ((b >> 13) & 1u);
    return __uint_as_float(b & 0xFFFFE000u);
}

__global__ void __launch_bounds__(GEMM_THREADS)
wino_f2_fused_kernel(const __grid_constant__ CUtensorMap tmU, const WfDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const int STAGES = g.stages, BN = g.BN;
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t b_chunk = 16u * (uint32_t)BN * 16u;             // one k-chunk of U: 16 planes x BN rows x 16 bytes
    const uint32_t b_stage = 2u * b_chunk;
    const uint32_t a_ring = sbase, b_ring = sbase + STAGES * WF_A_STAGE;
    const uint32_t bars = b_ring + STAGES * b_stage;
    auto full_b = [&](int s) { return bars + 8u * s; };
    auto conv_bar = [&](int s) { return bars + 8u * (WF_MAX_STAGES + s); };
    auto empty_bar = [&](int s) { return bars + 8u * (2 * WF_MAX_STAGES + s); };
    const uint32_t tmem_full_bar = bars + 8u * (3 * WF_MAX_STAGES);
    const uint32_t holder = tmem_full_bar + 8u;
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = blockIdx.x * BM, n0 = blockIdx.y * BN;

    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmU)) : "memory");
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_b(s), 1); mbar_init(conv_bar(s), 128); mbar_init(empty_bar(s), 1); }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
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
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < g.nsteps && ok; ++it) {
                ok = mbar_wait(empty_bar(s), ph ^ 1u);
                if (!ok) break;
                mbar_expect_tx(full_b(s), b_stage);
                const uint32_t dst = b_ring + s * b_stage;
                tma_load_3d(dst, &tmU, it * 8, n0, 0, full_b(s));
                tma_load_3d(dst + b_chunk, &tmU, it * 8 + 4, n0, 0, full_b(s));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            bool ok = true;
            int s = 0;
            uint32_t ph = 0;
            for (int it = 0; it < g.nsteps; ++it) {
                ok = mbar_wait(conv_bar(s), ph) && mbar_wait(full_b(s), ph);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_s = a_ring + s * WF_A_STAGE, b_s = b_ring + s * b_stage;
#pragma unroll 4
                for (int p = 0; p < 16; ++p) {
                    const uint64_t adesc = make_smem_desc_plain(a_s + (uint32_t)p * 4096u, 2048u, 128u);
                    const uint64_t bdesc = make_smem_desc_plain(b_s + (uint32_t)p * (uint32_t)BN * 16u, b_chunk, 128u);
                    umma<false>(tmem_base + (uint32_t)(p * BN), adesc, bdesc, idesc, it ? 1u : 0u);
                }
                umma_commit(empty_bar(s));
                if (++s == STAGES) { s = 0; ph ^= 1u; }
            }
            if (ok) umma_commit(tmem_full_bar);
            else atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        // ---- input transform: this thread's tile, 8 channels per stage ----
        const int row = (warp & 3) * 32 + lane;                  // MMA row = TMEM lane (a warp may read lanes 32 * (warp % 4) ...)
        const int t = t0 + row;
        const bool live = t < g.T;
        const int th = live ? t / g.TW : 0, tw = live ? t - th * g.TW : 0;
        const int h0 = th * 2 - g.pad, w0 = tw * 2 - g.pad;
        bool ok = true;
        int s = 0;
        uint32_t ph = 0;
        for (int it = 0; it < g.nsteps && ok; ++it) {
            ok = mbar_wait(empty_bar(s), ph ^ 1u);
            if (!ok) break;
            const uint32_t a_s = a_ring + s * WF_A_STAGE + (uint32_t)row * 16u;
#pragma unroll
            for (int j = 0; j < 2; ++j) {                        // two groups of 4 channels = the two k-chunks
                const int c = it * 8 + j * 4;
                float4 d[4][4];
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const int h = h0 + a, w = w0 + b;
                        d[a][b] = (live && h >= 0 && h < g.H && w >= 0 && w < g.W)
                                      ? __ldg(reinterpret_cast<const float4*>(g.x + ((long long)h * g.W + w) * g.C + c))
                                      : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                // tmp = B^T d (rows), B^T = [1 0 -1 0; 0 1 1 0; 0 -1 1 0; 0 -1 0 1]
                float4 m[4][4];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
#define WF_SUB(p, q) make_float4((p).x - (q).x, (p).y - (q).y, (p).z - (q).z, (p).w - (q).w)
#define WF_ADD(p, q) make_float4((p).x + (q).x, (p).y + (q).y, (p).z + (q).z, (p).w + (q).w)
                    m[0][b] = WF_SUB(d[0][b], d[2][b]);
                    m[1][b] = WF_ADD(d[1][b], d[2][b]);
                    m[2][b] = WF_SUB(d[2][b], d[1][b]);
                    m[3][b] = WF_SUB(d[3][b], d[1][b]);
                }
#pragma unroll
                for (int a = 0; a < 4; ++a) {                    // V = tmp B: the same combinations along the columns
                    float4 v[4];
                    v[0] = WF_SUB(m[a][0], m[a][2]);
                    v[1] = WF_ADD(m[a][1], m[a][2]);
                    v[2] = WF_SUB(m[a][2], m[a][1]);
                    v[3] = WF_SUB(m[a][3], m[a][1]);
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const uint32_t addr = a_s + (uint32_t)((a * 4 + b) * 2 + j) * 2048u;
                        asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "f"(wf_round_tf32(v[b].x)), "f"(wf_round_tf32(v[b].y)),
                                     "f"(wf_round_tf32(v[b].z)), "f"(wf_round_tf32(v[b].w)) : "memory");
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
            mbar_arrive(conv_bar(s));
            if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        // ---- output transform: Y = A^T M A, A^T = [1 1 1 0; 0 1 -1 1] ----
        ok = ok && mbar_wait(tmem_full_bar, 0);
        tc_fence_after();
        if (!ok) {
            if (lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        } else {
            const int quarter = warp & 3;                         // == row / 32: the TMEM lanes this warp may read
            for (int c0 = 0; c0 < BN; c0 += 8) {
                uint32_t r[16][8];
#pragma unroll
                for (int p = 0; p < 16; ++p) tmem_ld8(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(p * BN + c0), r[p]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                const int n = n0 + c0;
                if (!live || n >= g.K) continue;
                float yv[2][2][8];
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    float tm[2][4];
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const float m0 = __uint_as_float(r[0 * 4 + b][ch]), m1 = __uint_as_float(r[1 * 4 + b][ch]);
                        const float m2 = __uint_as_float(r[2 * 4 + b][ch]), m3 = __uint_as_float(r[3 * 4 + b][ch]);
                        tm[0][b] = m0 + m1 + m2;
                        tm[1][b] = m1 - m2 + m3;
                    }
#pragma unroll
                    for (int a = 0; a < 2; ++a) {
                        yv[a][0][ch] = tm[a][0] + tm[a][1] + tm[a][2];
                        yv[a][1][ch] = tm[a][1] - tm[a][2] + tm[a][3];
                    }
                }
#pragma unroll
                for (int a = 0; a < 2; ++a)
#pragma unroll
                    for (int b = 0; b < 2; ++b) {
                        const int oh = th * 2 + a, ow = tw * 2 + b;
                        if (oh >= g.OH || ow >= g.OW) continue;
                        const long long off = ((long long)oh * g.OW + ow) * g.K + n;
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            float4 v = make_float4(yv[a][b][q * 4], yv[a][b][q * 4 + 1], yv[a][b][q * 4 + 2], yv[a][b][q * 4 + 3]);
                            if (g.bias) {
                                const float4 bb = __ldg(reinterpret_cast<const float4*>(g.bias + n + q * 4));
                                v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                            }
                            if (g.addend) {
                                const float4 aa = __ldg(reinterpret_cast<const float4*>(g.addend + off + q * 4));
                                v.x += aa.x; v.y += aa.y; v.z += aa.z; v.w += aa.w;
                            }
                            v.x = act_fn(v.x, g.act); v.y = act_fn(v.y, g.act); v.z = act_fn(v.z, g.act); v.w = act_fn(v.w, g.act);
                            *reinterpret_cast<float4*>(g.y + off + q * 4) = v;
                        }
                    }
            }
        }
    }
#undef WF_SUB
#undef WF_ADD
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}
