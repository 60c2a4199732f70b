// The halo-resident 3x3 / stride 1 / pad 1 convolution (conv3x3_tc.cuh) on CTA PAIRS: two CTAs of a
// thread-block cluster own two neighbouring output patches of 16 x 8 pixels and run ONE stream of
// tcgen05.mma.cta_group::2 instructions of M = 256 -- rows 0..127 are the first CTA's patch, rows
// 128..255 the second's.  Each CTA fetches its own halo boxes and only HALF of every weight tile (BN / 2
// filters); the tensor cores of both SMs read both halves.  Against the one-CTA kernel this halves the
// weight bytes that go from L2 into shared memory (the larger share of the fill traffic: a 32-channel
// block needs three 18 KB boxes but nine weight tiles of BN x 128 bytes) and halves the number of MMA
// instructions per SM, and one thread can issue only one tcgen05.mma per ~82 cycles whatever its shape.
//
// Roles.  In both CTAs thread 0 issues the halo boxes and the first lane of warp 2 the weight half-tiles (the three
// tiles of the taps (0, s), (1, s), (2, s) that go with one halo box arrive as ONE four-dimensional box, so the MMA
// thread waits once per halo box and then issues twelve MMAs back to back);
// all of these loads complete on the barriers of the FIRST CTA of the pair (the leader), whose warp 1
// issues every MMA.  When the MMAs that read a ring slot have finished, the leader releases that slot in
// both CTAs (one commit whose arrival goes to the same barrier of both).  Each CTA's
// warps 2-5 write out the 128 accumulator rows of its own tensor memory.  With a K split (cluster
// dimension z) every pair takes a share of the channel blocks and the partial tiles are added through
// distributed shared memory, as in the one-CTA kernel.  No load here has more than one destination CTA.
#pragma once

struct ConvPairDev {
    unsigned long long* stamp;      // device-clock stamps of this launch, or null
    float* D;
    const float* bias;
    const float* addend;
    int C, H, W, K;
    int BN, act, tmem_cols, splits, na, nb, cblk, tiles_w;
    int tma_out;                    // 0: plain stores; 16 / 32: columns per TMA-stored sub-tile (no K split, no addend)
};

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The shared::cluster address of this CTA's shared-memory address `local` in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t mapa_u32(uint32_t local, uint32_t rank) {
    uint32_t remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    return remote;
}
// Tiled load into this CTA's shared memory whose bytes are counted on a barrier of this CTA or of its partner
// (`bar` is a shared::cluster address).
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
// The same with four coordinates (the three weight half-tiles of one horizontal tap offset in one load).
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void umma_pair_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on the barrier at this CTA's address `bar` in every CTA of the cluster whose rank is set in `mask`, once every
// MMA issued so far has finished (one arrival signal sent to several CTAs; no data moves).
__device__ __forceinline__ void umma_pair_commit(uint32_t bar, uint16_t mask) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar), "h"(mask) : "memory");
}

// Write-out of one CTA's 128 accumulator rows (one warp = 4 image rows x 8 pixels) through sub-tiles in the
// swizzled layout of the output tensor map {K, W, H}, box {CW, 8, 4}; `sbase` is idle ring memory.
__device__ __forceinline__ void pair_store_tma(const CUtensorMap* tmD, const ConvPairDev& g, uint32_t tmem_base, uint32_t sbase,
                                               int quarter, int lane, int oh0, int ow0, int n0) {
    const int BN = g.BN, CW = g.tma_out, nch = BN / CW;
    const uint32_t chunk_bytes = 32u * (uint32_t)CW * 4u;
    const int oh = oh0 + quarter * 4;
    for (int j = 0; j < nch; ++j) {
        const uint32_t buf = sbase + (uint32_t)(j * 4 + quarter) * chunk_bytes;
        const uint32_t rowa = buf + (uint32_t)lane * (uint32_t)CW * 4u;
        const int nbase = n0 + j * CW;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            if (h * 16 >= CW) break;
            uint32_t r[16];
            tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(j * CW + h * 16), r);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                const int c = h * 4 + c4;                           // 16-byte chunk of the row
                const int n = nbase + c * 4;
                const uint32_t sw = (CW == 32) ? (uint32_t)(c ^ (lane & 7)) : (uint32_t)(c ^ ((lane >> 1) & 3));
                float4 v = make_float4(__uint_as_float(r[c4 * 4]), __uint_as_float(r[c4 * 4 + 1]),
                                       __uint_as_float(r[c4 * 4 + 2]), __uint_as_float(r[c4 * 4 + 3]));
                if (g.bias && n < g.K) {
                    const float4 bb = __ldg(reinterpret_cast<const float4*>(g.bias + n));
                    v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                }
                v.x = act_fn(v.x, g.act); v.y = act_fn(v.y, g.act); v.z = act_fn(v.z, g.act); v.w = act_fn(v.w, g.act);
                asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(rowa + sw * 16u), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the TMA's reads
        __syncwarp();
        if (lane == 0 && oh < g.H && ow0 < g.W && nbase < g.K) {
            tma_store_3d(tmD, buf, nbase, ow0, oh);
            tma_store_commit();
        }
    }
    if (lane == 0) tma_store_wait_read();
}

// Write-out with plain stores (bias, residual addend, activation) through a per-warp 32 x 32 staging tile of pitch 36 words.
__device__ __forceinline__ void pair_store_plain(const ConvPairDev& g, uint32_t tmem_base, uint32_t sbase, int quarter, int lane,
                                                 int oh0, int ow0, int n0) {
    const int BN = g.BN;
    const bool vec = ((g.K & 3) == 0) && ((reinterpret_cast<uintptr_t>(g.D) & 15) == 0) &&
                     (!g.addend || (reinterpret_cast<uintptr_t>(g.addend) & 15) == 0) &&
                     (!g.bias || (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0);
    const uint32_t stage = sbase + (uint32_t)quarter * (32u * 36u * 4u);
    const int sub = lane >> 3, cc = (lane & 7) * 4;           // row within a group of four, first column
    for (int c0 = 0; c0 < BN; c0 += 32) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            if (c0 + half * 16 < BN) {                        // warp-uniform
                uint32_t r[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(c0 + half * 16), r);
#pragma unroll
                for (int j = 0; j < 16; j += 4)
                    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(stage + (uint32_t)(lane * 36 + half * 16 + j) * 4u),
                                 "r"(r[j]), "r"(r[j + 1]), "r"(r[j + 2]), "r"(r[j + 3]) : "memory");
            }
        }
        __syncwarp();
        const int n = n0 + c0 + cc;
        const bool col_ok = (c0 + cc < BN) && (n < g.K);
        float4 bb = make_float4(0.f, 0.f, 0.f, 0.f);
        if (vec && col_ok && g.bias) bb = __ldg(reinterpret_cast<const float4*>(g.bias + n));
#pragma unroll 2
        for (int it = 0; it < 8; ++it) {
            const int rl = it * 4 + sub, mrow = quarter * 32 + rl;
            const int oh = oh0 + (mrow >> 3), ow = ow0 + (mrow & 7);
            if (!col_ok || oh >= g.H || ow >= g.W) continue;
            float4 v;
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                         : "r"(stage + (uint32_t)(rl * 36 + cc) * 4u));
            const long long off = ((long long)oh * g.W + ow) * g.K + n;
            if (vec) {
                v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                if (g.addend) {
                    const float4 aa = __ldg(reinterpret_cast<const float4*>(g.addend + off));
                    v.x += aa.x; v.y += aa.y; v.z += aa.z; v.w += aa.w;
                }
                v.x = act_fn(v.x, g.act); v.y = act_fn(v.y, g.act); v.z = act_fn(v.z, g.act); v.w = act_fn(v.w, g.act);
                *reinterpret_cast<float4*>(g.D + off) = v;
            } else {
                const float vv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (n + j < g.K) {
                        float t = vv[j];
                        if (g.bias) t += __ldg(g.bias + n + j);
                        if (g.addend) t += __ldg(g.addend + off + j);
                        g.D[off + j] = act_fn(t, g.act);
                    }
                }
            }
        }
        __syncwarp();                                         // the staging tile is rewritten by the next chunk
    }
}

// Grid: x = patches rounded up to an even number, y = channel tiles, z = K splits; cluster {2, 1, splits}.
__global__ void __launch_bounds__(GEMM_THREADS)
conv3x3_tc_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                       const __grid_constant__ CUtensorMap tmD, const __grid_constant__ ConvPairDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int BN = g.BN, NA = g.na, NB = g.nb;
    constexpr uint32_t a_box_bytes = 18u * 1024u;             // (16 + 2) rows of 8 pixels x 128 bytes
    const uint32_t b_half_bytes = (uint32_t)(BN / 2) * (uint32_t)BK_BYTES;
    const uint32_t b_slot_bytes = 3u * b_half_bytes;          // a weight slot: this CTA's half tiles of the taps r = 0, 1, 2 of one s
    const uint32_t a_ring = sbase, b_ring = sbase + NA * a_box_bytes;
    const uint32_t bars = b_ring + NB * b_slot_bytes;
    auto a_full = [&](int s) { return bars + 8u * s; };
    auto a_empty = [&](int s) { return bars + 8u * (CONV_MAX_NA + s); };
    auto b_full = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + s); };
    auto b_empty = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + CONV_MAX_NB + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB);
    const uint32_t holder = tmem_full_bar + 8u;
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t crank = cluster_ctarank();                 // x + 2 * z inside the cluster
    const uint32_t half = crank & 1u;                         // 0: the leader of the pair, 1: its partner
    const uint32_t leader_rank = crank & ~1u;
    const uint16_t pair_mask = (uint16_t)(3u << leader_rank); // both CTAs of this pair
    const int splits = g.splits, sp = (int)blockIdx.z;
    const int patch = (int)blockIdx.x;
    const int tile_h = patch / g.tiles_w, tile_w = patch - tile_h * g.tiles_w;
    const int oh0 = tile_h * 16, ow0 = tile_w * 8, n0 = blockIdx.y * BN;   // a patch past the last one lies below the image: zero boxes, nothing stored
    const int cb0 = (g.cblk * sp) / splits;
    const int ncb = (g.cblk * (sp + 1)) / splits - cb0;

    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
        if (g.tma_out) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmD)) : "memory");
        for (int s = 0; s < NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
        for (int s = 0; s < NB; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
        mbar_init(tmem_full_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                          // the same warp of both CTAs of the pair
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"((uint32_t)g.tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    cluster_sync_all();                                       // the partner's loads arrive on the leader's barriers: initialised before any load
    tc_fence_after();
    const uint32_t tmem_base = *holder_ptr;
    pdl_wait();                                               // set-up above overlaps the previous kernel's tail
    if (threadIdx.x == 32) stamp_start(g.stamp);

    if (warp == 0) {
        if (lane == 0) {
            // halo boxes of this CTA's patch; their bytes are counted on the leader's barrier, which expects both CTAs' boxes
            bool ok = true;
            int sa = 0;
            uint32_t pa = 0;
            for (int cbi = 0; cbi < ncb && ok; ++cbi) {
                const int c0 = (cb0 + cbi) * 32;
                for (int s = 0; s < 3 && ok; ++s) {
                    ok = mbar_wait(a_empty(sa), pa ^ 1u);
                    if (!ok) break;
                    if (half == 0) mbar_expect_tx(a_full(sa), 2u * a_box_bytes);
                    tma_load_3d_pair(a_ring + sa * a_box_bytes, &tmA, c0, ow0 + s - 1, oh0 - 1, mapa_u32(a_full(sa), leader_rank));
                    if (++sa == NA) { sa = 0; pa ^= 1u; }
                }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && half == 0) {
            // instruction descriptor: fp32 accumulate, TF32 operands, both K-major, N = BN, M = 256 over the pair
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
            bool ok = true;
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            for (int cbi = 0; cbi < ncb && ok; ++cbi) {
                for (int s = 0; s < 3 && ok; ++s) {
                    ok = mbar_wait(a_full(sa), pa);
                    if (!ok) break;
                    const uint32_t a_box = a_ring + sa * a_box_bytes;
                    ok = mbar_wait(b_full(sb), pb);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t b_slot = b_ring + sb * b_slot_bytes;
#pragma unroll
                    for (int r = 0; r < 3; ++r) {
                        const uint64_t bdesc = make_smem_desc(b_slot + (uint32_t)r * b_half_bytes);
                        const uint64_t adesc = make_smem_desc(a_box + (uint32_t)r * 1024u);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)         // 4 MMAs of 32 bytes of K each
                            umma_pair_tf32(tmem_base, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (cbi | s | r | kk) ? 1u : 0u);
                    }
                    umma_pair_commit(b_empty(sb), pair_mask);          // both slots are free again in both CTAs
                    if (++sb == NB) { sb = 0; pb ^= 1u; }
                    if (ok) umma_pair_commit(a_empty(sa), pair_mask);
                    if (++sa == NA) { sa = 0; pa ^= 1u; }
                }
            }
            if (ok) umma_pair_commit(tmem_full_bar, pair_mask);
            else atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        bool ok = true;
        if (warp == 2 && lane == 0) {
            // this CTA's half of every weight tile: filters n0 + half * BN / 2 ...
            int sb = 0;
            uint32_t pb = 0;
            const int nrow = n0 + (int)half * (BN / 2);
            for (int cbi = 0; cbi < ncb && ok; ++cbi) {
                const int c0 = (cb0 + cbi) * 32;
                for (int s = 0; s < 3 && ok; ++s) {
                    ok = mbar_wait(b_empty(sb), pb ^ 1u);
                    if (!ok) break;
                    if (half == 0) mbar_expect_tx(b_full(sb), 2u * b_slot_bytes);
                    tma_load_4d_pair(b_ring + sb * b_slot_bytes, &tmB, c0, nrow, s, 0, mapa_u32(b_full(sb), leader_rank));
                    if (++sb == NB) { sb = 0; pb ^= 1u; }
                }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
        ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;       // the whole warp takes the producer's result
        ok = mbar_wait(tmem_full_bar, 0) && ok;
        ok = __all_sync(0xffffffffu, (int)ok) != 0;           // (the epilogue's TMEM reads are warp-wide instructions)
        tc_fence_after();
        const int quarter = warp & 3;                         // TMEM lanes this warp may read
        if (!ok) {
            if (lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        } else if (splits == 1 && g.tma_out) {
            pair_store_tma(&tmD, g, tmem_base, sbase, quarter, lane, oh0, ow0, n0);
        } else if (splits == 1) {
            pair_store_plain(g, tmem_base, sbase, quarter, lane, oh0, ow0, n0);
        } else {
            // park this CTA's partial tile in its own shared memory (both rings are idle by now): P[row][col], pitch BN + 4 words
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
    if (splits > 1) {
        // Split-K write-out: the CTAs that hold partial tiles of the same patch (same half, every z) each add a share of
        // the 128 rows through distributed shared memory, in the order of z, and apply the epilogue.
        cluster_sync_all();
        if (warp >= 2 && g_device_status == 0) {
            const int t = (int)threadIdx.x - 64;
            const int rows_per = BM / splits, r0 = sp * rows_per;
            const int c4n = BN / 4;
            const bool vec = ((g.K & 3) == 0) && ((reinterpret_cast<uintptr_t>(g.D) & 15) == 0) &&
                             (!g.addend || (reinterpret_cast<uintptr_t>(g.addend) & 15) == 0) &&
                             (!g.bias || (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0);
            const int total = rows_per * c4n;
#pragma unroll 1
            for (int idx = t; idx < total; idx += 128) {
                const int rq = idx / c4n;
                const int rr = r0 + rq, cc = (idx - rq * c4n) * 4;
                const uint32_t local = sbase + ((uint32_t)rr * (uint32_t)(BN + 4) + (uint32_t)cc) * 4u;
                float4 v[4];
#pragma unroll
                for (int rk = 0; rk < 4; ++rk) {
                    if (rk < splits) {
                        const uint32_t remote = mapa_u32(local, half + 2u * (uint32_t)rk);
                        asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v[rk].x), "=f"(v[rk].y), "=f"(v[rk].z), "=f"(v[rk].w) : "r"(remote));
                    }
                }
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int rk = 0; rk < 4; ++rk)
                    if (rk < splits) { acc.x += v[rk].x; acc.y += v[rk].y; acc.z += v[rk].z; acc.w += v[rk].w; }
                const int oh = oh0 + (rr >> 3), ow = ow0 + (rr & 7), n = n0 + cc;
                if (oh >= g.H || ow >= g.W || n >= g.K) continue;
                const long long pix = (long long)oh * g.W + ow;
                float* drow = g.D + pix * g.K;
                const float* arow = g.addend ? g.addend + pix * g.K : nullptr;
                float vv[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (vec || n + j < g.K) {
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
                        if (n + j < g.K) drow[n + j] = vv[j];
                }
            }
        }
    }
    // Nobody leaves while its partner's MMAs, barrier arrivals or reads of parked tiles may still touch its shared memory.
    tc_fence_before();
    cluster_sync_all();
    if (threadIdx.x == 0) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}
