// Tensor-core 3x3 / stride 1 / pad 1 convolution as an implicit GEMM whose A operand keeps its
// halo in shared memory.  Included by gemm_tc.cu (inside namespace nnv, after the PTX helpers).
//
// The plain implicit GEMM fetches one 128-pixel x 32-channel tile of the activation per filter tap:
// nine fetches of mostly the same pixels.  Here one CTA owns an output patch of TH x 8 pixels
// (TH = 16 or 32, i.e. one or two 128-row MMA tiles) and, per block of 32 input channels, fetches
// the patch's halo only three times -- once per horizontal tap offset s, as a (TH + 2) x 8 pixel
// box.  Inside such a box a vertical tap offset r is a whole number of 8-pixel rows, that is
// r x 1024 bytes of shared memory, which is exactly one 8-row group of the 128-byte-swizzled
// K-major layout: the MMA for tap (r, s) reads box s through a descriptor whose start address is
// moved down by r groups.  Every tile base stays 1024-byte aligned, so the swizzle phase of the
// TMA's writes and of the MMA's reads agree.  Activation bytes from L2 drop from 9 x 16 KB to
// 3 x (TH + 2) KB per channel block and MMA tile, and with TH = 32 the two MMA tiles share every
// weight tile.
//
// Output pixel (oh0 + g, ow0 + px) of MMA tile mt is TMEM lane / MMA row 8 * (g - 16 * mt) + px.
// Pixels outside the image are zero-filled by the TMA on the way in and skipped on the way out.
//
// Warp roles and the bounded waits are those of gemm_tc_kernel; there are two rings here, one of
// activation boxes (reused by three taps each) and one of weight tiles (one tap each).
#pragma once

struct ConvDev {
    unsigned long long* stamp;      // device-clock stamps of this launch, or null
    float* D;
    const float* bias;
    const float* addend;
    int C, H, W, K;                 // input channels, image (input = output grid), output channels
    int BN, MT, act, tmem_cols, splits, na, nb, cblk, tiles_w;
    int tma_out;                    // 0: plain stores; 16 / 32: columns per TMA-stored sub-tile (no K split, no addend)
    int bf16;                       // 1: BF16 math -- the fp32 halo boxes are rounded to bf16 in shared memory, the weights arrive as bf16
};

constexpr int CONV_MAX_NA = 4, CONV_MAX_NB = 8;

__global__ void __launch_bounds__(GEMM_THREADS)
conv3x3_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                  const __grid_constant__ CUtensorMap tmD, const ConvDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int BN = g.BN, MT = g.MT, NA = g.na, NB = g.nb;
    // BF16 math: a box slot holds the fp32 box as the TMA delivers it (128-byte rows, swizzled) and, behind it, the same
    // pixels rounded to bf16 in the un-swizzled core-matrix layout [8-channel chunk][pixel row][16 bytes]; there an
    // image row of the patch (8 pixels) is 128 bytes, so a vertical tap offset is again a shift of the descriptor's
    // start address.  The weights arrive as bf16 in the same layout (one box of four 8-element chunks x BN rows per tile).
    const bool bf16 = g.bf16 != 0;
    const uint32_t box_rows = (uint32_t)(16 * MT + 2) * 8u;        // pixel rows of a halo box
    const uint32_t a_box_bytes = box_rows * 128u;
    const uint32_t a_slot_bytes = a_box_bytes + (bf16 ? box_rows * 64u : 0u);
    const uint32_t b_slot_bytes = (uint32_t)BN * (bf16 ? 64u : (uint32_t)BK_BYTES);
    const uint32_t a_ring = sbase, b_ring = sbase + NA * a_slot_bytes;
    const uint32_t bars = b_ring + NB * b_slot_bytes;
    auto a_full = [&](int s) { return bars + 8u * s; };
    auto a_empty = [&](int s) { return bars + 8u * (CONV_MAX_NA + s); };
    auto b_full = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + s); };
    auto b_empty = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + CONV_MAX_NB + s); };
    const uint32_t tmem_full_bar = bars + 8u * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB);
    const uint32_t holder = tmem_full_bar + 8u;
    auto a_conv = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB + 2 + s); };   // box s is converted
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int splits = g.splits, sp = (int)blockIdx.z;       // the cluster spans grid z: one K split per CTA
    const int tile_h = (int)blockIdx.x / g.tiles_w, tile_w = (int)blockIdx.x - tile_h * g.tiles_w;
    const int oh0 = tile_h * 16 * MT, ow0 = tile_w * 8, n0 = blockIdx.y * BN;
    const int cb0 = (g.cblk * sp) / splits;
    const int ncb = (g.cblk * (sp + 1)) / splits - cb0;

    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
        if (g.tma_out) asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmD)) : "memory");
        for (int s = 0; s < NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); mbar_init(a_conv(s), 128); }
        for (int s = 0; s < NB; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
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
    pdl_wait();                                               // set-up above overlaps the previous kernel's tail
    if (threadIdx.x == 32) stamp_start(g.stamp);

    // One weight tile into ring slot `sb`: a 128-byte-swizzled fp32 tile, or a box of four 8-element bf16 chunks x BN rows
    auto issue_b = [&](int sb, int tap, int c0) {
        const uint32_t dst = b_ring + sb * b_slot_bytes;
        mbar_expect_tx(b_full(sb), b_slot_bytes);
        if (bf16) {
            tma_load_3d(dst, &tmB, 0, n0, (tap * g.C + c0) >> 3, b_full(sb));   // {8 elements, BN rows, 4 chunks} in one load
        } else {
            tma_load_3d(dst, &tmB, tap * g.C + c0, n0, 0, b_full(sb));
        }
    };

    // Two producers (TF32 math; with BF16 math warps 2-5 convert the boxes, so warp 0 issues the weight tiles too): a shared-memory fill costs its issuing thread ~150 cycles whatever its size, so the halo boxes
    // and the (smaller, three times as many) weight tiles are issued by different warps -- warp 2's first lane serves
    // the weight ring before it joins the epilogue.
    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int sa = 0, sb0 = 0;                              // ring slots and their phases, carried along (no divisions:
            uint32_t pa = 0, pb0 = 0;                         // every instruction of this single-thread loop is latency)
            for (int cbi = 0; cbi < ncb && ok; ++cbi) {
                const int c0 = (cb0 + cbi) * 32;
                for (int s = 0; s < 3 && ok; ++s) {
                    ok = mbar_wait(a_empty(sa), pa ^ 1u);
                    if (!ok) break;
                    mbar_expect_tx(a_full(sa), a_box_bytes);
                    tma_load_3d(a_ring + sa * a_slot_bytes, &tmA, c0, ow0 + s - 1, oh0 - 1, a_full(sa));
                    if (++sa == NA) { sa = 0; pa ^= 1u; }
                    if (bf16) {
                        for (int r = 0; r < 3; ++r) {
                            ok = mbar_wait(b_empty(sb0), pb0 ^ 1u);
                            if (!ok) break;
                            issue_b(sb0, r * 3 + s, c0);
                            if (++sb0 == NB) { sb0 = 0; pb0 ^= 1u; }
                        }
                    }
                }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // instruction descriptor: fp32 accumulate, TF32 (or bf16) operands, both K-major, N = BN, M = 128
            const uint32_t fmt = bf16 ? 1u : 2u;
            const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            const uint32_t lbo_a = box_rows * 16u, lbo_b = (uint32_t)BN * 16u;
            bool ok = true;
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            for (int cbi = 0; cbi < ncb && ok; ++cbi) {
                for (int s = 0; s < 3 && ok; ++s) {
                    ok = mbar_wait(bf16 ? a_conv(sa) : a_full(sa), pa);
                    if (!ok) break;
                    const uint32_t a_box = a_ring + sa * a_slot_bytes;
                    for (int r = 0; r < 3; ++r) {
                        ok = mbar_wait(b_full(sb), pb);
                        if (!ok) break;
                        tc_fence_after();
                        if (bf16) {
                            const uint32_t a_bf = a_box + a_box_bytes, b_bf = b_ring + sb * b_slot_bytes;
                            for (int mt = 0; mt < MT; ++mt) {
#pragma unroll
                                for (int kk = 0; kk < 2; ++kk)     // 2 MMAs of 16 bf16 of K = two core matrices each
                                    umma<true>(tmem_base + (uint32_t)(mt * BN),
                                               make_smem_desc_plain(a_bf + (uint32_t)(mt * 16 + r) * 128u + (uint32_t)kk * 2u * lbo_a, lbo_a, 128),
                                               make_smem_desc_plain(b_bf + (uint32_t)kk * 2u * lbo_b, lbo_b, 128), idesc, (cbi | s | r | kk) ? 1u : 0u);
                            }
                        } else {
                        const uint64_t bdesc = make_smem_desc(b_ring + sb * b_slot_bytes);
                        for (int mt = 0; mt < MT; ++mt) {
                            const uint64_t adesc = make_smem_desc(a_box + (uint32_t)(mt * 16 + r) * 1024u);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)     // 4 MMAs of 32 bytes of K each
                                umma<false>(tmem_base + (uint32_t)(mt * BN), adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2),
                                            idesc, (cbi | s | r | kk) ? 1u : 0u);
                        }
                        }
                        umma_commit(b_empty(sb));
                        if (++sb == NB) { sb = 0; pb ^= 1u; }
                    }
                    if (ok) umma_commit(a_empty(sa));
                    if (++sa == NA) { sa = 0; pa ^= 1u; }
                }
            }
            if (ok) umma_commit(tmem_full_bar);
            else atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        bool ok = true;
        if (bf16) {
            // warps 2-5 round every halo box to bf16 as it lands (one pixel row of 32 channels per thread and pass)
            int sa = 0;
            uint32_t pa = 0;
            for (int it = 0; it < 3 * ncb && ok; ++it) {
                ok = mbar_wait(a_full(sa), pa);
                if (!ok) break;
                const uint32_t a_box = a_ring + sa * a_slot_bytes;
                for (uint32_t row = threadIdx.x - 64; row < box_rows; row += 128) convert_row_bf16(a_box, a_box + a_box_bytes, (int)row, (int)box_rows);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
                mbar_arrive(a_conv(sa));
                if (++sa == NA) { sa = 0; pa ^= 1u; }
            }
            ok = __all_sync(0xffffffffu, (int)ok) != 0;
        } else if (warp == 2 && lane == 0) {                  // the weight-tile producer
            int sb = 0;
            uint32_t pb = 0;
            for (int cbi = 0; cbi < ncb && ok; ++cbi) {
                const int c0 = (cb0 + cbi) * 32;
                for (int s = 0; s < 3 && ok; ++s) {
                    for (int r = 0; r < 3; ++r) {
                        ok = mbar_wait(b_empty(sb), pb ^ 1u);
                        if (!ok) break;
                        issue_b(sb, r * 3 + s, c0);
                        if (++sb == NB) { sb = 0; pb ^= 1u; }
                    }
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
        const int row = quarter * 32 + lane;                  // MMA row = 8 * (patch row) + (patch column)
        if (!ok) {
            if (lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        } else if (splits == 1 && g.tma_out) {
            // Write-out by TMA.  A warp's 32 accumulator rows are 4 image rows x 8 pixels of the patch: per chunk of CW
            // output channels the lanes write their rows (+ bias, activation) into a sub-tile in the swizzled layout of
            // the output tensor map {K, W, H}, box {CW, 8, 4}, and one lane stores it; pixels and channels outside the
            // tensor are clipped by the TMA.  The sub-tiles reuse the rings, which are idle by now.
            const int CW = g.tma_out, nch = BN / CW;
            const uint32_t chunk_bytes = 32u * (uint32_t)CW * 4u;
            for (int mt = 0; mt < MT; ++mt) {
                const int oh = oh0 + mt * 16 + quarter * 4;
                for (int j = 0; j < nch; ++j) {
                    const uint32_t buf = sbase + (uint32_t)((mt * nch + j) * 4 + quarter) * chunk_bytes;
                    const uint32_t rowa = buf + (uint32_t)lane * (uint32_t)CW * 4u;
                    const int nbase = n0 + j * CW;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        if (h * 16 >= CW) break;
                        uint32_t r[16];
                        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * BN + j * CW + h * 16), r);
#pragma unroll
                        for (int c4 = 0; c4 < 4; ++c4) {
                            const int c = h * 4 + c4;                       // 16-byte chunk of the row
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
                        tma_store_3d(&tmD, buf, nbase, ow0, oh);
                        tma_store_commit();
                    }
                }
            }
            if (lane == 0) tma_store_wait_read();
        } else if (splits == 1) {
            // Each warp turns its 32 accumulator rows (one pixel per lane) into pixel-contiguous
            // stores through a private 32 x 32 staging tile (row pitch 36 words; both rings are idle
            // by now): lane = pixel on the way in, 8 lanes x 16 bytes = 128 contiguous bytes of one
            // pixel on the way out, so every global access covers whole 128-byte lines.
            const bool vec = ((g.K & 3) == 0) && ((reinterpret_cast<uintptr_t>(g.D) & 15) == 0) &&
                             (!g.addend || (reinterpret_cast<uintptr_t>(g.addend) & 15) == 0) &&
                             (!g.bias || (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0);
            const uint32_t stage = sbase + (uint32_t)quarter * (32u * 36u * 4u);
            const int sub = lane >> 3, cc = (lane & 7) * 4;       // row within a group of four, first column
            for (int mt = 0; mt < MT; ++mt) {
                for (int c0 = 0; c0 < BN; c0 += 32) {
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        if (c0 + half * 16 < BN) {                // warp-uniform
                            uint32_t r[16];
                            tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * BN + c0 + half * 16), r);
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
                        const int oh = oh0 + mt * 16 + (mrow >> 3), ow = ow0 + (mrow & 7);
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
                    __syncwarp();                                 // the staging tile is rewritten by the next chunk
                }
            }
        } else {
            // park this CTA's partial tiles in its own shared memory (both rings are idle by now):
            // P[mt * 128 + row][col], row pitch BN + 4 words
            for (int mt = 0; mt < MT; ++mt) {
                const uint32_t prow = sbase + (uint32_t)(mt * 128 + row) * (uint32_t)(BN + 4) * 4u;
                for (int c0 = 0; c0 < BN; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * BN + c0), r);
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(prow + (uint32_t)(c0 + j) * 4u), "r"(r[j]),
                                     "r"(r[j + 1]), "r"(r[j + 2]), "r"(r[j + 3]) : "memory");
                }
            }
        }
    }
    __syncwarp();
    if (splits > 1) {
        // Split-K write-out, as in gemm_tc_kernel: CTA `sp` sums its share of the 128 * MT rows over
        // the cluster through distributed shared memory in rank order, then applies the epilogue.
        cluster_sync_all();
        if (warp >= 2 && g_device_status == 0) {
            const int t = (int)threadIdx.x - 64;
            const int rows_per = (BM * MT) / splits, r0 = sp * rows_per;
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
                const int mt = rr >> 7, mrow = rr & 127;
                const int oh = oh0 + mt * 16 + (mrow >> 3), ow = ow0 + (mrow & 7), n = n0 + cc;
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
        cluster_sync_all();                                   // nobody leaves while its tiles may still be read
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

// ---- persistent form ----------------------------------------------------------------------------
// One CTA per SM walks over the output tiles t = blockIdx.x, blockIdx.x + gridDim.x, ...  The rings keep
// running from one tile into the next, so the producer is already filling tile t+1 while tile t drains; TMEM
// holds TWO accumulators, so the MMAs of tile t+1 run while the epilogue warps read and write out tile t
// (tmem_full / tmem_empty barriers per accumulator).  Set-up (barriers, TMEM allocation, descriptor fetch) is
// paid once per CTA instead of once per tile.  No K split here: layers that need one take the kernel above.
// The epilogue's per-warp staging tiles have their own shared memory, since the rings are never idle.
struct ConvPDev {
    unsigned long long* stamp;
    float* D;
    const float* bias;
    const float* addend;
    int C, H, W, K;
    int BN, act, tmem_cols, na, nb, cblk, tiles_w, n_tiles, tiles_total;   // n_tiles: channel tiles; tiles_total = patches x n_tiles
};

__global__ void __launch_bounds__(GEMM_THREADS)
conv3x3_tc_persistent_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const ConvPDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int BN = g.BN, NA = g.na, NB = g.nb;
    constexpr uint32_t a_slot_bytes = 18u * 1024u;                 // (16 + 2) rows of 8 pixels x 128 bytes
    const uint32_t b_slot_bytes = (uint32_t)BN * BK_BYTES;
    const uint32_t a_ring = sbase, b_ring = sbase + NA * a_slot_bytes;
    const uint32_t stage0 = b_ring + NB * b_slot_bytes;            // 4 warps x 32 rows x 36 words
    const uint32_t bars = stage0 + 4u * 32u * 36u * 4u;
    auto a_full = [&](int s) { return bars + 8u * s; };
    auto a_empty = [&](int s) { return bars + 8u * (CONV_MAX_NA + s); };
    auto b_full = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + s); };
    auto b_empty = [&](int s) { return bars + 8u * (2 * CONV_MAX_NA + CONV_MAX_NB + s); };
    auto t_full = [&](int a) { return bars + 8u * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB + a); };
    auto t_empty = [&](int a) { return bars + 8u * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB + 2 + a); };
    const uint32_t holder = bars + 8u * (2 * CONV_MAX_NA + 2 * CONV_MAX_NB + 4);
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
        for (int s = 0; s < NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
        for (int s = 0; s < NB; ++s) { mbar_init(b_full(s), 1); mbar_init(b_empty(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(t_full(a), 1); mbar_init(t_empty(a), 4); }
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
    pdl_wait();                                               // set-up above overlaps the previous kernel's tail
    if (threadIdx.x == 32) stamp_start(g.stamp);

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            for (int t = blockIdx.x; t < g.tiles_total && ok; t += gridDim.x) {
                const int patch = t / g.n_tiles, nt = t - patch * g.n_tiles;
                const int tile_h = patch / g.tiles_w, tile_w = patch - tile_h * g.tiles_w;
                const int oh0 = tile_h * 16, ow0 = tile_w * 8, n0 = nt * BN;
                for (int cbi = 0; cbi < g.cblk && ok; ++cbi) {
                    const int c0 = cbi * 32;
                    for (int s = 0; s < 3 && ok; ++s) {
                        ok = mbar_wait(a_empty(sa), pa ^ 1u);
                        if (!ok) break;
                        mbar_expect_tx(a_full(sa), a_slot_bytes);
                        tma_load_3d(a_ring + sa * a_slot_bytes, &tmA, c0, ow0 + s - 1, oh0 - 1, a_full(sa));
                        if (++sa == NA) { sa = 0; pa ^= 1u; }
                        for (int r = 0; r < 3; ++r) {
                            ok = mbar_wait(b_empty(sb), pb ^ 1u);
                            if (!ok) break;
                            mbar_expect_tx(b_full(sb), b_slot_bytes);
                            tma_load_3d(b_ring + sb * b_slot_bytes, &tmB, (r * 3 + s) * g.C + c0, n0, 0, b_full(sb));
                            if (++sb == NB) { sb = 0; pb ^= 1u; }
                        }
                    }
                }
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            bool ok = true;
            int sa = 0, sb = 0;
            uint32_t pa = 0, pb = 0;
            int lt = 0;                                           // this CTA's tile count so far
            for (int t = blockIdx.x; t < g.tiles_total && ok; t += gridDim.x, ++lt) {
                const int acc = lt & 1;
                ok = mbar_wait(t_empty(acc), (((uint32_t)lt >> 1) & 1u) ^ 1u);   // the epilogue has drained this accumulator
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
                for (int cbi = 0; cbi < g.cblk && ok; ++cbi) {
                    for (int s = 0; s < 3 && ok; ++s) {
                        ok = mbar_wait(a_full(sa), pa);
                        if (!ok) break;
                        const uint32_t a_box = a_ring + sa * a_slot_bytes;
                        for (int r = 0; r < 3; ++r) {
                            ok = mbar_wait(b_full(sb), pb);
                            if (!ok) break;
                            tc_fence_after();
                            const uint64_t bdesc = make_smem_desc(b_ring + sb * b_slot_bytes);
                            const uint64_t adesc = make_smem_desc(a_box + (uint32_t)r * 1024u);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                umma<false>(tmem_d, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (cbi | s | r | kk) ? 1u : 0u);
                            umma_commit(b_empty(sb));
                            if (++sb == NB) { sb = 0; pb ^= 1u; }
                        }
                        if (ok) umma_commit(a_empty(sa));
                        if (++sa == NA) { sa = 0; pa ^= 1u; }
                    }
                }
                if (ok) umma_commit(t_full(acc));
            }
            if (!ok) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        const int quarter = warp & 3;                         // TMEM lanes this warp may read
        const bool vec = ((g.K & 3) == 0) && ((reinterpret_cast<uintptr_t>(g.D) & 15) == 0) &&
                         (!g.addend || (reinterpret_cast<uintptr_t>(g.addend) & 15) == 0) &&
                         (!g.bias || (reinterpret_cast<uintptr_t>(g.bias) & 15) == 0);
        const uint32_t stage = stage0 + (uint32_t)quarter * (32u * 36u * 4u);
        const int sub = lane >> 3, cc = (lane & 7) * 4;
        int lt = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < g.tiles_total && ok; t += gridDim.x, ++lt) {
            const int acc = lt & 1;
            const int patch = t / g.n_tiles, nt = t - patch * g.n_tiles;
            const int tile_h = patch / g.tiles_w, tile_w = patch - tile_h * g.tiles_w;
            const int oh0 = tile_h * 16, ow0 = tile_w * 8, n0 = nt * BN;
            ok = mbar_wait(t_full(acc), ((uint32_t)lt >> 1) & 1u);
            if (!ok) break;
            tc_fence_after();
            for (int c0 = 0; c0 < BN; c0 += 32) {
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (c0 + half * 16 < BN) {                // warp-uniform
                        uint32_t r[16];
                        tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + c0 + half * 16), r);
#pragma unroll
                        for (int j = 0; j < 16; j += 4)
                            asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(stage + (uint32_t)(lane * 36 + half * 16 + j) * 4u),
                                         "r"(r[j]), "r"(r[j + 1]), "r"(r[j + 2]), "r"(r[j + 3]) : "memory");
                    }
                }
                if (c0 + 32 >= BN) {                          // every TMEM read of this tile is done: hand the accumulator back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(t_empty(acc));
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
                                float tt = vv[j];
                                if (g.bias) tt += __ldg(g.bias + n + j);
                                if (g.addend) tt += __ldg(g.addend + off + j);
                                g.D[off + j] = act_fn(tt, g.act);
                            }
                        }
                    }
                }
                __syncwarp();                                 // the staging tile is rewritten by the next chunk
            }
        }
        if (!ok && lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}

// ---- weights-stationary form ---------------------------------------------------------------------
// For layers whose whole weight slice of one channel tile fits shared memory (C x BN <= 4096 words per tap, e.g.
// 64 -> 64): every CTA of the one-tile kernel above re-reads that slice from L2 (147 KB for 46 KB of activation boxes
// per channel block), and on an SM the fill of shared memory, not the tensor pipe, is what the tile rate waits for.
// Here one CTA per SM loads its channel tile's 9 x C/32 weight tiles ONCE, each behind its own barrier so that the
// first MMAs start as soon as the first tap has landed, and then walks over output patches p = blockIdx.x,
// blockIdx.x + gridDim.x, ...: per patch only the halo boxes move.  TMEM holds two accumulators (the MMAs of patch
// t+1 run while patch t is written out), and the write-out goes through swizzled sub-tiles and TMA stores as above
// (one sub-tile per warp: a warp waits for its previous store to have read it before the next chunk overwrites it).
struct ConvWDev {
    unsigned long long* stamp;
    const float* bias;
    int C, H, W, K;
    int BN, act, tmem_cols, cblk, tiles_w, patches, cw;       // cw: columns per stored sub-tile (16 or 32)
};

constexpr int CONVW_NA = 3;                                    // halo boxes in flight
constexpr int CONVW_MAX_WT = 36;                               // weight tiles (9 taps x up to 4 channel blocks)

__global__ void __launch_bounds__(GEMM_THREADS)
conv3x3_tc_ws_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmD, const ConvWDev g) {
    extern __shared__ uint8_t smem_raw[];
    pdl_trigger();
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const int BN = g.BN, NWT = 9 * g.cblk;
    constexpr uint32_t a_slot_bytes = 18u * 1024u;                 // (16 + 2) rows of 8 pixels x 128 bytes
    const uint32_t w_tile_bytes = (uint32_t)BN * BK_BYTES;
    const uint32_t w_base = sbase, a_ring = sbase + (uint32_t)NWT * w_tile_bytes;
    const uint32_t stage0 = a_ring + CONVW_NA * a_slot_bytes;      // 4 warps x one sub-tile of 32 rows x 32 words
    const uint32_t bars = stage0 + 4u * 4096u;
    auto w_full = [&](int i) { return bars + 8u * i; };
    auto a_full = [&](int s) { return bars + 8u * (CONVW_MAX_WT + s); };
    auto a_empty = [&](int s) { return bars + 8u * (CONVW_MAX_WT + CONVW_NA + s); };
    auto t_full = [&](int a) { return bars + 8u * (CONVW_MAX_WT + 2 * CONVW_NA + a); };
    auto t_empty = [&](int a) { return bars + 8u * (CONVW_MAX_WT + 2 * CONVW_NA + 2 + a); };
    const uint32_t holder = bars + 8u * (CONVW_MAX_WT + 2 * CONVW_NA + 4);
    volatile uint32_t* holder_ptr = reinterpret_cast<volatile uint32_t*>(smem_raw + (holder - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.y * BN;
    if (warp == 0 && lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmA)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmB)) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmD)) : "memory");
        for (int i = 0; i < NWT; ++i) mbar_init(w_full(i), 1);
        for (int s = 0; s < CONVW_NA; ++s) { mbar_init(a_full(s), 1); mbar_init(a_empty(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(t_full(a), 1); mbar_init(t_empty(a), 4); }
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
    pdl_wait();                                               // set-up above overlaps the previous kernel's tail
    if (threadIdx.x == 32) stamp_start(g.stamp);

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int sa = 0;
            uint32_t pa = 0;
            bool first = true;
            for (int t = blockIdx.x; t < g.patches && ok; t += gridDim.x) {
                const int tile_h = t / g.tiles_w, tile_w = t - tile_h * g.tiles_w;
                const int oh0 = tile_h * 16, ow0 = tile_w * 8;
                for (int cbi = 0; cbi < g.cblk && ok; ++cbi) {
                    const int c0 = cbi * 32;
                    for (int s = 0; s < 3; ++s) {
                        ok = mbar_wait(a_empty(sa), pa ^ 1u);
                        if (!ok) break;
                        mbar_expect_tx(a_full(sa), a_slot_bytes);
                        tma_load_3d(a_ring + sa * a_slot_bytes, &tmA, c0, ow0 + s - 1, oh0 - 1, a_full(sa));
                        if (++sa == CONVW_NA) { sa = 0; pa ^= 1u; }
                        if (first) {                              // the weight tiles, in the order the MMAs will want them
                            for (int r = 0; r < 3; ++r) {
                                const int wi = cbi * 9 + r * 3 + s;
                                mbar_expect_tx(w_full(wi), w_tile_bytes);
                                tma_load_3d(w_base + (uint32_t)wi * w_tile_bytes, &tmB, (r * 3 + s) * g.C + c0, n0, 0, w_full(wi));
                            }
                        }
                    }
                }
                first = false;
            }
            if (!ok) {
                atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
                for (int i = 0; i < 1000; ++i) __nanosleep(1000);   // let loads already in flight land
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
            bool ok = true;
            int sa = 0;
            uint32_t pa = 0;
            int lt = 0;                                           // this CTA's patch count so far
            for (int t = blockIdx.x; t < g.patches && ok; t += gridDim.x, ++lt) {
                const int acc = lt & 1;
                ok = mbar_wait(t_empty(acc), (((uint32_t)lt >> 1) & 1u) ^ 1u);   // the epilogue has drained this accumulator
                if (!ok) break;
                tc_fence_after();
                const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BN);
                for (int cbi = 0; cbi < g.cblk && ok; ++cbi) {
                    for (int s = 0; s < 3 && ok; ++s) {
                        ok = mbar_wait(a_full(sa), pa);
                        if (!ok) break;
                        const uint32_t a_box = a_ring + sa * a_slot_bytes;
                        for (int r = 0; r < 3; ++r) {
                            const int wi = cbi * 9 + r * 3 + s;
                            if (lt == 0) {                        // later patches find every weight tile in place
                                ok = mbar_wait(w_full(wi), 0);
                                if (!ok) break;
                            }
                            tc_fence_after();
                            const uint64_t bdesc = make_smem_desc(w_base + (uint32_t)wi * w_tile_bytes);
                            const uint64_t adesc = make_smem_desc(a_box + (uint32_t)r * 1024u);
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk)
                                umma<false>(tmem_d, adesc + (uint64_t)(kk * 2), bdesc + (uint64_t)(kk * 2), idesc, (cbi | s | r | kk) ? 1u : 0u);
                        }
                        if (ok) umma_commit(a_empty(sa));
                        if (++sa == CONVW_NA) { sa = 0; pa ^= 1u; }
                    }
                }
                if (ok) umma_commit(t_full(acc));
            }
            if (!ok) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
        }
    } else {
        const int quarter = warp & 3;                         // TMEM lanes this warp may read: 4 image rows x 8 pixels
        const int CW = g.cw, nch = BN / CW;
        const uint32_t buf = stage0 + (uint32_t)quarter * 4096u;
        const uint32_t rowa = buf + (uint32_t)lane * (uint32_t)CW * 4u;
        int lt = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < g.patches && ok; t += gridDim.x, ++lt) {
            const int acc = lt & 1;
            const int tile_h = t / g.tiles_w, tile_w = t - tile_h * g.tiles_w;
            const int oh = tile_h * 16 + quarter * 4, ow0 = tile_w * 8;
            ok = mbar_wait(t_full(acc), ((uint32_t)lt >> 1) & 1u);
            if (!ok) break;
            tc_fence_after();
            for (int j = 0; j < nch; ++j) {
                const int nbase = n0 + j * CW;
                uint32_t ra[16], rb[16];
                tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + j * CW), ra);
                if (CW == 32) tmem_ld16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN + j * CW + 16), rb);
                if (j == nch - 1) {                           // every TMEM read of this patch is done: hand the accumulator back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(t_empty(acc));
                }
                if (lane == 0) tma_store_wait_read();         // the previous store has read the sub-tile
                __syncwarp();
#pragma unroll
                for (int c = 0; c < 8; ++c) {                 // 16-byte chunks of the row
                    if (c * 4 >= CW) break;
                    const int n = nbase + c * 4;
                    const uint32_t sw = (CW == 32) ? (uint32_t)(c ^ (lane & 7)) : (uint32_t)(c ^ ((lane >> 1) & 3));
                    const int q = (c & 3) * 4;
                    float4 v = c < 4 ? make_float4(__uint_as_float(ra[q]), __uint_as_float(ra[q + 1]), __uint_as_float(ra[q + 2]), __uint_as_float(ra[q + 3]))
                                     : make_float4(__uint_as_float(rb[q]), __uint_as_float(rb[q + 1]), __uint_as_float(rb[q + 2]), __uint_as_float(rb[q + 3]));
                    if (g.bias && n < g.K) {
                        const float4 bb = __ldg(reinterpret_cast<const float4*>(g.bias + n));
                        v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                    }
                    v.x = act_fn(v.x, g.act); v.y = act_fn(v.y, g.act); v.z = act_fn(v.z, g.act); v.w = act_fn(v.w, g.act);
                    asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(rowa + sw * 16u), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the TMA's reads
                __syncwarp();
                if (lane == 0 && oh < g.H && ow0 < g.W && nbase < g.K) {
                    tma_store_3d(&tmD, buf, nbase, ow0, oh);
                    tma_store_commit();
                }
            }
        }
        if (lane == 0) tma_store_wait_read();
        if (!ok && lane == 0) atomicExch(&g_device_status, (int)NNV_ERR_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0) stamp_end(g.stamp);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)g.tmem_cols) : "memory");
    }
}
