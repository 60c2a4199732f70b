// Single-operation entry points: the weights transformation and the execution of one layer.
#include "nnv_internal.h"

using namespace nnv;

namespace nnv {

// Where the one-kernel F(2x2,3x3) path is taken without being asked for (filled in from measurements).
static bool wino_fused_default(const nnv_layer_desc_t& L, const LayerGeom& g) {
    (void)L; (void)g;
    return false;
}

// host_src: d_raw is pinned host memory read in place (the zero-copy arm): the kernels then start loading
// before they wait for the previous kernel of their stream, which they do not depend on.
nnv_status_t do_transform(const nnv_plan& p, int layer, int v, int math, const void* d_raw, void* d_out,
                          cudaStream_t st, bool host_src) {
    const nnv_layer_desc_t& L = p.layers[layer];
    const LayerGeom& g = p.geom[layer];
    const bool bf16 = math == NNV_MATH_BF16;
    if (int m = wino_m(v)) return launch_filter_transform(m, bf16, (const float*)d_raw, d_out, L.K, L.C, g.Cp, st, host_src);
    if (v == NNV_VAR_IM2COL || v == NNV_VAR_GEMM1X1)
        return launch_pack(bf16, (const float*)d_raw, d_out, L.K, L.C, L.R * L.S, g.Qp, st, host_src);
    return fail(NNV_ERR_UNSUPPORTED, "variant %d reads raw weights and has no transform", v);
}

nnv_status_t do_exec(const nnv_plan& p, int layer, int v, int math, const void* d_in, const void* d_add,
                     const void* d_wt, const void* d_bias, void* d_out, void* d_ws, uint64_t ws_bytes,
                     cudaStream_t st) {
    const nnv_layer_desc_t& L = p.layers[layer];
    const LayerGeom& g = p.geom[layer];
    const bool bf16 = math == NNV_MATH_BF16;
    const uint64_t es = bf16 ? 2 : 4;
    const uint64_t need = exec_ws_bytes(p, layer, v, math);
    NNV_REQUIRE(ws_bytes >= need, NNV_ERR_WORKSPACE_TOO_SMALL, "layer %d needs %llu scratch bytes, got %llu", layer,
                (unsigned long long)need, (unsigned long long)ws_bytes);
    NNV_REQUIRE(need == 0 || (d_ws && aligned256(d_ws)), NNV_ERR_INVALID_ARG, "scratch pointer null or misaligned");
    const float* x = (const float*)d_in;
    const float* add = (const float*)d_add;
    const float* bias = (const float*)d_bias;
    float* y = (float*)d_out;

    if (v == NNV_VAR_DIRECT)
        return launch_direct(x, (const float*)d_wt, bias, add, y, L.act, L.C, L.H, L.W, L.K, L.R, L.S, L.stride, L.pad,
                             g.OH, g.OW, st);
    if (v == NNV_VAR_DEPTHWISE)
        return launch_depthwise(x, (const float*)d_wt, bias, add, y, L.act, L.C, L.H, L.W, L.R, L.S, L.stride, L.pad,
                                g.OH, g.OW, st);

    const SmallPPlan spp = small_p_plan(L, g, v, math);
    if (spp.use) return launch_gemm_sp(L, g, spp, x, (const float*)d_wt, bias, add, y, d_ws, st);

    GemmArgs a{};
    a.mode = bf16 ? GEMM_BF16 : GEMM_TF32;
    a.bias = bias; a.addend = add; a.act = L.act;
    a.D = y; a.ldd = L.K; a.strideD = (int64_t)g.P * L.K;
    a.N = L.K;

    if (wino_fused_applies(L, v, math)) {
        const int wf = tuning().winofused;
        if (wf == 1 || (wf < 0 && wino_fused_default(L, g)))
            return launch_wino_f2_fused(L, g, x, (const float*)d_wt, bias, add, y, st);
    }
    if (int m = wino_m(v)) {
        const int TH = ceil_div(g.OH, m), TW = ceil_div(g.OW, m), T = TH * TW, a2 = (m + 2) * (m + 2);
        uint8_t* ws = (uint8_t*)d_ws;
        void* V = ws;
        float* Mt = (float*)(ws + align_up((uint64_t)a2 * T * g.Cp * es, 256));
        // F(2,3) runs as one TF32 / BF16 pass; F(4,3) and F(6,3) amplify operand rounding too much for
        // that, so their tile GEMM multiplies fp32 operands with the compensated bf16 scheme.
        if (m != 2) a.mode = GEMM_X3;
        NNV_TRY(launch_wino_input(m, bf16, x, V, L.C, g.Cp, L.H, L.W, L.pad, TH, TW, st));
        a.A = V; a.B = d_wt; a.D = Mt;
        a.M = T; a.Kd = g.Cp; a.batch = a2;
        a.lda = g.Cp; a.ldb = g.Cp; a.ldd = L.K;
        a.strideA = (int64_t)T * g.Cp; a.strideB = (int64_t)L.K * g.Cp; a.strideD = (int64_t)T * L.K;
        a.bias = nullptr; a.addend = nullptr; a.act = 0;
        NNV_TRY(launch_gemm_tc(a, st));
        return launch_wino_output(m, Mt, y, bias, add, L.act, L.K, g.OH, g.OW, TH, TW, st);
    }

    // IM2COL and GEMM1X1: Y[P][K] = Xcol[P][Qp] * P[K][Qp]^T
    a.M = g.P; a.Kd = g.Qp; a.batch = 1;
    a.B = d_wt; a.ldb = g.Qp; a.strideB = (int64_t)L.K * g.Qp;
    const bool direct_operand = (v == NNV_VAR_GEMM1X1) && need == 0 && L.stride == 1;
    if ((direct_operand || need == 0) && bf16) a.mode = GEMM_BF16_CVT;   // fp32 activation rounded to bf16 inside the kernel
    if (direct_operand) {
        a.A = x; a.lda = L.C; a.Kd = L.C;                      // rows of X are the GEMM's rows
    } else if (need == 0) {
        // implicit GEMM: the TMA gathers the filter-window pixels from the activation itself
        a.A = x; a.lda = L.C;
        a.ic.on = 1; a.ic.C = L.C; a.ic.H = L.H; a.ic.W = L.W; a.ic.R = L.R; a.ic.S = L.S;
        a.ic.stride = L.stride; a.ic.pad = L.pad; a.ic.OW = g.OW;
    } else {
        NNV_TRY(launch_im2col(bf16, x, d_ws, L.C, L.H, L.W, L.R, L.S, L.stride, L.pad, g.OH, g.OW, g.Qp, st));
        a.A = d_ws; a.lda = g.Qp;
    }
    a.strideA = (int64_t)g.P * a.lda;
    return launch_gemm_tc(a, st);
}

nnv_status_t do_pool(const nnv_plan& p, int layer, const void* d_in, void* d_out, cudaStream_t st) {
    const nnv_layer_desc_t& L = p.layers[layer];
    const LayerGeom& g = p.geom[layer];
    if (L.op == NNV_OP_MAXPOOL)
        return launch_maxpool((const float*)d_in, (float*)d_out, L.C, L.H, L.W, L.R, L.stride, L.pad, g.OH, g.OW, st);
    if (L.op == NNV_OP_GAVGPOOL) return launch_gavgpool((const float*)d_in, (float*)d_out, L.C, L.H, L.W, st);
    return fail(NNV_ERR_INVALID_ARG, "layer %d is not a pooling layer", layer);
}

}  // namespace nnv

extern "C" {

nnv_status_t nnv_transform_weights(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math, const void* d_raw,
                                   void* d_out, void* stream) {
    NNV_REQUIRE(p && d_raw && d_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    NNV_REQUIRE(aligned256(d_raw) && aligned256(d_out), NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    return do_transform(*p, layer, v, math, d_raw, d_out, (cudaStream_t)stream, false);
}

nnv_status_t nnv_transformed_layout(const nnv_plan_t* p, const nnv_choice_t* choices, uint64_t* offsets, uint64_t* total) {
    NNV_REQUIRE(p && choices && offsets && total, NNV_ERR_INVALID_ARG, "null argument");
    uint64_t pos = 0;
    for (int i = 0; i < (int)p->layers.size(); ++i) {
        offsets[i] = 0;
        if (p->layers[i].op != NNV_OP_CONV) continue;
        NNV_TRY(check_choice(*p, i, choices[i].variant, choices[i].math));
        if (!variant_has_transform(choices[i].variant)) continue;
        offsets[i] = pos;
        pos += align_up(transformed_bytes(*p, i, choices[i].variant, choices[i].math), 256);
    }
    *total = pos;
    return NNV_OK;
}

nnv_status_t nnv_transform_all(const nnv_plan_t* p, const nnv_choice_t* choices, const void* d_weights, uint64_t w_bytes,
                               void* d_out, uint64_t out_bytes, void* stream) {
    NNV_REQUIRE(p && choices && d_weights && d_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(aligned256(d_weights) && aligned256(d_out), NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    const int n = (int)p->layers.size();
    std::vector<uint64_t> offs(n);
    uint64_t total = 0;
    NNV_TRY(nnv_transformed_layout(p, choices, offs.data(), &total));
    NNV_REQUIRE(out_bytes >= total, NNV_ERR_WORKSPACE_TOO_SMALL, "output needs %llu bytes, got %llu",
                (unsigned long long)total, (unsigned long long)out_bytes);
    std::vector<XformDesc> descs;
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p->layers[i];
        if (L.op != NNV_OP_CONV || !variant_has_transform(choices[i].variant)) continue;
        NNV_REQUIRE(L.w_off + raw_weight_bytes(L) <= w_bytes, NNV_ERR_INVALID_ARG, "layer %d: weights lie outside the weight blob", i);
        XformDesc d{};
        d.src = (const uint8_t*)d_weights + L.w_off;
        d.dst = (uint8_t*)d_out + offs[i];
        d.K = L.K; d.C = L.C; d.Cp = p->geom[i].Cp; d.RS = L.R * L.S; d.Qp = p->geom[i].Qp;
        d.bf16 = choices[i].math == NNV_MATH_BF16;
        const int m = wino_m(choices[i].variant);
        d.kind = m == 2 ? XF_WINO2 : m == 4 ? XF_WINO4 : m == 6 ? XF_WINO6 : (d.RS == 1 ? XF_PACK1X1 : XF_PACK);
        descs.push_back(d);
    }
    if (descs.empty()) return NNV_OK;
    return launch_transform_batch(descs.data(), (int)descs.size(), (cudaStream_t)stream);
}

nnv_status_t nnv_conv_exec(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math, const void* d_in,
                           const void* d_addend, const void* d_wt, const void* d_bias, void* d_out, void* d_ws,
                           uint64_t ws_bytes, void* stream) {
    NNV_REQUIRE(p && d_in && d_wt && d_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    NNV_REQUIRE(aligned256(d_in) && aligned256(d_wt) && aligned256(d_out) && (!d_addend || aligned256(d_addend)) &&
                    (!d_bias || aligned256(d_bias)),
                NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    NNV_REQUIRE(!p->layers[layer].has_bias || d_bias, NNV_ERR_INVALID_ARG, "layer %d has a bias but d_bias is null", layer);
    return do_exec(*p, layer, v, math, d_in, d_addend, d_wt, d_bias, d_out, d_ws, ws_bytes, (cudaStream_t)stream);
}

nnv_status_t nnv_wino_sizes(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math, int32_t* tiles, uint64_t* v_bytes,
                            uint64_t* m_bytes) {
    NNV_REQUIRE(p, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    const int m = wino_m(v);
    NNV_REQUIRE(m, NNV_ERR_INVALID_ARG, "variant %d is not a Winograd variant", v);
    const LayerGeom& g = p->geom[layer];
    const uint64_t T = (uint64_t)ceil_div(g.OH, m) * ceil_div(g.OW, m), a2 = (uint64_t)(m + 2) * (m + 2);
    if (tiles) *tiles = (int32_t)T;
    if (v_bytes) *v_bytes = a2 * T * g.Cp * (math == NNV_MATH_BF16 ? 2 : 4);
    if (m_bytes) *m_bytes = a2 * T * p->layers[layer].K * 4;
    return NNV_OK;
}

nnv_status_t nnv_wino_input_transform(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math, const void* d_in, void* d_V,
                                      void* stream) {
    NNV_REQUIRE(p && d_in && d_V, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    const int m = wino_m(v);
    NNV_REQUIRE(m, NNV_ERR_INVALID_ARG, "variant %d is not a Winograd variant", v);
    NNV_REQUIRE(aligned256(d_in) && aligned256(d_V), NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    const nnv_layer_desc_t& L = p->layers[layer];
    const LayerGeom& g = p->geom[layer];
    return launch_wino_input(m, math == NNV_MATH_BF16, (const float*)d_in, d_V, L.C, g.Cp, L.H, L.W, L.pad, ceil_div(g.OH, m),
                             ceil_div(g.OW, m), (cudaStream_t)stream);
}

nnv_status_t nnv_wino_output_transform(const nnv_plan_t* p, int32_t layer, int32_t v, const void* d_M, const void* d_addend,
                                       const void* d_bias, void* d_out, void* stream) {
    NNV_REQUIRE(p && d_M && d_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, NNV_MATH_TF32));
    const int m = wino_m(v);
    NNV_REQUIRE(m, NNV_ERR_INVALID_ARG, "variant %d is not a Winograd variant", v);
    NNV_REQUIRE(aligned256(d_M) && aligned256(d_out) && (!d_addend || aligned256(d_addend)) && (!d_bias || aligned256(d_bias)),
                NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    const nnv_layer_desc_t& L = p->layers[layer];
    const LayerGeom& g = p->geom[layer];
    NNV_REQUIRE(!L.has_bias || d_bias, NNV_ERR_INVALID_ARG, "layer %d has a bias but d_bias is null", layer);
    return launch_wino_output(m, (const float*)d_M, (float*)d_out, (const float*)d_bias, (const float*)d_addend, L.act, L.K, g.OH,
                              g.OW, ceil_div(g.OH, m), ceil_div(g.OW, m), (cudaStream_t)stream);
}

nnv_status_t nnv_pool_exec(const nnv_plan_t* p, int32_t layer, const void* d_in, void* d_out, void* stream) {
    NNV_REQUIRE(p && d_in && d_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(layer >= 0 && layer < (int)p->layers.size(), NNV_ERR_INVALID_ARG, "layer %d out of range", layer);
    NNV_REQUIRE(aligned256(d_in) && aligned256(d_out), NNV_ERR_INVALID_ARG, "device pointers must be 256-byte aligned");
    return do_pool(*p, layer, d_in, d_out, (cudaStream_t)stream);
}

nnv_status_t nnv_chw_to_hwc(const float* d_in, float* d_out, int32_t C, int32_t H, int32_t W, void* stream) {
    NNV_REQUIRE(d_in && d_out && C > 0 && H > 0 && W > 0, NNV_ERR_INVALID_ARG, "bad argument");
    return launch_chw_to_hwc(d_in, d_out, C, H, W, (cudaStream_t)stream);
}
nnv_status_t nnv_hwc_to_chw(const float* d_in, float* d_out, int32_t C, int32_t H, int32_t W, void* stream) {
    NNV_REQUIRE(d_in && d_out && C > 0 && H > 0 && W > 0, NNV_ERR_INVALID_ARG, "bad argument");
    return launch_hwc_to_chw(d_in, d_out, C, H, W, (cudaStream_t)stream);
}

nnv_status_t nnv_device_status(int32_t* code) {
    NNV_REQUIRE(code, NNV_ERR_INVALID_ARG, "null argument");
    return read_device_status(code);
}

}  // extern "C"
