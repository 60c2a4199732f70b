// Host-side plan logic: validation, eligibility, size queries, arena layout and the
// integer cold-cost selection.  No device work happens in this file.
#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "nnv_internal.h"

namespace nnv {

static thread_local char g_err[512] = "";

nnv_status_t fail(nnv_status_t code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

static std::mutex g_tuning_mu;
static Tuning g_tuning;

Tuning tuning() {
    std::lock_guard<std::mutex> lk(g_tuning_mu);
    return g_tuning;
}

// "key=value;key=value" -> *t.  Returns the offending item on a parse / range error, else nullptr.
static const char* parse_tuning(const char* spec, Tuning* t, char* item, size_t item_cap) {
    const char* s = spec;
    while (*s) {
        const char* e = std::strchr(s, ';');
        const size_t len = e ? (size_t)(e - s) : std::strlen(s);
        if (len >= item_cap) return "item too long";
        std::memcpy(item, s, len);
        item[len] = 0;
        s += len + (e ? 1 : 0);
        if (len == 0) continue;
        char* eq = std::strchr(item, '=');
        if (!eq) return item;
        *eq = 0;
        const char* key = item;
        const char* val = eq + 1;
        int a = 0, b = 0, c = 0, d = 0, f = 0;
        auto flag = [&](int* dst) { return std::sscanf(val, "%d", &a) == 1 && (a == 0 || a == 1) ? (*dst = a, true) : false; };
        bool ok = false;
        if (!std::strcmp(key, "gemm_tile")) {
            ok = std::sscanf(val, "%d,%d", &a, &b) == 2 && a >= 16 && a <= 128 && a % 16 == 0 && b >= 1 && b <= 8 && (b & (b - 1)) == 0;
            if (ok) { t->gemm_bn = a; t->gemm_splits = b; }
        } else if (!std::strcmp(key, "gemm_ring")) {
            ok = std::sscanf(val, "%d", &a) == 1 && a >= 2 && a <= 8;
            if (ok) t->gemm_ring = a;
        } else if (!std::strcmp(key, "gemm_prefill")) {
            ok = flag(&t->gemm_prefill);
        } else if (!std::strcmp(key, "conv3x3")) {
            if (!std::strcmp(val, "off")) { t->conv3x3 = 1; ok = true; }
            else if (!std::strcmp(val, "auto")) { t->conv3x3 = 0; ok = true; }
            else {
                const int got = std::sscanf(val, "%d,%d,%d,%d,%d", &a, &b, &c, &d, &f);
                ok = got >= 3 && (a == 1 || a == 2) && b >= 16 && b <= 128 && b % 16 == 0 && c >= 1 && c <= 8 && (c & (c - 1)) == 0 &&
                     (got < 4 || (d >= 0 && d <= 4)) && (got < 5 || (f >= 0 && f <= 8));
                if (ok) { t->conv3x3 = 2; t->conv_mt = a; t->conv_bn = b; t->conv_splits = c; t->conv_na = got >= 4 ? d : 0; t->conv_nb = got >= 5 ? f : 0; }
            }
        } else if (!std::strcmp(key, "conv3x3p")) {
            if (!std::strcmp(val, "off")) { t->convp = 1; ok = true; }
            else if (!std::strcmp(val, "auto")) { t->convp = 0; ok = true; }
            else {
                const int got = std::sscanf(val, "%d,%d,%d,%d", &a, &b, &c, &d);
                ok = got >= 2 && a >= 16 && a <= 128 && a % 16 == 0 && b >= 1 && b <= 4 && (got < 3 || (c >= 1 && c <= 4)) && (got < 4 || (d >= 1 && d <= 8));
                if (ok) { t->convp = 2; t->convp_bn = a; t->convp_per_sm = b; t->convp_na = got >= 3 ? c : 0; t->convp_nb = got >= 4 ? d : 0; }
            }
        } else if (!std::strcmp(key, "conv3x3w")) {
            if (!std::strcmp(val, "off")) { t->convw = 1; ok = true; }
            else if (!std::strcmp(val, "auto")) { t->convw = 0; ok = true; }
            else if (!std::strcmp(val, "on")) { t->convw = 2; ok = true; }
        } else if (!std::strcmp(key, "winofused")) {
            if (!std::strcmp(val, "auto")) { t->winofused = -1; ok = true; }
            else ok = flag(&t->winofused);
        } else if (!std::strcmp(key, "bf16cvt")) {
            ok = flag(&t->bf16cvt);
        } else if (!std::strcmp(key, "smallp")) {
            if (std::sscanf(val, "%d", &a) == 1 && a >= 0 && a <= 148) { t->smallp = a ? 1 : 0; t->smallp_splits = a > 1 ? a : 0; ok = true; }
        } else if (!std::strcmp(key, "side")) {
            ok = flag(&t->side);
        } else if (!std::strcmp(key, "merge")) {
            ok = flag(&t->merge);
        } else if (!std::strcmp(key, "group")) {
            ok = flag(&t->group);
        } else if (!std::strcmp(key, "copies_first")) {
            ok = flag(&t->copies_first);
        } else if (!std::strcmp(key, "chunk")) {
            ok = std::sscanf(val, "%d,%d", &a, &b) == 2 && a >= 16 && b >= a && b <= (1 << 20);
            if (ok) { t->chunk_first_kb = a; t->chunk_max_kb = b; }
        }
        if (!ok) { *eq = '='; return item; }
    }
    return nullptr;
}

bool variant_has_transform(int v) { return v != NNV_VAR_DIRECT && v != NNV_VAR_DEPTHWISE; }

bool math_valid_for(int v, int math) {
    if (v == NNV_VAR_DIRECT || v == NNV_VAR_DEPTHWISE) return math == NNV_MATH_FP32;
    // One bf16 pass in the F(4,3) / F(6,3) Winograd domain misses the 1e-2 output tolerance
    // (measured 2.6e-2 / 4.9e-2 relative L2), so these variants exist in the TF32 accuracy class only.
    if (v == NNV_VAR_WINO_F4 || v == NNV_VAR_WINO_F6) return math == NNV_MATH_TF32;
    return math == NNV_MATH_TF32 || math == NNV_MATH_BF16;
}

int wino_m(int v) {
    switch (v) {
        case NNV_VAR_WINO_F2: return 2;
        case NNV_VAR_WINO_F4: return 4;
        case NNV_VAR_WINO_F6: return 6;
        default: return 0;
    }
}

// Eligibility is keyed on filter size, stride and grouping only (the surviving keys of the
// paper's Figure 5 kernel tree); ragged channel counts are handled by padding, so there is no
// divisibility requirement.
bool is_eligible(const nnv_layer_desc_t& L, int v) {
    if (L.op != NNV_OP_CONV) return false;
    const bool dense = L.groups == 1;
    switch (v) {
        case NNV_VAR_DIRECT: return dense;
        case NNV_VAR_IM2COL: return dense;
        case NNV_VAR_GEMM1X1: return dense && L.R == 1 && L.S == 1 && L.pad == 0;
        case NNV_VAR_DEPTHWISE: return L.groups > 1 && L.groups == L.C && L.C == L.K;
        case NNV_VAR_WINO_F2:
        case NNV_VAR_WINO_F4:
        case NNV_VAR_WINO_F6: return dense && L.R == 3 && L.S == 3 && L.stride == 1;
        default: return false;
    }
}

uint64_t raw_weight_bytes(const nnv_layer_desc_t& L) {
    if (L.op != NNV_OP_CONV) return 0;
    return 4ull * L.K * (L.C / L.groups) * L.R * L.S;
}

uint64_t transformed_bytes(const nnv_plan& p, int layer, int v, int math) {
    const nnv_layer_desc_t& L = p.layers[layer];
    const LayerGeom& g = p.geom[layer];
    const uint64_t es = (math == NNV_MATH_BF16) ? 2 : 4;
    if (int m = wino_m(v)) {
        const uint64_t a = m + 2;
        return a * a * (uint64_t)L.K * g.Cp * es;
    }
    if (v == NNV_VAR_IM2COL || v == NNV_VAR_GEMM1X1) return (uint64_t)L.K * g.Qp * es;
    return 0;
}

static inline bool gemm1x1_direct_operand(const nnv_layer_desc_t& L, int math) {
    // The activation itself can be the GEMM's A operand when no subsampling, padding or
    // conversion is needed: stride 1, fp32 words (TF32), rows a multiple of 16 bytes.
    // BF16 math: the kernel rounds the fp32 rows to bf16 on their way through shared memory (C % 8: 16-byte weight chunks).
    return L.stride == 1 && ((math == NNV_MATH_TF32 && (L.C % 4) == 0) || (math == NNV_MATH_BF16 && (L.C % 8) == 0 && tuning().bf16cvt));
}

static inline bool implicit_gemm_operand(const nnv_layer_desc_t& L, int math) {
    // The TMA's im2col mode gathers filter-window pixels straight from the NHWC activation, so no
    // Xcol matrix is materialised: fp32 words (TF32), pixel rows a multiple of 16 bytes, and an
    // activation of at least 128 KiB (smaller tensors take the explicit path).
    return ((math == NNV_MATH_TF32 && (L.C % 4) == 0) || (math == NNV_MATH_BF16 && (L.C % 8) == 0 && tuning().bf16cvt)) &&
           4ull * L.C * L.H * L.W >= 131072ull && L.R <= 16 && L.S <= 16 && L.pad <= 8;
}

bool wino_fused_applies(const nnv_layer_desc_t& L, int v, int math) {
    return v == NNV_VAR_WINO_F2 && math == NNV_MATH_TF32 && L.groups == 1 && L.R == 3 && L.S == 3 && L.stride == 1 &&
           (L.C % 8) == 0 && (L.K % 8) == 0;
}

SmallPPlan small_p_plan(const nnv_layer_desc_t& L, const LayerGeom& g, int v, int math) {
    SmallPPlan sp{};
    const Tuning tn = tuning();
    if (!tn.smallp || (v != NNV_VAR_IM2COL && v != NNV_VAR_GEMM1X1) || math != NNV_MATH_TF32 || L.groups != 1 || L.stride != 1 ||
        L.R != L.S || (L.R & 1) == 0 || L.pad != (L.R - 1) / 2 || L.H * L.W > 256 || (L.C % 32) != 0 || (L.K % 4) != 0)
        return sp;
    // Measured on B200 (L2 flushed, weights cold): on 7 x 7 grids this kernel takes 0.55 - 0.9 of the pixel-on-rows
    // GEMM's time (512 -> 512 3x3: 9.2 against 15.9 us; 960 -> 160 1x1: 6.9 against 48 us), on 14 x 14 grids the two
    // are level or the other is ahead (its two row tiles are 77 % full there); so, unless forced, up to 64 pixels.
    if (L.H * L.W > 64 && !tn.smallp_splits) return sp;
    sp.Npad = ceil_div(g.P, 16) * 16;
    sp.b_slot_bytes = (uint32_t)align_up((uint64_t)sp.Npad * 128, 1024);
    const double stage = 16384.0 + sp.b_slot_bytes;
    sp.nkb = L.R * L.S * (L.C / 32);
    const int m_tiles = ceil_div(L.K, 128);
    const int s_max = std::min(sp.nkb, std::max(1, 148 / m_tiles));
    // microseconds: fixed cost + K blocks per CTA at ~70 GB/s of shared-memory fill per SM + (split) the second
    // kernel and the partial tiles' trip through L2.  Refit on sweeps of the split count (L2 flushed): 512 -> 2048 1x1 @7
    // takes 7.8 / 6.7 / 6.3 / 6.1 / 6.5 us with 1 / 2 / 3 / 6 / 9 splits, 2048 -> 512 1x1 @7 14.5 / 10.6 / 8.2 / 7.9 / 8.3 us
    // with 2 / 4 / 8 / 16 / 37, 512 -> 512 3x3 @7 11.7 / 9.6 / 9.7 us with 8 / 18 / 37.
    double best = 1e30;
    for (int s = 1; s <= s_max; ++s) {
        const double t = 2.0 + ceil_div(sp.nkb, s) * stage / 69e3 + (s > 1 ? 1.6 + 2.5 * s * g.P * L.K * 4.0 / 4e6 : 0.0);
        if (t < best - 1e-9) { best = t; sp.splits = s; }
    }
    if (tn.smallp_splits && tn.smallp_splits <= sp.nkb) sp.splits = tn.smallp_splits;
    sp.stages = std::max(1, std::min({8, ceil_div(sp.nkb, sp.splits), (int)(200.0 * 1024.0 / stage)}));
    sp.ws_bytes = sp.splits > 1 ? align_up((uint64_t)sp.splits * g.P * L.K * 4, 256) : 0;
    sp.use = true;
    return sp;
}

uint64_t exec_ws_bytes(const nnv_plan& p, int layer, int v, int math) {
    const nnv_layer_desc_t& L = p.layers[layer];
    const LayerGeom& g = p.geom[layer];
    const uint64_t es = (math == NNV_MATH_BF16) ? 2 : 4;
    const SmallPPlan spp = small_p_plan(L, g, v, math);
    if (spp.use) return spp.ws_bytes;
    if (int m = wino_m(v)) {
        const uint64_t a2 = (uint64_t)(m + 2) * (m + 2);
        const uint64_t T = (uint64_t)ceil_div(g.OH, m) * ceil_div(g.OW, m);
        return align_up(a2 * T * g.Cp * es, 256) + align_up(a2 * T * L.K * 4, 256);
    }
    if (v == NNV_VAR_IM2COL) return implicit_gemm_operand(L, math) ? 0 : align_up((uint64_t)g.P * g.Qp * es, 256);
    if (v == NNV_VAR_GEMM1X1)
        return (gemm1x1_direct_operand(L, math) || implicit_gemm_operand(L, math)) ? 0
                                                                                  : align_up((uint64_t)g.P * g.Qp * es, 256);
    return 0;
}

uint64_t exec_flops(const nnv_plan& p, int layer, int v) {
    const nnv_layer_desc_t& L = p.layers[layer];
    const LayerGeom& g = p.geom[layer];
    if (int m = wino_m(v)) {
        const uint64_t a2 = (uint64_t)(m + 2) * (m + 2);
        const uint64_t T = (uint64_t)ceil_div(g.OH, m) * ceil_div(g.OW, m);
        return 2ull * a2 * T * L.K * L.C;
    }
    return 2ull * g.P * L.K * g.Cg * L.R * L.S;
}

nnv_status_t check_choice(const nnv_plan& p, int layer, int v, int math) {
    NNV_REQUIRE(layer >= 0 && layer < (int)p.layers.size(), NNV_ERR_INVALID_ARG, "layer %d out of range", layer);
    NNV_REQUIRE(p.layers[layer].op == NNV_OP_CONV, NNV_ERR_INVALID_ARG, "layer %d is not a convolution", layer);
    NNV_REQUIRE(v >= 0 && v < NNV_NUM_VARIANTS, NNV_ERR_INVALID_ARG, "variant %d is not a variant", v);
    NNV_REQUIRE(is_eligible(p.layers[layer], v), NNV_ERR_UNSUPPORTED, "variant %d cannot run layer %d", v, layer);
    NNV_REQUIRE(math_valid_for(v, math), NNV_ERR_UNSUPPORTED, "math mode %d does not exist for variant %d", math, v);
    return NNV_OK;
}

nnv_status_t layout_arena(const nnv_plan& p, const nnv_choice_t* choices, int depth, ArenaLayout* out) {
    const int n = (int)p.layers.size();
    ArenaLayout a;
    uint64_t pos = 0;
    auto take = [&](uint64_t bytes) {
        uint64_t off = pos;
        pos += align_up(bytes ? bytes : 1, 1024);
        return off;
    };
    const nnv_layer_desc_t& L0 = p.layers[0];
    const uint64_t in_bytes = 4ull * L0.C * L0.H * L0.W;
    a.in_chw = take(in_bytes);
    a.in_hwc = take(in_bytes);
    a.act_off.resize(n);
    uint64_t max_raw = 0, max_bias = 0, max_xf = 0, max_ws = 0;
    for (int i = 0; i < n; ++i) {
        const nnv_layer_desc_t& L = p.layers[i];
        const LayerGeom& g = p.geom[i];
        a.act_off[i] = take(4ull * g.P * L.K);
        if (L.op != NNV_OP_CONV) continue;
        NNV_TRY(check_choice(p, i, choices[i].variant, choices[i].math));
        max_raw = std::max(max_raw, raw_weight_bytes(L));
        max_bias = std::max<uint64_t>(max_bias, 4ull * L.K);
        max_xf = std::max(max_xf, transformed_bytes(p, i, choices[i].variant, choices[i].math));
        max_ws = std::max(max_ws, exec_ws_bytes(p, i, choices[i].variant, choices[i].math));
    }
    const nnv_layer_desc_t& Ln = p.layers[n - 1];
    a.out_chw = take(4ull * p.geom[n - 1].P * Ln.K);
    if (depth == 0) {
        // no staging limit: every conv layer owns a raw (weights + bias) and a transformed buffer
        // The raw buffers mirror the host weight blob (same distances between layers) and the
        // transformed buffers of layers read from the cached blob mirror that blob, so that one copy can
        // serve several consecutive layers.
        a.raw_off.assign(n, 0); a.bias_off.assign(n, 0); a.xf_off.assign(n, 0);
        uint64_t lo = ~0ull, hi = 0;
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p.layers[i];
            if (L.op != NNV_OP_CONV) continue;
            lo = std::min<uint64_t>(lo, L.w_off); hi = std::max<uint64_t>(hi, L.w_off + raw_weight_bytes(L));
            if (L.has_bias) { lo = std::min<uint64_t>(lo, L.b_off); hi = std::max<uint64_t>(hi, L.b_off + 4ull * L.K); }
        }
        if (lo > hi) lo = hi = 0;
        const uint64_t raw_region = take(hi - lo);
        std::vector<uint64_t> coff(n, 0);
        uint64_t ctotal = 0;
        NNV_TRY(nnv_cached_layout(&p, choices, coff.data(), &ctotal));
        const uint64_t cached_region = take(ctotal);
        for (int i = 0; i < n; ++i) {
            const nnv_layer_desc_t& L = p.layers[i];
            if (L.op != NNV_OP_CONV) continue;
            a.raw_off[i] = raw_region + (L.w_off - lo);
            a.bias_off[i] = L.has_bias ? raw_region + (L.b_off - lo) : raw_region;
            const bool cached = variant_has_transform(choices[i].variant) && choices[i].cached == NNV_ARM_CACHED;
            a.xf_off[i] = cached ? cached_region + coff[i] : take(transformed_bytes(p, i, choices[i].variant, choices[i].math));
        }
    } else {
        a.raw_bias_off = align_up(max_raw ? max_raw : 1, 1024);
        a.raw_slot_bytes = a.raw_bias_off + align_up(max_bias ? max_bias : 1, 1024);
        a.raw_slot0 = take(a.raw_slot_bytes * depth);
        a.xf_slot_bytes = align_up(max_xf ? max_xf : 1, 1024);
        a.xf_slot0 = take(a.xf_slot_bytes * depth);
    }
    a.ws_bytes = align_up(max_ws ? max_ws : 1, 1024);
    a.ws_off = take(a.ws_bytes);
    a.total = pos;
    *out = a;
    return NNV_OK;
}

// ---- selection ------------------------------------------------------------------------------
static inline bool rank_less(const Option& a, const Option& b) {
    if (a.variant != b.variant) return a.variant < b.variant;
    if (a.math != b.math) return a.math < b.math;
    return a.cached < b.cached;
}

nnv_status_t gather_options(const nnv_plan& p, int layer, const nnv_cost_t* costs, int n_costs,
                                   int allow_cached, std::vector<Option>* opts) {
    for (int i = 0; i < n_costs; ++i) {
        const nnv_cost_t& c = costs[i];
        if (c.layer != layer) continue;
        NNV_REQUIRE(c.variant >= 0 && c.variant < NNV_NUM_VARIANTS && is_eligible(p.layers[layer], c.variant) &&
                        math_valid_for(c.variant, c.math),
                    NNV_ERR_INVALID_ARG, "cost row %d names a kernel layer %d cannot use", i, layer);
        opts->push_back({c.variant, c.math, 0, c.h2d_raw_ns + c.xform_ns, c.exec_ns});
        if ((allow_cached & 1) && variant_has_transform(c.variant))
            opts->push_back({c.variant, c.math, NNV_ARM_CACHED, c.h2d_cached_ns, c.exec_ns});
        if ((allow_cached & 2) && variant_has_transform(c.variant) && c.zc_ns > 0)
            opts->push_back({c.variant, c.math, NNV_ARM_ZERO_COPY, c.zc_ns, c.exec_ns});
    }
    return NNV_OK;
}

void pareto(const std::vector<Option>& in, std::vector<Option>* out) {
    for (size_t i = 0; i < in.size(); ++i) {
        const Option& o = in[i];
        bool drop = false;
        for (size_t j = 0; j < in.size() && !drop; ++j) {
            if (j == i) continue;
            const Option& q = in[j];
            if (q.prep <= o.prep && q.exec <= o.exec) {
                if (q.prep < o.prep || q.exec < o.exec) drop = true;
                else if (rank_less(q, o)) drop = true;          // exact duplicate, lower rank wins
            }
        }
        if (!drop) out->push_back(o);
    }
    std::sort(out->begin(), out->end(), rank_less);
}

}  // namespace nnv

using namespace nnv;

extern "C" {

const char* nnv_last_error(void) { return g_err; }
int32_t nnv_version(void) { return 100; }

nnv_status_t nnv_tuning_set(const char* spec) {
    Tuning t;                                                   // every call starts from the defaults
    char item[128];
    if (spec && *spec) {
        const char* bad = parse_tuning(spec, &t, item, sizeof(item));
        NNV_REQUIRE(!bad, NNV_ERR_INVALID_ARG, "tuning item not understood or out of range: %s", bad);
    }
    std::lock_guard<std::mutex> lk(g_tuning_mu);
    t.generation = g_tuning.generation + 1;
    g_tuning = t;
    return NNV_OK;
}

nnv_status_t nnv_plan_create(const nnv_layer_desc_t* layers, int32_t n, const nnv_plan_opts_t* opts,
                             nnv_plan_t** out) {
    NNV_REQUIRE(layers && out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(n > 0 && n <= 4096, NNV_ERR_INVALID_ARG, "layer count %d out of range", n);
    nnv_plan* p = new (std::nothrow) nnv_plan();
    NNV_REQUIRE(p, NNV_ERR_STATE, "out of host memory");
    p->layers.assign(layers, layers + n);
    p->geom.resize(n);
    p->opts = nnv_plan_opts_t{NNV_MATH_TF32, 1, 4, 0, 1};
    if (opts) {
        p->opts = *opts;
        if (p->opts.max_depth <= 0) p->opts.max_depth = 4;
    }
    nnv_status_t st = NNV_OK;
    for (int i = 0; i < n && st == NNV_OK; ++i) {
        const nnv_layer_desc_t& L = p->layers[i];
        LayerGeom& g = p->geom[i];
        auto bad = [&](const char* what) { st = fail(NNV_ERR_INVALID_ARG, "layer %d: %s", i, what); };
        if (L.op < NNV_OP_CONV || L.op > NNV_OP_GAVGPOOL) { bad("unknown op"); break; }
        if (L.C <= 0 || L.K <= 0 || L.H <= 0 || L.W <= 0 || L.R <= 0 || L.S <= 0 || L.stride <= 0 || L.pad < 0 ||
            L.groups <= 0) { bad("non-positive dimension"); break; }
        if ((int64_t)L.C * L.H * L.W > (1ll << 30)) { bad("activation too large"); break; }
        if (L.in0 < -1 || L.in0 >= i || L.in1 < -1 || L.in1 >= i) { bad("producer index must be -1 or an earlier layer"); break; }
        if (L.act < 0 || L.act > 2) { bad("unknown activation"); break; }
        if (L.op == NNV_OP_GAVGPOOL) {
            g.OH = g.OW = 1;
        } else {
            if (L.H + 2 * L.pad < L.R || L.W + 2 * L.pad < L.S) { bad("window larger than padded input"); break; }
            g.OH = (L.H + 2 * L.pad - L.R) / L.stride + 1;
            g.OW = (L.W + 2 * L.pad - L.S) / L.stride + 1;
        }
        g.P = g.OH * g.OW;
        if (L.op != NNV_OP_CONV) {
            if (L.K != L.C) { bad("pool layers keep the channel count"); break; }
            if (L.op == NNV_OP_MAXPOOL && L.pad >= L.R) { bad("max-pool padding must be smaller than its window"); break; }
            g.Cg = L.C; g.Q = g.Qp = 0; g.Cp = L.C;
        } else {
            if (L.C % L.groups || L.K % L.groups) { bad("channels not divisible by groups"); break; }
            if ((L.w_off & 255) || (L.has_bias && (L.b_off & 255))) { bad("weight / bias offsets must be 256-byte aligned"); break; }
            g.Cg = L.C / L.groups;
            g.Q = L.R * L.S * g.Cg;
            g.Qp = (g.Q + 7) / 8 * 8;
            g.Cp = (L.C + 7) / 8 * 8;
            bool any = false;
            for (int v = 0; v < NNV_NUM_VARIANTS; ++v) any = any || is_eligible(L, v);
            if (!any) { st = fail(NNV_ERR_UNSUPPORTED, "layer %d: no kernel variant supports this grouping", i); break; }
        }
        // shape agreement with the producers
        const int src = L.in0;
        if (src >= 0) {
            const nnv_layer_desc_t& S = p->layers[src];
            if (S.K != L.C || p->geom[src].OH != L.H || p->geom[src].OW != L.W) { bad("input shape differs from its producer's output"); break; }
        } else if (i != 0 && (L.C != p->layers[0].C || L.H != p->layers[0].H || L.W != p->layers[0].W)) {
            bad("layers reading the model input must share its shape"); break;
        }
        if (L.in1 >= 0) {
            const nnv_layer_desc_t& A = p->layers[L.in1];
            if (L.op != NNV_OP_CONV || A.K != L.K || p->geom[L.in1].OH != g.OH || p->geom[L.in1].OW != g.OW) { bad("residual addend shape differs from the output"); break; }
        }
    }
    if (st == NNV_OK && p->layers[0].in0 != -1) st = fail(NNV_ERR_INVALID_ARG, "layer 0 must read the model input");
    if (st != NNV_OK) { delete p; return st; }
    *out = p;
    return NNV_OK;
}

nnv_status_t nnv_plan_destroy(nnv_plan_t* p) {
    if (!p) return NNV_OK;
    if (p->warm_pending)                                       // reads / transforms of K_warm - K_cold may still be queued
        for (cudaEvent_t e : p->warm_ev)
            if (e) cudaEventSynchronize(e);
    for (cudaEvent_t e : p->ev) cudaEventDestroy(e);
    for (cudaEvent_t e : p->tev) cudaEventDestroy(e);
    for (cudaEvent_t e : p->warm_ev)
        if (e) cudaEventDestroy(e);
    if (p->h_status) cudaFreeHost(p->h_status);
    if (p->s_side) cudaStreamDestroy(p->s_side);
    for (nnv::CachedGraph& g : p->graphs)
        if (g.exec) cudaGraphExecDestroy(g.exec);
    delete p;
    return NNV_OK;
}

nnv_status_t nnv_eligible(const nnv_plan_t* p, int32_t layer, int32_t* out, int32_t cap, int32_t* n_out) {
    NNV_REQUIRE(p && out && n_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(layer >= 0 && layer < (int)p->layers.size(), NNV_ERR_INVALID_ARG, "layer %d out of range", layer);
    int cnt = 0;
    for (int v = 0; v < NNV_NUM_VARIANTS; ++v) {
        if (!is_eligible(p->layers[layer], v)) continue;
        NNV_REQUIRE(cnt < cap, NNV_ERR_INVALID_ARG, "output capacity %d too small", cap);
        out[cnt++] = v;
    }
    *n_out = cnt;
    return NNV_OK;
}

nnv_status_t nnv_transformed_bytes(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math, uint64_t* bytes) {
    NNV_REQUIRE(p && bytes, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    *bytes = transformed_bytes(*p, layer, v, math);
    return NNV_OK;
}

nnv_status_t nnv_exec_workspace_bytes(const nnv_plan_t* p, int32_t layer, int32_t v, int32_t math, uint64_t* bytes) {
    NNV_REQUIRE(p && bytes, NNV_ERR_INVALID_ARG, "null argument");
    NNV_TRY(check_choice(*p, layer, v, math));
    *bytes = exec_ws_bytes(*p, layer, v, math);
    return NNV_OK;
}

nnv_status_t nnv_arena_bytes(const nnv_plan_t* p, const nnv_choice_t* choices, int32_t depth, uint64_t* bytes) {
    NNV_REQUIRE(p && choices && bytes, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(depth >= 0 && depth <= p->opts.max_depth, NNV_ERR_INVALID_ARG, "depth %d outside 0..%d", depth, p->opts.max_depth);
    ArenaLayout a;
    NNV_TRY(layout_arena(*p, choices, depth, &a));
    *bytes = a.total;
    return NNV_OK;
}

nnv_status_t nnv_cached_layout(const nnv_plan_t* p, const nnv_choice_t* choices, uint64_t* offsets, uint64_t* total) {
    NNV_REQUIRE(p && choices && offsets && total, NNV_ERR_INVALID_ARG, "null argument");
    uint64_t pos = 0;
    for (int i = 0; i < (int)p->layers.size(); ++i) {
        offsets[i] = 0;
        if (p->layers[i].op != NNV_OP_CONV) continue;
        NNV_TRY(check_choice(*p, i, choices[i].variant, choices[i].math));
        NNV_REQUIRE(choices[i].cached >= NNV_ARM_RAW && choices[i].cached <= NNV_ARM_ZERO_COPY, NNV_ERR_INVALID_ARG,
                    "layer %d: %d is not a preparation arm", i, choices[i].cached);
        NNV_REQUIRE(choices[i].cached == NNV_ARM_RAW || variant_has_transform(choices[i].variant), NNV_ERR_INVALID_ARG,
                    "layer %d: variant %d has no transform to cache or fuse", i, choices[i].variant);
        if (choices[i].cached != NNV_ARM_CACHED) continue;
        NNV_REQUIRE(variant_has_transform(choices[i].variant), NNV_ERR_INVALID_ARG,
                    "layer %d: variant %d has no transform to cache", i, choices[i].variant);
        offsets[i] = pos;
        pos += align_up(transformed_bytes(*p, i, choices[i].variant, choices[i].math), 256);
    }
    *total = pos;
    return NNV_OK;
}

nnv_status_t nnv_filter_candidates(const nnv_plan_t* p, int32_t layer, const nnv_cost_t* costs, int32_t n_costs,
                                   int32_t allow_cached, nnv_choice_t* out, int32_t cap, int32_t* n_out) {
    NNV_REQUIRE(p && costs && out && n_out, NNV_ERR_INVALID_ARG, "null argument");
    NNV_REQUIRE(layer >= 0 && layer < (int)p->layers.size() && p->layers[layer].op == NNV_OP_CONV,
                NNV_ERR_INVALID_ARG, "layer %d is not a convolution layer", layer);
    std::vector<Option> opts, surv;
    NNV_TRY(gather_options(*p, layer, costs, n_costs, allow_cached, &opts));
    pareto(opts, &surv);
    NNV_REQUIRE((int)surv.size() <= cap, NNV_ERR_INVALID_ARG, "output capacity %d too small", cap);
    for (size_t i = 0; i < surv.size(); ++i) out[i] = nnv_choice_t{surv[i].variant, surv[i].math, surv[i].cached};
    *n_out = (int)surv.size();
    return NNV_OK;
}

nnv_status_t nnv_select_kernels(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, int32_t allow_cached,
                                nnv_choice_t* out) {
    NNV_REQUIRE(p && costs && out, NNV_ERR_INVALID_ARG, "null argument");
    for (int i = 0; i < (int)p->layers.size(); ++i) {
        out[i] = nnv_choice_t{-1, -1, 0};
        if (p->layers[i].op != NNV_OP_CONV) continue;
        std::vector<Option> opts, surv;
        NNV_TRY(gather_options(*p, i, costs, n_costs, allow_cached, &opts));
        NNV_REQUIRE(!opts.empty(), NNV_ERR_STATE, "no cost rows for conv layer %d", i);
        pareto(opts, &surv);
        const Option* best = nullptr;
        for (const Option& o : surv)                        // surv is in rank order: first minimum wins ties
            if (!best || o.prep + o.exec < best->prep + best->exec) best = &o;
        out[i] = nnv_choice_t{best->variant, best->math, best->cached};
    }
    return NNV_OK;
}

nnv_status_t nnv_select_warm(const nnv_plan_t* p, const nnv_cost_t* costs, int32_t n_costs, nnv_choice_t* out) {
    NNV_REQUIRE(p && costs && out, NNV_ERR_INVALID_ARG, "null argument");
    for (int i = 0; i < (int)p->layers.size(); ++i) {
        out[i] = nnv_choice_t{-1, -1, 0};
        if (p->layers[i].op != NNV_OP_CONV) continue;
        std::vector<Option> opts;
        NNV_TRY(gather_options(*p, i, costs, n_costs, 0, &opts));     // raw arms only: one option per kernel, rank order
        NNV_REQUIRE(!opts.empty(), NNV_ERR_STATE, "no cost rows for conv layer %d", i);
        const Option* best = nullptr;
        for (const Option& o : opts)
            if (!best || o.exec < best->exec) best = &o;             // first minimum wins ties
        out[i] = nnv_choice_t{best->variant, best->math, variant_has_transform(best->variant) ? 1 : 0};
    }
    return NNV_OK;
}

nnv_status_t nnv_switch_set(const nnv_plan_t* p, const nnv_choice_t* cold, const nnv_choice_t* warm, int32_t* layers_out,
                            int32_t cap, int32_t* n_out) {
    NNV_REQUIRE(p && cold && warm && layers_out && n_out, NNV_ERR_INVALID_ARG, "null argument");
    int cnt = 0;
    for (int i = 0; i < (int)p->layers.size(); ++i) {
        if (p->layers[i].op != NNV_OP_CONV) continue;
        if (cold[i].variant == warm[i].variant && cold[i].math == warm[i].math) continue;
        if (!variant_has_transform(warm[i].variant)) continue;
        NNV_REQUIRE(cnt < cap, NNV_ERR_INVALID_ARG, "output capacity %d too small", cap);
        layers_out[cnt++] = i;
    }
    *n_out = cnt;
    return NNV_OK;
}

}  // extern "C"
