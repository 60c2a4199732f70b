"""CPU-only checks of the C-ABI library: it loads, exports what include/nnv.h declares, and its
host-side logic (eligibility, sizes, selection, validation) agrees with the oracle exactly."""
import ctypes
import os
import re

import numpy as np
import pytest

import workloads as wl
from oracle import selection as osel
from oracle import winograd as owin
from oracle import pack as opack
from paper_2206_07446_b200 import binding as nb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _plan(layers):
    ws, bs = wl.make_weights(layers)
    # offsets only: sizes of the arrays, not their contents, matter here
    _, w_off, b_off = wl.weight_blob(layers, [None if w is None else np.zeros(w.shape, np.float32) for w in ws], bs)
    return nb.Plan(layers, w_off, b_off)


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "nnv.h")).read()
    declared = set(re.findall(r"^(?:nnv_status_t|const char\*|int32_t)\s+(nnv_[a-z0-9_]+)\s*\(", hdr, re.M))
    assert {"nnv_plan_create", "nnv_select_kernels", "nnv_transform_weights", "nnv_conv_exec", "nnv_cold_run"} <= declared
    lib = ctypes.CDLL(nb.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert declared == set(nb.EXPORTED_SYMBOLS)
    assert nb.nnv_version() >= 100


@pytest.mark.parametrize("name", list(wl.CONFIGS) + ["tiny"])
def test_eligibility_matches_oracle(name):
    layers = wl.tiny_net() if name == "tiny" else wl.CONFIGS[name]()
    plan = _plan(layers)
    for i, L in enumerate(layers):
        want = osel.eligible(L) if L["op"] == wl.OP_CONV else []
        assert nb.nnv_eligible(plan, i) == want, (i, L)


def test_transformed_bytes_match_oracle_shapes():
    layers = wl.tiny_net()
    plan = _plan(layers)
    ws, _ = wl.make_weights(layers)
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            continue
        for v in nb.nnv_eligible(plan, i):
            for m in osel.math_modes(v):
                got = nb.nnv_transformed_bytes(plan, i, v, m)
                es = 2 if m == osel.BF16 else 4
                if v in (osel.WINO_F2, osel.WINO_F4, osel.WINO_F6):
                    mm = {osel.WINO_F2: 2, osel.WINO_F4: 4, osel.WINO_F6: 6}[v]
                    U = owin.pad_channels(owin.filter_transform(ws[i], mm), -(-L["C"] // 8) * 8)
                    assert got == U.size * es
                elif v in (osel.IM2COL, osel.GEMM1X1):
                    assert got == opack.pack_weights(ws[i]).size * es
                else:
                    assert got == 0


def _random_costs(layers, rng, hi=50):
    costs = []
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            continue
        for v in osel.eligible(L):
            for m in osel.math_modes(v):
                if rng.random() < 0.15 and len([c for c in costs if c["layer"] == i]) > 0:
                    continue
                costs.append(dict(layer=i, variant=v, math=m, h2d_raw_ns=int(rng.integers(0, hi)),
                                  xform_ns=int(rng.integers(0, hi)) if osel.has_transform(v) else 0,
                                  h2d_cached_ns=int(rng.integers(0, hi)), exec_ns=int(rng.integers(0, hi)),
                                  zc_ns=int(rng.integers(0, 2 * hi)) if (osel.has_transform(v) and rng.random() < 0.7) else 0))
    return costs


@pytest.mark.parametrize("seed", range(20))
def test_selection_matches_oracle_bit_exact(seed):
    rng = np.random.default_rng(seed)
    layers = [wl.tiny_net, wl.cfg2_resnet18, wl.cfg3_mobilenetv2, wl.cfg5_vgg16][seed % 4]()
    plan = _plan(layers)
    costs = _random_costs(layers, rng, hi=8 if seed % 2 else 10 ** 9)
    for allow in (0, 1, 2, 3):                              # bit 0: cached arm, bit 1: zero-copy arm
        assert nb.nnv_select_kernels(plan, costs, allow) == osel.select_kernels(layers, costs, allow)
        for i, L in enumerate(layers):
            if L["op"] != wl.OP_CONV:
                continue
            rows = [c for c in costs if c["layer"] == i]
            want = [o[0] for o in osel.pareto_filter(osel.options_from_costs(rows, allow))]
            assert nb.nnv_filter_candidates(plan, i, costs, allow) == want


@pytest.mark.parametrize("seed", range(6))
def test_warm_selection_and_switch_set_match_oracle(seed):
    """K_warm (least execution time) and K_warm - K_cold, exactly as the oracle has them."""
    rng = np.random.default_rng(100 + seed)
    layers = [wl.tiny_net, wl.cfg2_resnet18, wl.cfg3_mobilenetv2][seed % 3]()
    plan = _plan(layers)
    costs = _random_costs(layers, rng, hi=6 if seed % 2 else 10 ** 9)
    warm = nb.nnv_select_warm(plan, costs)
    assert warm == osel.select_warm(layers, costs)
    for allow in (0, 1):
        cold = nb.nnv_select_kernels(plan, costs, allow)
        assert nb.nnv_switch_set(plan, cold, warm) == osel.switch_set(cold, warm)
    assert nb.nnv_switch_set(plan, warm, warm) == []


def test_selection_on_paper_table2_shaped_costs():
    """The paper's Table 2 numbers mapped onto this library's variants for a 64->192 3x3 layer:
    winograd-pack4 -> WINO_F6/TF32, winograd -> WINO_F4/TF32, sgemm-pack4 -> IM2COL/TF32, 3x3s1 -> DIRECT."""
    layers = [dict(op=0, C=64, K=192, R=3, S=3, stride=1, pad=1, groups=1, H=28, W=28, in0=-1, in1=-1, act=1, has_bias=0)]
    plan = _plan(layers)
    rows = {}
    for line in open(os.path.join(ROOT, "tests", "golden", "table2_costs.txt")):
        if line.strip() and not line.startswith("#"):
            name, rr, wt, rc, ex = line.split()
            rows[name] = (int(rr), int(wt), int(rc), int(ex))
    m = {"3x3s1-winograd-pack4": (nb.VAR_WINO_F6, 1), "3x3s1-winograd": (nb.VAR_WINO_F4, 1),
         "sgemm-pack4": (nb.VAR_IM2COL, 1), "3x3s1": (nb.VAR_DIRECT, 0)}
    costs = [dict(layer=0, variant=v, math=mm, h2d_raw_ns=rows[k][0], xform_ns=rows[k][1], h2d_cached_ns=rows[k][2],
                  exec_ns=rows[k][3]) for k, (v, mm) in m.items()]
    assert nb.nnv_select_kernels(plan, costs, 1) == [(nb.VAR_WINO_F4, 1, 1)]       # cached winograd: 7.49 ms
    assert nb.nnv_select_kernels(plan, costs, 0) == [(nb.VAR_DIRECT, 0, 0)]        # raw only: 3x3s1, 8.71 ms
    assert nb.nnv_filter_candidates(plan, 0, costs, 1) == [(nb.VAR_DIRECT, 0, 0), (nb.VAR_WINO_F4, 1, 1), (nb.VAR_WINO_F6, 1, 1)]
    # warm inference: winograd-pack4 executes fastest (2.98 ms), so K_warm differs from both cold choices
    warm = nb.nnv_select_warm(plan, costs)
    assert warm == [(nb.VAR_WINO_F6, 1, 1)]
    assert nb.nnv_switch_set(plan, nb.nnv_select_kernels(plan, costs, 1), warm) == [0]


def test_plan_validation_errors():
    good = wl.cfg1()
    for mutate, status in [
        (dict(C=0), 1), (dict(in0=0), 1), (dict(act=7), 1), (dict(groups=3), 1), (dict(groups=2), 2),
        (dict(R=99, S=99), 1), (dict(op=9), 1),
    ]:
        L = [dict(good[0], **mutate)]
        with pytest.raises(nb.NnvError) as e:
            nb.Plan(L, [0], [0])
        assert e.value.status == status, (mutate, str(e.value))
    with pytest.raises(nb.NnvError):
        nb.Plan(good, [4], [0])                      # misaligned weight offset
    # producer shape mismatch
    two = wl.tiny_net()[:2]
    two[1] = dict(two[1], C=13)
    with pytest.raises(nb.NnvError):
        nb.Plan(two, [0, 0], [0, 0])


def test_host_side_argument_errors_before_any_launch():
    plan = _plan(wl.cfg1())
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_transformed_bytes(plan, 0, nb.VAR_GEMM1X1, nb.MATH_TF32)          # 3x3 layer is not 1x1
    assert e.value.status == 2
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_transformed_bytes(plan, 0, nb.VAR_WINO_F2, nb.MATH_FP32)          # no fp32 tensor-core mode
    assert e.value.status == 2
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_transformed_bytes(plan, 5, nb.VAR_DIRECT, nb.MATH_FP32)
    assert e.value.status == 1
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_transform_weights(plan, 0, nb.VAR_WINO_F2, nb.MATH_TF32, 0, 0)    # null pointers
    assert e.value.status == 1
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_transform_weights(plan, 0, nb.VAR_WINO_F2, nb.MATH_TF32, 260, 512)  # misaligned pointer
    assert e.value.status == 1
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_arena_bytes(plan, [(nb.VAR_WINO_F2, 1, 0)], 9)                    # depth beyond max_depth
    assert e.value.status == 1
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_select_kernels(plan, [dict(layer=0, variant=nb.VAR_DEPTHWISE, math=0, h2d_raw_ns=1, xform_ns=0,
                                          h2d_cached_ns=1, exec_ns=1)], 1)
    assert e.value.status == 1
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_select_kernels(plan, [], 1)
    assert e.value.status == 3


def test_arena_and_workspace_sizes_are_consistent():
    layers = wl.cfg2_resnet18()
    plan = _plan(layers)
    ch = []
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            ch.append(None)
        else:
            el = nb.nnv_eligible(plan, i)
            ch.append((nb.VAR_WINO_F4, 1, 0) if nb.VAR_WINO_F4 in el else (nb.VAR_IM2COL, 1, 0))
    a1, a4 = nb.nnv_arena_bytes(plan, ch, 1), nb.nnv_arena_bytes(plan, ch, 4)
    assert a4 > a1
    # the largest F(4,3) transform of a 512x512 layer is 36 planes * 512 * 512 * 4 bytes
    assert nb.nnv_transformed_bytes(plan, 19, nb.VAR_WINO_F4, 1) == 36 * 512 * 512 * 4
    assert nb.nnv_transformed_bytes(plan, 19, nb.VAR_WINO_F2, 2) == 16 * 512 * 512 * 2
    with pytest.raises(nb.NnvError) as e:            # F(4,3)/F(6,3) exist in the TF32 accuracy class only
        nb.nnv_transformed_bytes(plan, 19, nb.VAR_WINO_F4, 2)
    assert e.value.status == 2
    offs, total = nb.nnv_cached_layout(plan, [None if c is None else (c[0], c[1], 1) for c in ch])
    assert total >= sum(nb.nnv_transformed_bytes(plan, i, c[0], c[1]) for i, c in enumerate(ch) if c)
    assert all(o % 256 == 0 for o in offs)


def test_tuning_overrides_parse_and_reject():
    """nnv_tuning_set: documented items are accepted, anything else is refused and changes nothing."""
    try:
        for ok in ("gemm_tile=64,4", "gemm_ring=6;gemm_prefill=0", "conv3x3=off", "conv3x3=auto", "conv3x3=2,64,4",
                   "conv3x3=1,128,2,1,3", "side=0;merge=0;group=0", "", None, "gemm_tile=16,1;;side=1",
                   "conv3x3p=64,2,2,6", "conv3x3p=off", "conv3x3w=on", "conv3x3w=auto;conv3x3w=off", "bf16cvt=0", "winofused=auto",
                   "smallp=0", "smallp=24", "copies_first=0", "chunk=64,8192", "chunk=256,256"):
            nb.nnv_tuning_set(ok)
        for bad in ("gemm_tile=48", "gemm_tile=24,2", "gemm_tile=64,3", "gemm_ring=9", "conv3x3=3,64,1", "conv3x3=1,64,16",
                    "side=2", "unknown=1", "gemm_tile", "x" * 300, "conv3x3w=2", "conv3x3p=24,1", "copies_first=2", "chunk=8,64",
                    "chunk=512,256", "chunk=256", "bf16cvt=yes", "smallp=149"):
            with pytest.raises(nb.NnvError) as e:
                nb.nnv_tuning_set(bad)
            assert e.value.status == 1, bad
    finally:
        nb.nnv_tuning_set(None)
