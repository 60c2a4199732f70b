"""GPU parity: execution of one layer with every kernel variant against the fp64 direct-convolution
oracle, through the C ABI, with oracle-fed inputs."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import conv as oconv
from oracle import model as omodel
from paper_2206_07446_b200 import binding as nb
from gpu_util import TOL, dev, poisoned, chw_to_hwc, hwc_to_chw, rel_l2, run_conv, assert_conv_close

pytestmark = pytest.mark.gpu


def _maths(v):
    if v in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
        return [nb.MATH_FP32]
    if v in (nb.VAR_WINO_F4, nb.VAR_WINO_F6):
        return [nb.MATH_TF32]
    return [nb.MATH_TF32, nb.MATH_BF16]


def _check_layer(layers, i, x, w, b, add, variants=None):
    L = layers[i]
    plan = nb.Plan(layers, [0] * len(layers), [0] * len(layers))
    ref = omodel.run_layer(L, x, w, b, add)
    seen = []
    for v in nb.nnv_eligible(plan, i):
        if variants is not None and v not in variants:
            continue
        for m in _maths(v):
            y = run_conv(plan, i, L, v, m, x, w, b, add)
            err = assert_conv_close(y, ref, TOL[m], (nb.VARIANT_NAMES[v], nb.MATH_NAMES[m]))
            seen.append((nb.VARIANT_NAMES[v], nb.MATH_NAMES[m], err))
    return seen


def test_cfg1_all_variants():
    """Config 1: 3x3 s1 p1, 64->64, 56x56: direct, im2col, Winograd F(2,3)/F(4,3)/F(6,3)."""
    layers = wl.cfg1()
    ws, bs = wl.make_weights(layers)
    x = wl.make_input(layers)[0]
    seen = _check_layer(layers, 0, x, ws[0], None, None)
    assert len(seen) == 1 + 2 + 4
    print(seen)


def test_tiny_net_every_layer_every_variant():
    """Ragged shapes (C=5, 9x7 grid, K=12/20/9), residual, bias, ReLU6, strides, depthwise; oracle-fed inputs."""
    layers = wl.tiny_net()
    ws, bs = wl.make_weights(layers, seed=3)
    x = wl.make_input(layers, seed=3)
    acts = omodel.run_model(layers, ws, bs, x)
    plan = nb.Plan(layers, [0] * len(layers), [0] * len(layers))
    for i, L in enumerate(layers):
        src = x[0] if L["in0"] < 0 else acts[L["in0"]].astype(np.float32)
        if L["op"] == wl.OP_CONV:
            add = None if L["in1"] < 0 else acts[L["in1"]].astype(np.float32)
            _check_layer(layers, i, src, ws[i], bs[i], add)
        else:
            oh, ow = wl.out_hw(L)
            d_out = poisoned(4 * oh * ow * L["K"])
            nb.nnv_pool_exec(plan, i, dev(chw_to_hwc(src)), d_out, torch.cuda.current_stream())
            torch.cuda.synchronize()
            y = hwc_to_chw(d_out[:4 * oh * ow * L["K"]].view(torch.float32).reshape(oh, ow, L["K"]).cpu().numpy())
            ref = omodel.run_layer(L, src)
            tol = 0.0 if L["op"] == wl.OP_MAXPOOL else 1e-6
            assert np.max(np.abs(y - ref)) <= tol * max(1.0, np.max(np.abs(ref)))


@pytest.mark.parametrize("shape", [
    # C, K, R, stride, H, W, groups
    (3, 64, 7, 2, 224, 224, 1),        # ResNet stem
    (512, 512, 3, 1, 7, 7, 1),         # ResNet-18 last stage (tiny grid, large K reduction)
    (64, 128, 1, 2, 56, 56, 1),        # strided 1x1 downsample
    (256, 256, 3, 2, 28, 28, 1),       # strided 3x3
    (16, 96, 1, 1, 112, 112, 1),       # MobileNetV2 expand, narrow C
    (96, 24, 1, 1, 56, 56, 1),         # project to K=24 (not a multiple of 16)
    (320, 1280, 1, 1, 7, 7, 1),        # wide 1x1 on a tiny grid
    (144, 144, 3, 2, 56, 56, 144),     # depthwise stride 2
    (384, 384, 3, 1, 14, 14, 384),     # depthwise stride 1
    (512, 2048, 1, 1, 7, 7, 1),        # ResNet-50 last 1x1
    (128, 128, 3, 1, 28, 28, 1),       # Winograd edge tiles: 28 = 4*7 = 6*4+4
    (256, 256, 3, 1, 14, 14, 1),       # 14 = 4*3+2 = 6*2+2
    (3, 64, 3, 1, 224, 224, 1),        # VGG conv1_1 (C=3 padded to 8 in the Winograd domain)
    (64, 64, 3, 1, 112, 112, 1),       # large-grid VGG-like layer (scaled down from 224 for oracle time)
])
def test_config_layer_shapes(shape):
    C, K, R, stride, H, W, groups = shape
    pad = R // 2
    L = dict(op=0, C=C, K=K, R=R, S=R, stride=stride, pad=pad, groups=groups, H=H, W=W, in0=-1, in1=-1, act=1, has_bias=0)
    rng = np.random.default_rng(list(shape))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    cg = C // groups
    w = (rng.standard_normal((K, cg, R, R)) * np.sqrt(2.0 / (cg * R * R))).astype(np.float32)
    seen = _check_layer([L], 0, x, w, None, None)
    print(shape, seen)


@pytest.mark.parametrize("shape", [
    # C, K, R, H, W, pad -- stride 1; every eligible variant and math mode runs on each
    (1, 1, 3, 1, 1, 1),               # one channel in, one out, a grid of one pixel (smaller than any Winograd tile)
    (1, 8, 3, 2, 3, 1),               # C = 1
    (8, 1, 3, 3, 2, 1),               # K = 1
    (5, 7, 3, 3, 3, 0),               # pad 0: 3x3 input -> 1x1 output
    (16, 16, 3, 6, 5, 0),             # pad 0 on a Winograd layer, output 4x3
    (24, 40, 3, 14, 14, 0),           # pad 0, output 12x12 = whole F(2,3)/F(4,3)/F(6,3) tiles
    (1, 1, 3, 9, 7, 1),               # C = K = 1 on a ragged grid
    (4, 1, 1, 10, 10, 0),             # 1x1 with K = 1
    (1, 4, 1, 7, 7, 0),               # 1x1 with C = 1
    (3, 5, 3, 2, 2, 1),               # 2x2 grid
])
def test_degenerate_shapes_on_every_variant(shape):
    """A layer with a handful of outputs gives a rel-L2 that is the norm of a handful of rounding errors and
    fluctuates by +-50 % from draw to draw (one TF32 F(2,3) pass on a 5-channel 1x1-output layer: median 6e-4,
    one draw in twelve above 1e-3), so the error is pooled over 16 seeded instances of the shape."""
    C, K, R, H, W, pad = shape
    L = dict(op=0, C=C, K=K, R=R, S=R, stride=1, pad=pad, groups=1, H=H, W=W, in0=-1, in1=-1, act=0, has_bias=1)
    plan = nb.Plan([L], [0], [0])
    got, want = {}, []
    for inst in range(16):
        rng = np.random.default_rng([11, inst] + list(shape))
        x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
        w = (rng.standard_normal((K, C, R, R)) * np.sqrt(2.0 / (C * R * R))).astype(np.float32)
        b = rng.uniform(-1, 1, K).astype(np.float32)
        want.append(omodel.run_layer(L, x, w, b, None))
        for v in nb.nnv_eligible(plan, 0):
            for m in _maths(v):
                got.setdefault((v, m), []).append(run_conv(plan, 0, L, v, m, x, w, b, None))
    assert len(got) >= 3
    ref = np.stack(want)
    for (v, m), ys in got.items():
        err = assert_conv_close(np.stack(ys), ref, TOL[m], (nb.VARIANT_NAMES[v], nb.MATH_NAMES[m]))
        print(shape, nb.VARIANT_NAMES[v], nb.MATH_NAMES[m], "%.2e" % err)


def test_halo_kernel_on_a_ragged_full_size_grid():
    """128 -> 128, 3x3 on 57 x 59 (H % 16 != 0, W % 8 != 0) with bias, residual addend and ReLU: the library's own choice,
    the plain implicit GEMM and the halo-resident 3x3 kernel (tiling forced, with and without a K split) agree."""
    L = dict(op=0, C=128, K=128, R=3, S=3, stride=1, pad=1, groups=1, H=57, W=59, in0=-1, in1=-1, act=1, has_bias=1)
    rng = np.random.default_rng(57)
    x = rng.uniform(-1, 1, (128, 57, 59)).astype(np.float32)
    w = (rng.standard_normal((128, 128, 3, 3)) * np.sqrt(2.0 / (128 * 9))).astype(np.float32)
    b = rng.uniform(-1, 1, 128).astype(np.float32)
    add = rng.uniform(-1, 1, (128, 57, 59)).astype(np.float32)
    ref = omodel.run_layer(L, x, w, b, add)
    plan = nb.Plan([L], [0], [0])
    y = run_conv(plan, 0, L, nb.VAR_IM2COL, nb.MATH_TF32, x, w, b, add)
    assert_conv_close(y, ref, TOL[nb.MATH_TF32], "library's choice")
    nb.nnv_tuning_set("conv3x3=off")
    try:
        y_plain = run_conv(plan, 0, L, nb.VAR_IM2COL, nb.MATH_TF32, x, w, b, add)
    finally:
        nb.nnv_tuning_set(None)
    assert_conv_close(y_plain, ref, TOL[nb.MATH_TF32], "plain implicit GEMM")
    assert rel_l2(y, y_plain) <= 1e-5
    for tiling in ("1,128,4", "1,128,1", "2,64,2"):
        nb.nnv_tuning_set("conv3x3=" + tiling)
        try:
            y_halo = run_conv(plan, 0, L, nb.VAR_IM2COL, nb.MATH_TF32, x, w, b, add)
        finally:
            nb.nnv_tuning_set(None)
        assert_conv_close(y_halo, ref, TOL[nb.MATH_TF32], "halo kernel " + tiling)
        assert rel_l2(y_halo, y_plain) <= 1e-5


def test_residual_and_bias_epilogues_on_every_variant():
    """bias + addend + ReLU6 through each kernel's epilogue (K = 40 is not a multiple of 16)."""
    base = dict(op=0, C=24, K=40, R=3, S=3, stride=1, pad=1, groups=1, H=13, W=11, in0=-1, in1=-1, act=0, has_bias=0)
    layers = [base, dict(base, C=40, in0=0, in1=0, act=2, has_bias=1)]
    rng = np.random.default_rng(5)
    x = rng.uniform(-1, 1, (40, 13, 11)).astype(np.float32)
    w = (rng.standard_normal((40, 40, 3, 3)) * 0.05).astype(np.float32)
    b = rng.uniform(-1, 1, 40).astype(np.float32)
    add = rng.uniform(-3, 3, (40, 13, 11)).astype(np.float32)
    seen = _check_layer(layers, 1, x, w, b, add)
    assert len(seen) == 7


def test_layout_helpers_roundtrip():
    rng = np.random.default_rng(6)
    x = rng.uniform(-1, 1, (5, 7, 9)).astype(np.float32)
    d_in = dev(x)
    d_hwc = poisoned(x.nbytes)
    d_back = poisoned(x.nbytes)
    nb.nnv_chw_to_hwc(d_in, d_hwc, 5, 7, 9, torch.cuda.current_stream())
    nb.nnv_hwc_to_chw(d_hwc, d_back, 5, 7, 9, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert np.array_equal(d_hwc[:x.nbytes].view(torch.float32).reshape(7, 9, 5).cpu().numpy(), chw_to_hwc(x))
    assert np.array_equal(d_back[:x.nbytes].view(torch.float32).reshape(5, 7, 9).cpu().numpy(), x)


def test_workspace_too_small_is_reported():
    layers = wl.cfg1()
    plan = nb.Plan(layers, [0], [0])
    buf = poisoned(1 << 20)
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_conv_exec(plan, 0, nb.VAR_WINO_F4, nb.MATH_TF32, buf, None, buf, None, buf, buf, 1024, torch.cuda.current_stream())
    assert e.value.status == 4


@pytest.mark.parametrize("shape", [
    # C, K, R, stride, H, W
    (64, 64, 3, 1, 56, 56),           # implicit im2col, bf16 rounding inside the GEMM
    (128, 128, 3, 1, 28, 28),         # K split over a cluster
    (256, 512, 3, 2, 28, 28),         # stride 2
    (256, 64, 1, 1, 56, 56),          # 1x1: the activation itself is the operand
    (64, 24, 1, 1, 57, 43),           # ragged pixels, K = 24
    (40, 72, 3, 1, 64, 64),           # C = 40: the last channel block is partly outside the tensor
])
def test_bf16_math_without_a_bf16_copy_of_the_activation(shape):
    """BF16-class GEMM layers whose fp32 activation is rounded to bf16 inside the kernel (no Xcol matrix, no scratch)
    against the oracle, and against the explicit bf16 im2col path: the same rounded operands, so fp32-rounding apart."""
    C, K, R, stride, H, W = shape
    L = dict(op=0, C=C, K=K, R=R, S=R, stride=stride, pad=R // 2, groups=1, H=H, W=W, in0=-1, in1=-1, act=1, has_bias=1)
    rng = np.random.default_rng([51] + list(shape))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, R, R)) * np.sqrt(2.0 / (C * R * R))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32)
    ref = omodel.run_layer(L, x, w, b, None)
    v = nb.VAR_GEMM1X1 if R == 1 else nb.VAR_IM2COL
    plan = nb.Plan([L], [0], [0])
    assert nb.nnv_exec_workspace_bytes(plan, 0, v, nb.MATH_BF16) == 0
    y = run_conv(plan, 0, L, v, nb.MATH_BF16, x, w, b, None)
    assert_conv_close(y, ref, TOL[nb.MATH_BF16], "rounded in the kernel")
    nb.nnv_tuning_set("bf16cvt=0")
    try:
        plan2 = nb.Plan([L], [0], [0])
        assert nb.nnv_exec_workspace_bytes(plan2, 0, v, nb.MATH_BF16) > 0
        y2 = run_conv(plan2, 0, L, v, nb.MATH_BF16, x, w, b, None)
    finally:
        nb.nnv_tuning_set(None)
    assert_conv_close(y2, ref, TOL[nb.MATH_BF16], "explicit bf16 im2col")
    assert rel_l2(y, y2) <= 1e-5, rel_l2(y, y2)


@pytest.mark.parametrize("shape", [
    # C, H, W, stride, pad, bias + addend + ReLU6
    (8, 9, 7, 1, 1, True),             # ragged grid: output width 7 = one group of four pixels and a tail of three
    (8, 9, 7, 2, 1, True),             # stride 2, output 5 x 4
    (32, 17, 21, 1, 0, False),         # pad 0
    (32, 18, 22, 2, 0, True),          # stride 2, pad 0
    (96, 112, 112, 1, 1, False),       # MobileNetV2-shaped, stride 1
    (96, 112, 112, 2, 1, True),        # MobileNetV2-shaped, stride 2
    (4, 1, 1, 1, 1, True),             # one pixel
    (6, 9, 7, 1, 1, True),             # C % 4 != 0: the one-channel-per-thread kernel
])
def test_depthwise_kernels(shape):
    """3x3 depthwise layers on the vectorised kernel (four channels x four output pixels per thread) and its scalar
    fallback: fp32 arithmetic, so the fp32 tolerance, element by element."""
    C, H, W, stride, pad, epi = shape
    L = dict(op=0, C=C, K=C, R=3, S=3, stride=stride, pad=pad, groups=C, H=H, W=W, in0=-1, in1=-1, act=2 if epi else 1,
             has_bias=1 if epi else 0)
    rng = np.random.default_rng([13] + [int(v) for v in shape])
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((C, 1, 3, 3)) * np.sqrt(2.0 / 9)).astype(np.float32)
    oh, ow = wl.out_hw(L)
    b = rng.uniform(-1, 1, C).astype(np.float32) if epi else None
    add = rng.uniform(-1, 1, (C, oh, ow)).astype(np.float32) if epi else None
    seen = _check_layer([L], 0, x, w, b, add, variants=[nb.VAR_DEPTHWISE])
    assert [s[:2] for s in seen] == [("depthwise", "fp32")]


def _random_shapes(count, seed):
    """Seeded layer shapes that no hand-written list would think of: ragged channels, grids, strides and pads.
    Kept to >= 2048 outputs (the tolerance is a statement about many rounding errors, see the degenerate-shape test)
    and to a reduction of >= 32 products per output."""
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < count:
        R = int(rng.choice([1, 3, 3, 5]))
        stride = int(rng.choice([1, 1, 2]))
        pad = int(rng.choice([0, R // 2]))
        C = int(rng.choice([int(rng.integers(1, 48)), int(rng.integers(48, 200)), int(8 * rng.integers(1, 40))]))
        K = int(rng.choice([int(rng.integers(1, 48)), int(rng.integers(48, 200)), int(16 * rng.integers(1, 20))]))
        H, W = int(rng.integers(R, 48)), int(rng.integers(R, 48))
        oh, ow = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - R) // stride + 1
        if oh < 1 or ow < 1 or K * oh * ow < 2048 or C * R * R < 32:
            continue
        out.append((C, K, R, stride, pad, H, W, int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.integers(0, 3))))
    return out


@pytest.mark.parametrize("shape", _random_shapes(36, 20240607))
def test_random_shapes_on_every_variant(shape):
    """Every eligible variant and math mode of a randomly drawn layer against the fp64 oracle."""
    C, K, R, stride, pad, H, W, has_bias, has_add, act = shape
    L = dict(op=0, C=C, K=K, R=R, S=R, stride=stride, pad=pad, groups=1, H=H, W=W, in0=-1, in1=-1, act=act, has_bias=has_bias)
    rng = np.random.default_rng([5] + [int(v) for v in shape])
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, R, R)) * np.sqrt(2.0 / (C * R * R))).astype(np.float32)
    oh, ow = wl.out_hw(L)
    b = rng.uniform(-1, 1, K).astype(np.float32) if has_bias else None
    add = rng.uniform(-1, 1, (K, oh, ow)).astype(np.float32) if has_add else None
    seen = _check_layer([L], 0, x, w, b, add)
    assert len(seen) >= 2


def _random_kernel_shapes(seed):
    """Random shapes inside the domains of the two specialised tensor-core kernels: the halo 3x3 kernel (3x3, stride
    1, pad 1, C % 32 == 0, enough patches to fill the GPU) and the weights-on-rows kernel (grids of at most 64 pixels,
    C % 32 == 0, K % 4 == 0)."""
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(6):
        out.append((int(32 * rng.integers(1, 4)), int(rng.integers(8, 140)), 3, int(rng.integers(130, 200)), int(rng.integers(100, 150)), 1))
    for _ in range(8):
        R = int(rng.choice([1, 3]))
        out.append((int(32 * rng.integers(1, 17)), int(4 * rng.integers(1, 130)), R, int(rng.integers(1, 9)), int(rng.integers(1, 9)), R // 2))
    return out


@pytest.mark.parametrize("shape", _random_kernel_shapes(77))
def test_random_shapes_in_the_domains_of_the_specialised_kernels(shape):
    C, K, R, H, W, pad = shape
    L = dict(op=0, C=C, K=K, R=R, S=R, stride=1, pad=pad, groups=1, H=H, W=W, in0=-1, in1=-1, act=1, has_bias=1)
    rng = np.random.default_rng([6] + [int(v) for v in shape])
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, R, R)) * np.sqrt(2.0 / (C * R * R))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32)
    variants = [nb.VAR_IM2COL] + ([nb.VAR_GEMM1X1] if R == 1 else [])
    if K * H * W < 2048:                                   # few outputs: pool the error over instances (see the degenerate-shape test)
        errs = {}
        for inst in range(8):
            xi = np.random.default_rng([7, inst] + [int(v) for v in shape]).uniform(-1, 1, (C, H, W)).astype(np.float32)
            ref = omodel.run_layer(L, xi, w, b, None)
            plan = nb.Plan([L], [0], [0])
            for v in variants:
                for m in _maths(v):
                    y = run_conv(plan, 0, L, v, m, xi, w, b, None)
                    assert np.all(np.isfinite(y))
                    num, den = errs.get((v, m), (0.0, 0.0))
                    errs[(v, m)] = (num + float(np.sum((y - ref) ** 2)), den + float(np.sum(ref * ref)))
        for (v, m), (num, den) in errs.items():
            assert np.sqrt(num / max(den, 1e-30)) <= TOL[m], (v, m, np.sqrt(num / den))
    else:
        seen = _check_layer([L], 0, x, w, b, None, variants=variants)
        assert seen
