"""GPU parity of the weights-on-rows tensor-core kernel for layers with few pixels (H * W <= 256): every K
split it can take, against the fp64 direct-convolution oracle and against the pixel-on-rows GEMM it replaces."""
import numpy as np
import pytest

from oracle import model as omodel
from paper_2206_07446_b200 import binding as nb
from gpu_util import TOL, rel_l2, run_conv, assert_conv_close

pytestmark = pytest.mark.gpu


def _run(L, x, w, b, add, setting, variant):
    nb.nnv_tuning_set(setting)
    try:
        plan = nb.Plan([L], [0], [0])
        ws = nb.nnv_exec_workspace_bytes(plan, 0, variant, nb.MATH_TF32)
        return run_conv(plan, 0, L, variant, nb.MATH_TF32, x, w, b, add), ws
    finally:
        nb.nnv_tuning_set(None)


@pytest.mark.parametrize("shape", [
    # C, K, R, H, W, bias/addend/act
    (512, 512, 3, 7, 7, False),       # ResNet last stage: 144 K blocks
    (256, 256, 3, 14, 14, True),      # 196 pixels -> 208 MMA columns
    (512, 2048, 1, 7, 7, True),       # 16 channel tiles
    (2048, 512, 1, 7, 7, False),
    (64, 40, 3, 5, 3, True),          # K = 40: one partly filled channel tile; 15 pixels -> 16 columns
    (32, 132, 1, 1, 1, True),         # one pixel; K = 132 = 128 + 4
    (96, 64, 3, 16, 16, False),       # 256 pixels: the largest tile; three channel blocks
    (160, 24, 1, 13, 15, True),       # ragged grid, K = 24
    (32, 8, 5, 9, 4, False),          # 5x5 filter with pad 2
])
def test_every_split_matches_the_oracle(shape):
    C, K, R, H, W, epi = shape
    L = dict(op=0, C=C, K=K, R=R, S=R, stride=1, pad=(R - 1) // 2, groups=1, H=H, W=W, in0=-1, in1=-1,
             act=2 if epi else 1, has_bias=1 if epi else 0)
    variant = nb.VAR_GEMM1X1 if R == 1 else nb.VAR_IM2COL
    rng = np.random.default_rng([21] + list(shape[:5]))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, R, R)) * np.sqrt(2.0 / (C * R * R))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32) if epi else None
    add = rng.uniform(-1, 1, (K, H, W)).astype(np.float32) if epi else None
    ref = omodel.run_layer(L, x, w, b, add)
    plain, _ = _run(L, x, w, b, add, "smallp=0", variant)
    assert_conv_close(plain, ref, TOL[nb.MATH_TF32], "pixels on rows")
    nkb = R * R * C // 32
    ran = 0
    for sp in sorted({1, 2, 3, 5, 8, 37, nkb}):
        if sp > nkb:
            continue
        y, ws = _run(L, x, w, b, add, "smallp=%d" % sp if sp > 1 else "smallp=1", variant)
        if sp > 1:
            assert ws >= sp * H * W * K * 4                  # the partial tiles' scratch is part of the size query
        assert_conv_close(y, ref, TOL[nb.MATH_TF32], ("splits", sp))
        # against the pixel-on-rows kernel: the same weights; the activations reach the tensor core truncated
        # to TF32 here and (where that kernel builds an explicit im2col matrix) rounded there
        assert rel_l2(y, plain) <= 1e-3, (sp, rel_l2(y, plain))
        y2, _ = _run(L, x, w, b, add, "smallp=%d" % sp if sp > 1 else "smallp=1", variant)
        assert np.array_equal(y.view(np.uint32), y2.view(np.uint32))          # run to run: the same bits
        ran += 1
    assert ran >= min(2, nkb)
    auto, _ = _run(L, x, w, b, add, None, variant)              # whatever the library picks by itself
    assert_conv_close(auto, ref, TOL[nb.MATH_TF32], "library's choice")
