"""GPU parity of the one-kernel Winograd F(2x2,3x3) path (input transform, 16 tile GEMMs with the accumulators in
TMEM, output transform) against the fp64 direct-convolution oracle and against the three-kernel path it replaces."""
import numpy as np
import pytest

from oracle import model as omodel
from paper_2206_07446_b200 import binding as nb
from gpu_util import TOL, rel_l2, run_conv, assert_conv_close

pytestmark = pytest.mark.gpu


def _run(L, x, w, b, add, setting):
    nb.nnv_tuning_set(setting)
    try:
        plan = nb.Plan([L], [0], [0])
        return run_conv(plan, 0, L, nb.VAR_WINO_F2, nb.MATH_TF32, x, w, b, add)
    finally:
        nb.nnv_tuning_set(None)


@pytest.mark.parametrize("shape", [
    # C, K, H, W, pad, bias/addend/act
    (64, 64, 56, 56, 1, False),       # config 1: 784 tiles, 16 channels per CTA
    (64, 64, 112, 112, 1, True),      # 3136 tiles: 32 channels per CTA (all of TMEM), epilogue terms
    (24, 40, 13, 11, 1, True),        # ragged grid (odd sizes: clipped tiles), K = 40, three channel steps
    (8, 8, 3, 3, 1, False),           # one channel step, four tiles
    (16, 16, 6, 5, 0, True),          # pad 0
    (128, 128, 28, 28, 1, False),
    (512, 512, 7, 7, 1, True),        # 64 channel steps: the ring wraps many times
    (8, 48, 130, 3, 1, False),        # a tall, narrow image: 65 x 2 tiles
])
def test_fused_path_matches_oracle_and_the_three_kernel_path(shape):
    C, K, H, W, pad, epi = shape
    L = dict(op=0, C=C, K=K, R=3, S=3, stride=1, pad=pad, groups=1, H=H, W=W, in0=-1, in1=-1, act=2 if epi else 1,
             has_bias=1 if epi else 0)
    OH, OW = H + 2 * pad - 2, W + 2 * pad - 2
    rng = np.random.default_rng([41] + list(shape[:5]))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, 3, 3)) * np.sqrt(2.0 / (C * 9))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32) if epi else None
    add = rng.uniform(-1, 1, (K, OH, OW)).astype(np.float32) if epi else None
    ref = omodel.run_layer(L, x, w, b, add)
    three = _run(L, x, w, b, add, "winofused=0")
    fused = _run(L, x, w, b, add, "winofused=1")
    if OH * OW * K >= 256:                                     # tiny outputs: the pooled test of the degenerate shapes covers them
        assert_conv_close(three, ref, TOL[nb.MATH_TF32], "three kernels")
        assert_conv_close(fused, ref, TOL[nb.MATH_TF32], "one kernel")
    # the same rounded operands and the same channel order; only the fp32 additions of the two small transforms
    # may be associated differently
    assert rel_l2(fused, three) <= 2e-6, rel_l2(fused, three)
    again = _run(L, x, w, b, add, "winofused=1")
    assert np.array_equal(fused.view(np.uint32), again.view(np.uint32))
