"""GPU parity of the halo-resident 3x3 tensor-core kernel: every tiling it can take (one or two MMA
tiles per CTA, several channel-tile widths, K splits over a thread-block cluster) against the fp64
direct-convolution oracle, and against the plain implicit GEMM that it replaces."""
import numpy as np
import pytest

from oracle import model as omodel
from paper_2206_07446_b200 import binding as nb
from gpu_util import TOL, rel_l2, run_conv

pytestmark = pytest.mark.gpu

def _run(L, x, w, b, add, setting, math=nb.MATH_TF32):
    """One layer with the 3x3 kernel's tiling forced through nnv_tuning_set (None = the library's own pick)."""
    nb.nnv_tuning_set(None if setting is None else "conv3x3=" + setting)
    try:
        plan = nb.Plan([L], [0], [0])
        return run_conv(plan, 0, L, nb.VAR_IM2COL, math, x, w, b, add)
    finally:
        nb.nnv_tuning_set(None)


@pytest.mark.parametrize("shape", [
    # C, K, H, W, bias/addend/act
    (64, 64, 56, 56, False),         # config 1 / ResNet stage 1
    (32, 48, 40, 30, True),          # ragged: H % 16 != 0, W % 8 != 0, K = 48, epilogue terms
    (128, 128, 28, 28, True),        # four channel blocks: K splits 2 and 4
    (96, 40, 19, 21, False),         # K = 40 (not a multiple of 16), three channel blocks
    (256, 20, 17, 9, True),          # K = 20: scalar epilogue stores; eight channel blocks: split 8
])
def test_every_tiling_matches_the_oracle(shape):
    C, K, H, W, epi = shape
    L = dict(op=0, C=C, K=K, R=3, S=3, stride=1, pad=1, groups=1, H=H, W=W, in0=-1, in1=-1, act=2 if epi else 1,
             has_bias=1 if epi else 0)
    rng = np.random.default_rng([7] + list(shape[:4]))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, 3, 3)) * np.sqrt(2.0 / (C * 9))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32) if epi else None
    add = rng.uniform(-1, 1, (K, H, W)).astype(np.float32) if epi else None
    ref = omodel.run_layer(L, x, w, b, add)
    plain = _run(L, x, w, b, add, "off")
    assert rel_l2(plain, ref) <= TOL[nb.MATH_TF32]
    bn_full = min(128, -(-K // 16) * 16)
    cblk = C // 32
    ran = 0
    for mt in (1, 2):
        for bn in sorted({bn_full, 16, min(bn_full, 64)}):
            for sp in (1, 2, 4, 8):
                if sp > cblk:
                    continue
                y = _run(L, x, w, b, add, "%d,%d,%d" % (mt, bn, sp))
                assert np.all(np.isfinite(y)), (mt, bn, sp)
                err = rel_l2(y, ref)
                assert err <= TOL[nb.MATH_TF32], (mt, bn, sp, err)
                # same products, other summation order than the plain kernel: fp32 rounding apart only
                assert rel_l2(y, plain) <= 1e-5, (mt, bn, sp, rel_l2(y, plain))
                ran += 1
    assert ran >= 4
    # whatever the library picks by itself is one of the two kernels above
    auto = _run(L, x, w, b, add, None)
    assert rel_l2(auto, ref) <= TOL[nb.MATH_TF32]
    # BF16 math on the same tilings: the halo boxes are rounded to bf16 in shared memory, the weights arrive as bf16;
    # the same products as the converting implicit GEMM (conv3x3=off), summed in another order
    plain16 = _run(L, x, w, b, add, "off", nb.MATH_BF16)
    assert rel_l2(plain16, ref) <= TOL[nb.MATH_BF16]
    ran16 = 0
    for mt in (1, 2):
        for bn in sorted({bn_full, 16, min(bn_full, 64)}):
            for sp in (1, 2, 4, 8):
                if sp > cblk:
                    continue
                y = _run(L, x, w, b, add, "%d,%d,%d" % (mt, bn, sp), nb.MATH_BF16)
                assert np.all(np.isfinite(y)), (mt, bn, sp)
                assert rel_l2(y, ref) <= TOL[nb.MATH_BF16], (mt, bn, sp, rel_l2(y, ref))
                assert rel_l2(y, plain16) <= 1e-5, (mt, bn, sp, rel_l2(y, plain16))
                ran16 += 1
    assert ran16 >= 4


def _run_p(L, x, w, b, add, setting):
    nb.nnv_tuning_set(setting)
    try:
        plan = nb.Plan([L], [0], [0])
        return run_conv(plan, 0, L, nb.VAR_IM2COL, nb.MATH_TF32, x, w, b, add)
    finally:
        nb.nnv_tuning_set(None)


@pytest.mark.parametrize("shape", [
    # C, K, H, W, bias/addend/act
    (64, 64, 56, 56, False),         # 49 patches: with one CTA per SM forced to few CTAs, several tiles per CTA
    (32, 48, 40, 30, True),          # ragged: H % 16 != 0, W % 8 != 0, K = 48, epilogue terms
    (96, 200, 35, 21, True),         # K = 200: two channel tiles at BN = 128, the second partly filled; three channel blocks
    (64, 20, 100, 9, False),         # K = 20: scalar epilogue stores; many patches
])
def test_persistent_form_matches_the_oracle(shape):
    """The persistent 3x3 kernel (tiles walked by resident CTAs, two TMEM accumulators): every tile width and ring
    depth it can take, with more tiles than CTAs, against the oracle and the one-tile-per-CTA kernel."""
    C, K, H, W, epi = shape
    L = dict(op=0, C=C, K=K, R=3, S=3, stride=1, pad=1, groups=1, H=H, W=W, in0=-1, in1=-1, act=2 if epi else 1,
             has_bias=1 if epi else 0)
    rng = np.random.default_rng([9] + list(shape[:4]))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, 3, 3)) * np.sqrt(2.0 / (C * 9))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32) if epi else None
    add = rng.uniform(-1, 1, (K, H, W)).astype(np.float32) if epi else None
    ref = omodel.run_layer(L, x, w, b, add)
    one_tile = _run_p(L, x, w, b, add, "conv3x3p=off;conv3x3=1,%d,1" % min(128, -(-K // 16) * 16))
    assert rel_l2(one_tile, ref) <= TOL[nb.MATH_TF32]
    bn_full = min(128, -(-K // 16) * 16)
    for bn in sorted({bn_full, 16, min(bn_full, 64)}):
        for per_sm, na, nb_ in ((1, 2, 3), (1, 4, 8), (2, 1, 2), (3, 2, 4)):
            y = _run_p(L, x, w, b, add, "conv3x3p=%d,%d,%d,%d" % (bn, per_sm, na, nb_))
            assert np.all(np.isfinite(y)), (bn, per_sm, na, nb_)
            err = rel_l2(y, ref)
            assert err <= TOL[nb.MATH_TF32], (bn, per_sm, na, nb_, err)
            # the same MMAs in the same order as the one-tile kernel with this tile width: the same bits
            if bn == bn_full:
                assert np.array_equal(y.view(np.uint32), one_tile.view(np.uint32)), (bn, per_sm, na, nb_)


@pytest.mark.parametrize("shape", [
    # C, K, H, W, bias + ReLU6, addend
    (64, 64, 200, 100, True, False),    # 169 patches for 148 CTAs: some CTAs walk two patches (both accumulators, ring wrap)
    (32, 128, 150, 90, False, False),   # one channel block, channel tile 128
    (64, 96, 57, 59, True, False),      # ragged patches; the slice fits at a channel tile of 64 only: two tiles, the second half full
    (128, 40, 40, 30, True, False),     # four channel blocks (36 weight tiles), channel tile 32, K = 40 clipped by the store
    (64, 20, 100, 9, False, False),     # K = 20
    (64, 64, 40, 24, True, True),       # a residual addend: the layer stays on the one-tile kernel
])
def test_weights_stationary_form_matches_the_oracle(shape):
    """The weights-stationary 3x3 kernel (the channel tile's whole weight slice resident in shared memory, patches
    walked by one CTA per SM, write-out by TMA): against the oracle, and bit for bit against the one-tile kernel with
    the same channel tile, which issues the same MMAs in the same order."""
    C, K, H, W, epi, with_add = shape
    L = dict(op=0, C=C, K=K, R=3, S=3, stride=1, pad=1, groups=1, H=H, W=W, in0=-1, in1=-1, act=2 if epi else 1,
             has_bias=1 if epi else 0)
    rng = np.random.default_rng([11] + list(shape[:4]))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = (rng.standard_normal((K, C, 3, 3)) * np.sqrt(2.0 / (C * 9))).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32) if epi else None
    add = rng.uniform(-1, 1, (K, H, W)).astype(np.float32) if with_add else None
    ref = omodel.run_layer(L, x, w, b, add)
    y = _run_p(L, x, w, b, add, "conv3x3w=on")
    assert np.all(np.isfinite(y))
    assert rel_l2(y, ref) <= TOL[nb.MATH_TF32], rel_l2(y, ref)
    assert np.max(np.abs(y - ref)) <= 8 * TOL[nb.MATH_TF32] * np.max(np.abs(ref))
    bn = min(128, -(-K // 16) * 16)
    while 9 * (C // 32) * bn * 128 > 150 * 1024:
        bn -= 16
    one_tile = _run_p(L, x, w, b, add, "conv3x3w=off;conv3x3=1,%d,1" % bn)
    if with_add:                                           # another kernel took the layer: fp32 summation order apart
        assert rel_l2(y, one_tile) <= 1e-5
    else:
        assert np.array_equal(y.view(np.uint32), one_tile.view(np.uint32))
    again = _run_p(L, x, w, b, add, "conv3x3w=on")
    assert np.array_equal(y.view(np.uint32), again.view(np.uint32))
