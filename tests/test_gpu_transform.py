"""GPU parity: weight transformation kernels against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import pack as opack
from oracle import winograd as owin
from paper_2206_07446_b200 import binding as nb
from gpu_util import dev, poisoned

pytestmark = pytest.mark.gpu

WINO = {2: nb.VAR_WINO_F2, 4: nb.VAR_WINO_F4, 6: nb.VAR_WINO_F6}


def _layer(C, K, R=3, stride=1, H=8, W=8):
    return dict(op=0, C=C, K=K, R=R, S=R, stride=stride, pad=R // 2, groups=1, H=H, W=W, in0=-1, in1=-1, act=0, has_bias=0)


def _weights(K, C, R, seed):
    rng = np.random.default_rng([seed, K, C, R])
    return (rng.standard_normal((K, C, R, R)) * np.sqrt(2.0 / (C * R * R))).astype(np.float32)


@pytest.mark.parametrize("m", [2, 4, 6])
@pytest.mark.parametrize("K,C", [(64, 64), (5, 3), (13, 20), (192, 64), (64, 3), (1, 1), (300, 136), (512, 512)])
def test_filter_transform_fp32(m, K, C):
    """max |U_gpu - U_ref| / max |U_ref| <= 1e-5 (fp32 FFMA against the fp64 literal G g G^T)."""
    plan = nb.Plan([_layer(C, K)], [0], [0])
    w = _weights(K, C, 3, m)
    Cp = -(-C // 8) * 8
    ref = owin.pad_channels(owin.filter_transform(w, m), Cp)
    nbytes = nb.nnv_transformed_bytes(plan, 0, WINO[m], nb.MATH_TF32)
    assert nbytes == ref.size * 4
    d_out = poisoned(nbytes)
    nb.nnv_transform_weights(plan, 0, WINO[m], nb.MATH_TF32, dev(w), d_out, torch.cuda.current_stream())
    torch.cuda.synchronize()
    got = d_out[:nbytes].view(torch.float32).cpu().numpy().reshape(ref.shape)
    assert np.all(np.isfinite(got))
    err = np.max(np.abs(got.astype(np.float64) - ref)) / np.max(np.abs(ref))
    assert err <= 1e-5, err
    if Cp != C:                                       # channel padding is exactly +0
        assert np.all(got[:, :, C:].view(np.uint32) == 0)


@pytest.mark.parametrize("m", [2])
@pytest.mark.parametrize("K,C", [(64, 64), (13, 20), (64, 3), (256, 256)])
def test_filter_transform_bf16(m, K, C):
    """bf16 U equals RNE-to-bf16 of the oracle except for rare 1-ulp double-rounding differences."""
    plan = nb.Plan([_layer(C, K)], [0], [0])
    w = _weights(K, C, 3, 10 + m)
    Cp = -(-C // 8) * 8
    ref = owin.pad_channels(owin.filter_transform(w, m), Cp)
    ref_bits = opack.bf16_bits_rne(ref.astype(np.float32)).astype(np.int32)
    nbytes = nb.nnv_transformed_bytes(plan, 0, WINO[m], nb.MATH_BF16)
    assert nbytes == ref.size * 2
    d_out = poisoned(nbytes)
    nb.nnv_transform_weights(plan, 0, WINO[m], nb.MATH_BF16, dev(w), d_out, torch.cuda.current_stream())
    torch.cuda.synchronize()
    got_bits = d_out[:nbytes].view(torch.int16).cpu().numpy().view(np.uint16).astype(np.int32).reshape(ref.shape)
    diff = np.abs(got_bits - ref_bits)
    # values straddling zero may differ in sign bit only when both are (sub)tiny; compare magnitudes there
    bad = diff > 1
    if np.any(bad):
        g = opack.bf16_to_f32(got_bits[bad].astype(np.uint16))
        r = opack.bf16_to_f32(ref_bits[bad].astype(np.uint16))
        assert np.max(np.abs(g - r)) <= 1e-6 * np.max(np.abs(ref)), "bf16 values differ by more than one ulp"
    assert np.mean(diff != 0) <= 1e-3


@pytest.mark.parametrize("K,C,R", [(64, 64, 3), (64, 3, 7), (5, 3, 3), (9, 5, 1), (24, 144, 1), (1280, 320, 1),
                                   (128, 64, 1), (7, 1000, 3), (512, 512, 3), (3, 2, 5)])
@pytest.mark.parametrize("bf16", [False, True])
def test_pack_is_bit_exact(K, C, R, bf16):
    """The repack is a pure permutation (+ zero pad, + RNE to bf16): byte-for-byte equal to the oracle."""
    variant = nb.VAR_GEMM1X1 if R == 1 else nb.VAR_IM2COL
    math = nb.MATH_BF16 if bf16 else nb.MATH_TF32
    L = _layer(C, K, R, H=max(8, R), W=max(8, R))
    if R == 1:
        L["pad"] = 0
    plan = nb.Plan([L], [0], [0])
    w = _weights(K, C, R, 3)
    ref = opack.pack_weights(w, bf16=bf16)
    nbytes = nb.nnv_transformed_bytes(plan, 0, variant, math)
    assert nbytes == ref.nbytes
    d_out = poisoned(nbytes)
    nb.nnv_transform_weights(plan, 0, variant, math, dev(w), d_out, torch.cuda.current_stream())
    torch.cuda.synchronize()
    got = d_out[:nbytes].cpu().numpy()
    assert np.array_equal(got, ref.view(np.uint8).reshape(-1))
    if R == 1:                                        # IM2COL on a 1x1 layer uses the same layout
        d2 = poisoned(nbytes)
        nb.nnv_transform_weights(plan, 0, nb.VAR_IM2COL, math, dev(w), d2, torch.cuda.current_stream())
        torch.cuda.synchronize()
        assert np.array_equal(d2[:nbytes].cpu().numpy(), got)


def test_transform_rejects_variants_without_transform():
    plan = nb.Plan([_layer(8, 8)], [0], [0])
    buf = poisoned(4096)
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_transform_weights(plan, 0, nb.VAR_DIRECT, nb.MATH_FP32, buf, buf, torch.cuda.current_stream())
    assert e.value.status == 2


def _random_banks(count, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        K = int(rng.choice([int(rng.integers(1, 40)), int(rng.integers(40, 700)), int(64 * rng.integers(1, 9))]))
        C = int(rng.choice([int(rng.integers(1, 40)), int(rng.integers(40, 700)), int(64 * rng.integers(1, 9))]))
        out.append((K, C))
    return out


@pytest.mark.parametrize("K,C", _random_banks(16, 31))
def test_random_filter_banks(K, C):
    """Seeded random filter-bank sizes (ragged and multiples of the kernels' block sizes alike): all three Winograd
    filter transforms to 1e-5 of the largest element, the 3x3 and 1x1 repacks byte for byte in both precisions."""
    w = _weights(K, C, 3, 77)
    plan = nb.Plan([_layer(C, K)], [0], [0])
    Cp = -(-C // 8) * 8
    for m in (2, 4, 6):
        ref = owin.pad_channels(owin.filter_transform(w, m), Cp)
        nbytes = nb.nnv_transformed_bytes(plan, 0, WINO[m], nb.MATH_TF32)
        d_out = poisoned(nbytes)
        nb.nnv_transform_weights(plan, 0, WINO[m], nb.MATH_TF32, dev(w), d_out, torch.cuda.current_stream())
        torch.cuda.synchronize()
        got = d_out[:nbytes].view(torch.float32).cpu().numpy().reshape(ref.shape)
        assert np.max(np.abs(got.astype(np.float64) - ref)) <= 1e-5 * np.max(np.abs(ref)), m
    for R in (3, 1):
        wr = _weights(K, C, R, 78)
        L = _layer(C, K, R)
        L["pad"] = R // 2
        planr = nb.Plan([L], [0], [0])
        variant = nb.VAR_GEMM1X1 if R == 1 else nb.VAR_IM2COL
        for bf16 in (False, True):
            math = nb.MATH_BF16 if bf16 else nb.MATH_TF32
            ref = opack.pack_weights(wr, bf16=bf16)
            nbytes = nb.nnv_transformed_bytes(planr, 0, variant, math)
            assert nbytes == ref.nbytes
            d_out = poisoned(nbytes)
            nb.nnv_transform_weights(planr, 0, variant, math, dev(wr), d_out, torch.cuda.current_stream())
            torch.cuda.synchronize()
            assert np.array_equal(d_out[:nbytes].cpu().numpy(), ref.view(np.uint8).reshape(-1)), (R, bf16)
