"""GPU parity of the Winograd data transforms as single operations: the input transform V = B^T d B and the
output transform Y = A^T M A (+ bias, addend, activation), element by element against oracle/winograd.py."""
import numpy as np
import pytest
import torch

from oracle import conv as oconv
from oracle import winograd as owin
from paper_2206_07446_b200 import binding as nb
from gpu_util import dev, poisoned, chw_to_hwc, hwc_to_chw

pytestmark = pytest.mark.gpu

M_OF = {nb.VAR_WINO_F2: 2, nb.VAR_WINO_F4: 4, nb.VAR_WINO_F6: 6}
SHAPES = [  # C, K, H, W, pad
    (64, 64, 56, 56, 1), (5, 12, 9, 7, 1), (24, 40, 14, 14, 0), (3, 8, 33, 20, 1), (1, 1, 3, 3, 1), (130, 36, 13, 11, 1)]


def _layer(C, K, H, W, pad, act=0, bias=0):
    return dict(op=0, C=C, K=K, R=3, S=3, stride=1, pad=pad, groups=1, H=H, W=W, in0=-1, in1=-1, act=act, has_bias=bias)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("variant,math", [(nb.VAR_WINO_F2, nb.MATH_TF32), (nb.VAR_WINO_F2, nb.MATH_BF16),
                                          (nb.VAR_WINO_F4, nb.MATH_TF32), (nb.VAR_WINO_F6, nb.MATH_TF32)])
def test_input_transform_matches_oracle(shape, variant, math):
    C, K, H, W, pad = shape
    m = M_OF[variant]
    L = _layer(C, K, H, W, pad)
    plan = nb.Plan([L], [0], [0])
    rng = np.random.default_rng([31, m, math] + list(shape))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    V_ref, TH, TW = owin.input_transform(x, m, pad)                       # (alpha^2, T, C) fp64
    T, vb, mb = nb.nnv_wino_sizes(plan, 0, variant, math)
    assert T == TH * TW
    Cp = -(-C // 8) * 8
    es = 2 if math == nb.MATH_BF16 else 4
    assert vb == (m + 2) ** 2 * T * Cp * es and mb == (m + 2) ** 2 * T * K * 4
    d_V = poisoned(vb)
    nb.nnv_wino_input_transform(plan, 0, variant, math, dev(chw_to_hwc(x)), d_V, torch.cuda.current_stream())
    torch.cuda.synchronize()
    dt = torch.bfloat16 if math == nb.MATH_BF16 else torch.float32
    V = d_V[:vb].view(dt).reshape((m + 2) ** 2, T, Cp).float().cpu().numpy()
    assert np.all(V[:, :, C:] == 0) and not np.any(np.signbit(V[:, :, C:]))    # padded channels hold +0
    scale = np.max(np.abs(V_ref))
    # fp32 FFMA arithmetic: 1e-5; F(2,3) feeds one TF32 (or bf16) pass and is rounded to that precision on the way out
    tol = 2.0 ** -8 if math == nb.MATH_BF16 else (1.05 * 2.0 ** -11 if m == 2 else 1e-5)
    assert np.max(np.abs(V[:, :, :C] - V_ref)) <= tol * scale, np.max(np.abs(V[:, :, :C] - V_ref)) / scale


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("variant", [nb.VAR_WINO_F2, nb.VAR_WINO_F4, nb.VAR_WINO_F6])
@pytest.mark.parametrize("epi", [False, True])
def test_output_transform_matches_oracle(shape, variant, epi):
    C, K, H, W, pad = shape
    m = M_OF[variant]
    L = _layer(C, K, H, W, pad, act=2 if epi else 0, bias=1 if epi else 0)
    plan = nb.Plan([L], [0], [0])
    OH, OW = H + 2 * pad - 2, W + 2 * pad - 2
    TH, TW = -(-OH // m), -(-OW // m)
    rng = np.random.default_rng([32, m, int(epi)] + list(shape))
    Mt = rng.uniform(-1, 1, ((m + 2) ** 2, TH * TW, K)).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32) if epi else None
    add = rng.uniform(-3, 3, (K, OH, OW)).astype(np.float32) if epi else None
    ref = owin.output_transform(Mt.astype(np.float64), m, K, OH, OW, TH, TW)
    scale = np.max(np.abs(ref))
    if epi:
        ref = oconv.activation(ref + b[:, None, None] + add, 2)
    d_out = poisoned(4 * OH * OW * K)
    nb.nnv_wino_output_transform(plan, 0, variant, dev(Mt), dev(chw_to_hwc(add)) if epi else None, dev(b) if epi else None, d_out,
                                 torch.cuda.current_stream())
    torch.cuda.synchronize()
    y = hwc_to_chw(d_out[:4 * OH * OW * K].view(torch.float32).reshape(OH, OW, K).cpu().numpy())
    assert np.max(np.abs(y - ref)) <= 1e-5 * max(scale, 1.0), np.max(np.abs(y - ref))
