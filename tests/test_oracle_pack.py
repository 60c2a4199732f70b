"""Pins for oracle/pack.py (CPU only)."""
import itertools

import numpy as np
import pytest
import torch

from oracle import pack as op


@pytest.mark.parametrize("C,K,R", [(c, k, r) for c in (1, 3, 4, 5, 8, 9) for k in (1, 3, 8, 9) for r in (1, 3, 7)])
def test_pack_is_a_bijection_with_zero_padding(C, K, R):
    """Brute force: (k,c,r,s) -> offset is injective, its image plus the pad set is the
    whole array, pad entries are +0.0 and every weight lands at its offset bit-exactly."""
    S = R
    Qp = op.padded_q(C, R, S)
    assert Qp % 8 == 0 and 0 <= Qp - R * S * C < 8
    offs = {}
    for k, c, r, s in itertools.product(range(K), range(C), range(R), range(S)):
        o = op.pack_offset(k, c, r, s, C, R, S)
        assert 0 <= o < K * Qp and o not in offs
        offs[o] = (k, c, r, s)
    w = (np.arange(K * C * R * S, dtype=np.float32) + 1.0).reshape(K, C, R, S)   # all non-zero, distinct
    P = op.pack_weights(w).reshape(-1)
    bits = P.view(np.uint32)
    for o in range(K * Qp):
        if o in offs:
            assert P[o] == op.tf32_round_rne(w)[offs[o]]
        else:
            assert bits[o] == 0                      # +0.0 exactly
    assert len(offs) == K * C * R * S


def test_pack_order_channel_innermost_then_taps():
    w = np.zeros((2, 3, 3, 3), np.float32)
    w[1, 2, 0, 1] = 5.0
    P = op.pack_weights(w)
    assert P.shape == (2, 32)
    assert P[1, (0 * 3 + 1) * 3 + 2] == 5.0 and np.count_nonzero(P) == 1


def test_tf32_rne_hand_patterns():
    """TF32 keeps 10 explicit mantissa bits: spacing 2^-10 in [1,2)."""
    f = lambda v: float(op.tf32_round_rne(np.array([v], np.float32))[0])
    assert f(1.0) == 1.0 and f(-3.5) == -3.5 and f(0.0) == 0.0
    assert f(1.0 + 2.0 ** -11) == 1.0                       # exact tie -> even (down)
    assert f(1.0 + 3 * 2.0 ** -11) == 1.0 + 2.0 ** -9       # exact tie -> even (up)
    assert f(1.0 + 2.0 ** -11 + 2.0 ** -22) == 1.0 + 2.0 ** -10
    assert f(2049.0) == 2048.0 and f(2051.0) == 2052.0
    rng = np.random.default_rng(12)
    a = rng.standard_normal(10000).astype(np.float32)
    r = op.tf32_round_rne(a)
    assert np.all(r.view(np.uint32) & 0x1FFF == 0)
    assert np.max(np.abs(r - a) / np.abs(a)) <= 2.0 ** -11
    assert np.array_equal(op.tf32_round_rne(r), r)          # idempotent


def test_bf16_rne_hand_patterns():
    cases = [
        (1.0, 0x3F80),
        (1.0 + 2.0 ** -8, 0x3F80),            # exact tie -> even (down)
        (1.0 + 3 * 2.0 ** -8, 0x3F82),        # exact tie -> even (up)
        (1.0 + 2.0 ** -8 + 2.0 ** -20, 0x3F81),   # just above the tie -> up
        (-2.5, 0xC020),
        (0.0, 0x0000),
        (3.0e-39, None),                      # subnormal fp32: compare with the library only
    ]
    for v, bits in cases:
        got = int(op.bf16_bits_rne(np.array([v], np.float32))[0])
        if bits is not None:
            assert got == bits, (v, hex(got))


def test_bf16_rne_vs_library_conversion():
    rng = np.random.default_rng(9)
    a = np.concatenate([rng.standard_normal(20000).astype(np.float32) * s for s in (1e-3, 1.0, 1e4)])
    got = op.bf16_bits_rne(a)
    ref = torch.from_numpy(a).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, ref)
    back = op.bf16_to_f32(got)
    assert np.max(np.abs(back - a) / np.abs(a)) <= 2.0 ** -8


def test_pack_rounding_is_applied_to_the_permuted_raw_weights():
    rng = np.random.default_rng(10)
    w = rng.standard_normal((5, 3, 3, 3)).astype(np.float32)
    assert np.array_equal(op.pack_weights(w, bf16=True), op.bf16_bits_rne(op.permute_weights(w)))
    assert np.array_equal(op.pack_weights(w), op.tf32_round_rne(op.permute_weights(w)))
