"""Pins for oracle/conv.py and oracle/model.py (CPU only)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import conv as oc
from oracle import model as om
import workloads as wl


@pytest.mark.parametrize("cfg", [
    # C, H, W, K, R, stride, pad, groups
    (3, 9, 11, 4, 3, 1, 1, 1),
    (4, 10, 7, 6, 3, 2, 1, 1),
    (3, 15, 15, 5, 7, 2, 3, 1),
    (6, 8, 8, 6, 3, 1, 1, 6),
    (6, 9, 8, 6, 3, 2, 1, 6),
    (8, 6, 5, 3, 1, 1, 0, 1),
    (8, 7, 5, 3, 1, 2, 0, 1),
    (4, 6, 6, 8, 3, 1, 0, 2),
])
def test_direct_conv_vs_library_fp64(cfg):
    """The C loops agree with torch's CPU conv2d in float64 (a library routine for the same definition)."""
    C, H, W, K, R, st, pad, g = cfg
    rng = np.random.default_rng(list(cfg))
    x = rng.uniform(-1, 1, (C, H, W)).astype(np.float32)
    w = rng.standard_normal((K, C // g, R, R)).astype(np.float32)
    b = rng.uniform(-1, 1, K).astype(np.float32)
    y = oc.direct_conv(x, w, b, st, pad, g)
    ref = F.conv2d(torch.from_numpy(x).double()[None], torch.from_numpy(w).double(),
                   torch.from_numpy(b).double(), stride=st, padding=pad, groups=g)[0].numpy()
    assert y.shape == ref.shape
    assert np.max(np.abs(y - ref)) < 1e-12
    y2 = oc.direct_conv_py(x, w, b, st, pad, g)
    assert np.max(np.abs(y - y2)) < 1e-12
    y3 = oc.direct_conv(x.astype(np.float64), w, b, st, pad, g)
    assert np.array_equal(y, y3)


def test_1x1_conv_is_matmul():
    rng = np.random.default_rng(3)
    x = rng.uniform(-1, 1, (16, 5, 7)).astype(np.float32)
    w = rng.standard_normal((9, 16, 1, 1)).astype(np.float32)
    y = oc.direct_conv(x, w)
    ref = w.reshape(9, 16).astype(np.float64) @ x.reshape(16, 35).astype(np.float64)
    assert np.max(np.abs(y.reshape(9, 35) - ref)) < 1e-13


def test_delta_filters_are_shifts():
    """A unit tap at (r,s) copies the input shifted by (r-pad, s-pad) with zero fill: pins
    the correlation (no flip) convention and the padding arithmetic."""
    rng = np.random.default_rng(4)
    x = rng.uniform(-1, 1, (1, 6, 7)).astype(np.float32)
    for r in range(3):
        for s in range(3):
            w = np.zeros((1, 1, 3, 3), np.float32)
            w[0, 0, r, s] = 1.0
            y = oc.direct_conv(x, w, None, 1, 1, 1)[0]
            want = np.zeros((6, 7))
            for oh in range(6):
                for ow in range(7):
                    ih, iw = oh + r - 1, ow + s - 1
                    if 0 <= ih < 6 and 0 <= iw < 7:
                        want[oh, ow] = x[0, ih, iw]
            assert np.array_equal(y, want)


def test_depthwise_is_per_channel_correlation():
    from scipy.signal import correlate2d
    rng = np.random.default_rng(5)
    x = rng.uniform(-1, 1, (4, 8, 9)).astype(np.float32)
    w = rng.standard_normal((4, 1, 3, 3)).astype(np.float32)
    y = oc.direct_conv(x, w, None, 1, 1, 4)
    for c in range(4):
        ref = correlate2d(x[c].astype(np.float64), w[c, 0].astype(np.float64), mode="same")
        assert np.max(np.abs(y[c] - ref)) < 1e-13


def test_output_size_floor_convention():
    assert oc.out_size(224, 224, 7, 7, 2, 3) == (112, 112)
    assert oc.out_size(112, 112, 3, 3, 2, 1) == (56, 56)
    assert oc.out_size(7, 8, 3, 3, 2, 1) == (4, 4)
    assert oc.out_size(6, 6, 3, 3, 2, 0) == (2, 2)


def test_glue_ops():
    x = np.arange(2 * 4 * 4, dtype=np.float64).reshape(2, 4, 4) - 10.0
    assert np.array_equal(oc.activation(x, 1), np.maximum(x, 0))
    assert oc.activation(x, 2).max() == 6.0 and oc.activation(x, 2).min() == 0.0
    assert np.array_equal(oc.activation(x, 0), x)
    mp = oc.maxpool(x, 2, 2, 0)
    assert np.array_equal(mp[0], np.array([[-5.0, -3.0], [3.0, 5.0]]))
    for (R, st, pad) in [(3, 2, 1), (2, 2, 0), (3, 1, 1)]:
        ref = F.max_pool2d(torch.from_numpy(x)[None], R, st, pad)[0].numpy()
        assert np.array_equal(oc.maxpool(x, R, st, pad), ref)
    ga = oc.gavgpool(x)
    assert ga.shape == (2, 1, 1) and ga[0, 0, 0] == x[0].mean() and ga[1, 0, 0] == x[1].mean()


def test_model_chain_matches_library_chain():
    """The whole-model walk (residual adds, activations, pools) against a torch fp64 chain."""
    layers = wl.tiny_net()
    ws, bs = wl.make_weights(layers, seed=7)
    x = wl.make_input(layers, seed=7)
    acts = om.run_model(layers, ws, bs, x)
    tacts = []
    tx = torch.from_numpy(x).double()
    for i, L in enumerate(layers):
        src = tx if L["in0"] < 0 else tacts[L["in0"]]
        if L["op"] == wl.OP_CONV:
            y = F.conv2d(src, torch.from_numpy(ws[i]).double(),
                         None if bs[i] is None else torch.from_numpy(bs[i]).double(),
                         stride=L["stride"], padding=L["pad"], groups=L["groups"])
            if L["in1"] >= 0:
                y = y + tacts[L["in1"]]
            if L["act"] == 1:
                y = torch.relu(y)
            elif L["act"] == 2:
                y = torch.clamp(y, 0, 6)
        elif L["op"] == wl.OP_MAXPOOL:
            y = F.max_pool2d(src, L["R"], L["stride"], L["pad"])
        else:
            y = src.mean(dim=(2, 3), keepdim=True)
        tacts.append(y)
    for a, t in zip(acts, tacts):
        assert a.shape == tuple(t.shape[1:])
        assert np.max(np.abs(a - t[0].numpy())) < 1e-12
