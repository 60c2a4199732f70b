"""Helpers shared by the GPU parity tests (no method arithmetic)."""
import numpy as np
import torch

from paper_2206_07446_b200 import binding as nb

TOL = {nb.MATH_FP32: 1e-5, nb.MATH_TF32: 1e-3, nb.MATH_BF16: 1e-2}   # relative L2 error of a conv output


def dev(arr):
    """numpy array -> 256-byte aligned CUDA tensor of the same dtype."""
    t = torch.from_numpy(np.ascontiguousarray(arr)).cuda()
    assert t.data_ptr() % 256 == 0
    return t


def poisoned(nbytes):
    t = torch.empty(max(256, int(nbytes)), dtype=torch.uint8, device="cuda")
    t.fill_(0xFF)
    return t


def chw_to_hwc(x):
    return np.ascontiguousarray(np.transpose(x, (1, 2, 0)))


def hwc_to_chw(x):
    return np.ascontiguousarray(np.transpose(x, (2, 0, 1)))


def rel_l2(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    den = np.sqrt(np.sum(ref * ref))
    return float(np.sqrt(np.sum((got - ref) ** 2)) / (den if den > 0 else 1.0))


def max_abs_rel(got, ref):
    """Largest element-wise error relative to the largest reference magnitude."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    den = float(np.max(np.abs(ref))) if ref.size else 0.0
    return float(np.max(np.abs(got - ref))) / (den if den > 0 else 1.0) if ref.size else 0.0


ELEMENTWISE_FACTOR = 8.0     # max |y - ref| <= 8 * tol * max |ref|: a norm alone would let single wrong outputs of a large layer through


def assert_conv_close(got, ref, tol, what=None):
    """The tolerance of a conv output: relative L2 error <= tol, and no single element off by more than
    ELEMENTWISE_FACTOR * tol of the largest reference magnitude."""
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    assert np.all(np.isfinite(got)), what
    err = rel_l2(got, ref)
    assert err <= tol, (what, "rel L2", err)
    worst = max_abs_rel(got, ref)
    assert worst <= ELEMENTWISE_FACTOR * tol, (what, "element-wise", worst)
    return err


def run_conv(plan, i, L, variant, math, x_chw, w, bias=None, addend_chw=None):
    """Transform (if the variant has one) and execute layer i through the C ABI; returns CHW numpy."""
    d_raw = dev(w.astype(np.float32))
    if variant in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
        d_wt = d_raw
    else:
        d_wt = poisoned(nb.nnv_transformed_bytes(plan, i, variant, math))
        nb.nnv_transform_weights(plan, i, variant, math, d_raw, d_wt, torch.cuda.current_stream())
    oh = (L["H"] + 2 * L["pad"] - L["R"]) // L["stride"] + 1
    ow = (L["W"] + 2 * L["pad"] - L["S"]) // L["stride"] + 1
    d_in = dev(chw_to_hwc(x_chw.astype(np.float32)))
    d_add = dev(chw_to_hwc(addend_chw.astype(np.float32))) if addend_chw is not None else None
    d_bias = dev(bias.astype(np.float32)) if bias is not None else None
    d_out = poisoned(4 * oh * ow * L["K"])
    wsb = nb.nnv_exec_workspace_bytes(plan, i, variant, math)
    d_ws = poisoned(wsb) if wsb else None
    nb.nnv_conv_exec(plan, i, variant, math, d_in, d_add, d_wt, d_bias, d_out, d_ws, wsb, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert nb.nnv_device_status() == 0
    y = d_out[:4 * oh * ow * L["K"]].view(torch.float32).reshape(oh, ow, L["K"]).cpu().numpy()
    return hwc_to_chw(y)
