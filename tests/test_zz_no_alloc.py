"""nnv_conv_exec_static: layer execution for callers that cannot allocate device scratch.

Some users of the library have no way to obtain a scratch buffer: they run inside an application
that owns all device memory, or in a loop where an allocation's device-wide synchronisation is not
acceptable.  For them the library carries a fixed scratch array.  This file checks, through the
C ABI, that the entry point gives the same result as nnv_conv_exec with a caller-provided buffer,
twice in a row (the second call finds the array dirty from the first), and that it refuses layers
whose scratch does not fit.  It is collected last so that a failure here cannot hide another test.
"""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import conv as oconv
from paper_2206_07446_b200 import binding as nb
from gpu_util import TOL, dev, poisoned, chw_to_hwc, hwc_to_chw, rel_l2, run_conv

pytestmark = pytest.mark.gpu


def _run_static(plan, i, L, variant, math, x_chw, w, addend_chw=None):
    d_raw = dev(w)
    d_wt = poisoned(nb.nnv_transformed_bytes(plan, i, variant, math))
    nb.nnv_transform_weights(plan, i, variant, math, d_raw, d_wt, torch.cuda.current_stream())
    oh, ow = wl.out_hw(L)
    d_in = dev(chw_to_hwc(x_chw))
    d_add = dev(chw_to_hwc(addend_chw)) if addend_chw is not None else None
    d_out = poisoned(4 * oh * ow * L["K"])
    nb.nnv_conv_exec_static(plan, i, variant, math, d_in, d_add, d_wt, None, d_out, torch.cuda.current_stream())
    torch.cuda.synchronize()
    assert nb.nnv_device_status() == 0
    return hwc_to_chw(d_out[:4 * oh * ow * L["K"]].view(torch.float32).reshape(oh, ow, L["K"]).cpu().numpy())


@pytest.mark.parametrize("variant,math", [(nb.VAR_WINO_F2, nb.MATH_TF32), (nb.VAR_WINO_F4, nb.MATH_TF32),
                                          (nb.VAR_WINO_F2, nb.MATH_BF16)])
def test_static_scratch_matches_conv_exec_on_two_calls_in_a_row(variant, math):
    layers = wl.cfg1()
    L = layers[0]
    plan = nb.Plan(layers, [0], [0])
    assert 0 < nb.nnv_exec_workspace_bytes(plan, 0, variant, math) <= nb.STATIC_SCRATCH_BYTES
    rng = np.random.default_rng(21)
    for call in range(2):                                  # second call: the shared array holds the first call's data
        x = rng.uniform(-1, 1, (L["C"], L["H"], L["W"])).astype(np.float32)
        w = (rng.standard_normal((L["K"], L["C"], 3, 3)) * 0.06).astype(np.float32)
        want = run_conv(plan, 0, L, variant, math, x, w)    # nnv_conv_exec with a caller-provided buffer
        got = _run_static(plan, 0, L, variant, math, x, w)
        assert np.all(np.isfinite(got))
        assert rel_l2(got, want) <= TOL[math], (call, rel_l2(got, want))
        ref = oconv.direct_conv(x, w, None, 1, 1, 1)
        assert rel_l2(np.maximum(ref, 0), got) <= TOL[math]


def test_static_scratch_refuses_layers_that_do_not_fit():
    L = dict(op=0, C=64, K=64, R=3, S=3, stride=1, pad=1, groups=1, H=224, W=224, in0=-1, in1=-1, act=1, has_bias=0)
    plan = nb.Plan([L], [0], [0])
    assert nb.nnv_exec_workspace_bytes(plan, 0, nb.VAR_WINO_F4, nb.MATH_TF32) > nb.STATIC_SCRATCH_BYTES
    buf = poisoned(1 << 20)
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_conv_exec_static(plan, 0, nb.VAR_WINO_F4, nb.MATH_TF32, buf, None, buf, None, buf, torch.cuda.current_stream())
    assert e.value.status == 4 and "scratch" in str(e.value)
