"""GPU: continuous mode (kernel switching for warm inference).  A cold inference with the kernels
K_cold leaves K_warm prepared on the device; the following warm inferences execute K_warm only.
Every result must be bit-identical to a plain cold run with the same kernels, which the other
tests compare with the oracle."""
import numpy as np
import pytest
import torch

import workloads as wl
from oracle import model as omodel
from oracle import selection as osel
from paper_2206_07446_b200 import binding as nb
from paper_2206_07446_b200 import harness
from gpu_util import rel_l2

pytestmark = pytest.mark.gpu


def _model(layers, seed=0):
    ws, bs = wl.make_weights(layers, seed=seed)
    x = wl.make_input(layers, seed=seed)
    return harness.model_from_workload(layers, ws, bs, wl.weight_blob), ws, bs, x


@pytest.mark.parametrize("cold_pref,cold_cached,warm_pref", [
    ([nb.VAR_GEMM1X1, nb.VAR_IM2COL], 0, [nb.VAR_WINO_F2, nb.VAR_GEMM1X1, nb.VAR_IM2COL]),   # switch on the 3x3 layers
    ([nb.VAR_GEMM1X1, nb.VAR_IM2COL], 1, [nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL]),   # cold reads cached blobs: raw read late
    ([nb.VAR_WINO_F2, nb.VAR_GEMM1X1, nb.VAR_IM2COL], 0, [nb.VAR_DIRECT]),                 # warm kernels without a transform
    ([nb.VAR_GEMM1X1, nb.VAR_IM2COL], 0, [nb.VAR_GEMM1X1, nb.VAR_IM2COL]),                 # K_warm = K_cold: nothing to switch
])
def test_tiny_net_cold_then_warm_runs(cold_pref, cold_cached, warm_pref):
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=4)
    ref = omodel.run_model(layers, ws, bs, x)[-1]
    cold = model.default_choices(prefer=cold_pref, math=nb.MATH_TF32)
    if cold_cached:
        cold = [None if c is None else (c[0], c[1], 1 if osel.has_transform(c[0]) else 0) for c in cold]
        model.build_cached_blob(cold)
    warm = model.default_choices(prefer=warm_pref, math=nb.MATH_TF32)
    sw = nb.nnv_switch_set(model.plan, cold, warm)
    assert sw == osel.switch_set(cold, warm)

    y_cold_plain, _ = model.cold_run(x, cold, depth=0)
    y_warm_plain, _ = model.cold_run(x, warm, depth=0)
    y1, _ = model.cold_run_continuous(x, cold, warm)
    assert np.array_equal(y1, y_cold_plain)                       # the first inference runs K_cold
    assert rel_l2(y1[0], ref) <= 2e-3
    x2 = wl.make_input(layers, seed=5)
    ref2 = omodel.run_model(layers, ws, bs, x2)[-1]
    y2, _ = model.warm_run(x, warm)                               # second inference: waits for what is still being prepared
    assert np.array_equal(y2, y_warm_plain)
    y3, _ = model.warm_run(x2, warm)                              # third: everything resident
    assert rel_l2(y3[0], ref2) <= 2e-3
    y4, _ = model.warm_run(x, warm)                               # replayed graph, same input again
    assert np.array_equal(y4, y_warm_plain)
    assert nb.nnv_device_status() == 0


def test_resnet18_kernel_switching_timings():
    """Config 2: cold kernels from the measured table, warm kernels = least execution time.  The warm
    runs move no weights: their h2d byte counts are zero and nothing is transformed."""
    layers = wl.cfg2_resnet18()
    model, ws, bs, x = _model(layers)
    costs = model.profile(x, reps=2)
    cold = nb.nnv_select_kernels(model.plan, costs, 0)
    warm = nb.nnv_select_warm(model.plan, costs)
    assert warm == osel.select_warm(layers, costs)
    y_warm_plain, _ = model.cold_run(x, [None if w is None else (w[0], w[1], 0) for w in warm], depth=0)
    y1, _ = model.cold_run_continuous(x, cold, warm)
    y2, tm2 = model.warm_run(x, warm, want_timings=True)
    assert np.array_equal(y2, y_warm_plain)
    for i, L in enumerate(layers):
        if L["op"] == wl.OP_CONV:
            assert tm2[i]["h2d_bytes"] == 0 and tm2[i]["xform_bytes"] == 0
    y3, _ = model.warm_run(x, warm)
    assert np.array_equal(y3, y_warm_plain)
    ref = omodel.run_model(layers, ws, bs, x)[-1]
    assert rel_l2(y3[0], ref) <= 1e-2                             # 20 chained TF32 layers
