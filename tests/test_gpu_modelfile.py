"""GPU: cold runs fed from the model file (storage -> pinned memory -> HBM -> transform -> execute)
are bit-identical to cold runs fed from the host blob, for raw and cached choices."""
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


@pytest.mark.parametrize("cached", [0, 1])
@pytest.mark.parametrize("depth", [0, 2])
def test_tiny_net_from_file(tmp_path, cached, depth):
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=6)
    ch = model.default_choices(prefer=[nb.VAR_WINO_F2, nb.VAR_GEMM1X1, nb.VAR_IM2COL], math=nb.MATH_TF32)
    if cached:
        ch = [None if c is None else (c[0], c[1], 1 if osel.has_transform(c[0]) else 0) for c in ch]
        model.build_cached_blob(ch)
    want, _ = model.cold_run(x, ch, depth=depth)
    path = str(tmp_path / "tiny.nnv")
    model.write_model_file(path, ch)
    cache = nb.CacheFile(path)
    model.h_stage_w = torch.full((cache.w_bytes,), 0xFF, dtype=torch.uint8).pin_memory()      # nothing but the file fills these
    model.h_stage_c = torch.full((max(1, cache.c_bytes),), 0xFF, dtype=torch.uint8).pin_memory()
    got, tm, ns, nbytes = model.cold_run_file(x, ch, cache, depth=depth, want_timings=True)
    assert np.array_equal(got, want)
    expect = 0
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            continue
        c = ch[i]
        expect += nb.nnv_transformed_bytes(model.plan, i, c[0], c[1]) if c[2] else 4 * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"]
        expect += 4 * L["K"] if L["has_bias"] else 0
        assert tm[i]["h2d_bytes"] > 0
    assert nbytes == expect and ns > 0
    got2, _, _, _ = model.cold_run_file(x, ch, cache, depth=depth)
    assert np.array_equal(got2, want)
    ref = omodel.run_model(layers, ws, bs, x)[-1]
    assert rel_l2(got[0], ref) <= 2e-3
    assert nb.nnv_device_status() == 0


def test_file_with_other_cached_kernels_is_refused(tmp_path):
    layers = wl.cfg1()
    model, ws, bs, x = _model(layers)
    stored = [(nb.VAR_WINO_F2, nb.MATH_TF32, 1)]
    path = str(tmp_path / "c1.nnv")
    model.write_model_file(path, stored)
    cache = nb.CacheFile(path)
    y, _, _, _ = model.cold_run_file(x, stored, cache, depth=1)
    ref = omodel.run_model(layers, ws, bs, x)[-1]
    assert rel_l2(y[0], ref) <= 1e-3
    y_raw, _, _, _ = model.cold_run_file(x, [(nb.VAR_IM2COL, nb.MATH_TF32, 0)], cache, depth=1)   # raw arm of another kernel: fine
    assert rel_l2(y_raw[0], ref) <= 1e-3
    with pytest.raises(nb.NnvError) as e:
        model.cold_run_file(x, [(nb.VAR_IM2COL, nb.MATH_TF32, 1)], cache, depth=1)            # cached arm the file does not hold
    assert e.value.status == 1
