"""GPU parity: whole-model cold runs (host weights -> H2D -> transform -> exec, three streams),
pipeline-depth invariance, the cached bypass, and profiling + selection."""
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


def _choices(model, prefer, math):
    return model.default_choices(prefer=prefer, math=math)


@pytest.mark.parametrize("prefer,math,tol", [
    ([nb.VAR_DIRECT], nb.MATH_FP32, 1e-5),
    ([nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32, 2e-3),
    ([nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32, 2e-3),
    ([nb.VAR_WINO_F2, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_BF16, 2e-2),
])
def test_tiny_net_cold_run_matches_oracle(prefer, math, tol):
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=2)
    acts = omodel.run_model(layers, ws, bs, x)
    ch = _choices(model, prefer, math)
    y, _ = model.cold_run(x, ch, depth=2)
    assert np.all(np.isfinite(y))
    # end-to-end error accumulates over layers: twice the per-layer tolerance
    assert rel_l2(y[0], acts[-1]) <= tol
    for i in range(len(layers)):
        assert rel_l2(model.layer_output(i), acts[i]) <= tol, i


def test_cfg1_cold_run_each_variant():
    layers = wl.cfg1()
    model, ws, bs, x = _model(layers)
    ref = omodel.run_model(layers, ws, bs, x)[-1]
    for v, m, tol in [(nb.VAR_DIRECT, 0, 1e-5), (nb.VAR_IM2COL, 1, 1e-3), (nb.VAR_WINO_F2, 1, 1e-3),
                      (nb.VAR_IM2COL, 2, 1e-2), (nb.VAR_WINO_F2, 2, 1e-2)]:
        y, tm = model.cold_run(x, [(v, m, 0)], depth=1, want_timings=True)
        assert rel_l2(y[0], ref) <= tol, (v, m)
        assert tm[0]["h2d_bytes"] == 64 * 64 * 9 * 4
        assert tm[0]["choice"] == (v, m, 0)


def test_resnet18_cold_run_pipeline_depths_bitwise_equal_and_ordered():
    """Config 2 end to end; the pipelined result is bitwise the serial one for depth 1..4, and the
    recorded stamps obey the dependency constraints (no operation starts before its precursors end)."""
    layers = wl.cfg2_resnet18()
    model, ws, bs, x = _model(layers)
    acts = omodel.run_model(layers, ws, bs, x)
    ch = _choices(model, [nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    outs = []
    for depth in (1, 2, 3, 4):
        y, tm = model.cold_run(x, ch, depth=depth, want_timings=True)
        outs.append(y.copy())
        conv = [i for i, L in enumerate(layers) if L["op"] == wl.OP_CONV]
        slack = 2000      # event stamps have 0.5 us resolution; allow 2 us
        for j, i in enumerate(conv):
            t = tm[i]
            assert t["h2d_end_ns"] >= t["h2d_start_ns"] and t["exec_end_ns"] >= t["exec_start_ns"]
            if t["xform_bytes"]:
                assert t["xform_start_ns"] + slack >= t["h2d_end_ns"]
                assert t["exec_start_ns"] + slack >= t["xform_end_ns"]
            else:
                assert t["exec_start_ns"] + slack >= t["h2d_end_ns"]
            for src in (layers[i]["in0"], layers[i]["in1"]):
                if src >= 0:
                    assert t["exec_start_ns"] + slack >= tm[src]["exec_end_ns"]
            if j >= depth:
                assert t["h2d_start_ns"] + slack >= tm[conv[j - depth]]["exec_end_ns"]
    for y in outs[1:]:
        assert np.array_equal(y.view(np.uint32), outs[0].view(np.uint32))
    assert rel_l2(outs[0][0], acts[-1]) <= 5e-3          # 20 TF32 layers chained


def test_resident_run_equals_cold_run_bitwise():
    """With the read stage already done the result is bit-identical to the run that copies from the host."""
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=6)
    ch = _choices(model, [nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    y_cold, _ = model.cold_run(x, ch, depth=2)
    for depth in (1, 3):
        y_res, tm = model.resident_run(x, ch, depth=depth, want_timings=True)
        assert np.array_equal(y_cold.view(np.uint32), y_res.view(np.uint32))
        assert all(t["h2d_bytes"] == 0 for t in tm)


def test_depth_zero_and_grouped_transforms_give_the_same_bits():
    """depth 0 (own buffers per layer, no staging waits; in the resident run the transforms become two
    multi-layer launches) changes scheduling only."""
    for layers, seed in ((wl.tiny_net(), 8), (wl.cfg2_resnet18(), 0)):
        model, ws, bs, x = _model(layers, seed=seed)
        ch = _choices(model, [nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
        y1, _ = model.cold_run(x, ch, depth=1)
        y0, tm0 = model.cold_run(x, ch, depth=0, want_timings=True)
        yr, tmr = model.resident_run(x, ch, depth=0, want_timings=True)
        yg, _ = model.resident_run(x, ch, depth=0)            # graph replay path
        assert np.array_equal(y1.view(np.uint32), y0.view(np.uint32))
        assert np.array_equal(y1.view(np.uint32), yr.view(np.uint32))
        assert np.array_equal(y1.view(np.uint32), yg.view(np.uint32))
        groups = {(t["xform_start_ns"], t["xform_end_ns"]) for t in tmr if t["xform_bytes"]}
        assert 1 <= len(groups) <= 3                           # three multi-layer launches at most


def test_transform_all_equals_per_layer_transforms():
    layers = wl.cfg2_resnet18()
    model, ws, bs, x = _model(layers)
    model.to_device()
    for prefer, math in (([nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32),
                         ([nb.VAR_WINO_F2, nb.VAR_IM2COL], nb.MATH_BF16), ([nb.VAR_WINO_F6, nb.VAR_IM2COL], nb.MATH_TF32)):
        ch = _choices(model, prefer, math)
        offs, total = nb.nnv_transformed_layout(model.plan, ch)
        out = harness.dev_bytes(total)
        nb.nnv_transform_all(model.plan, ch, model.d_weights, model.w_bytes, out, total, torch.cuda.current_stream())
        torch.cuda.synchronize()
        for i, c in enumerate(ch):
            if c is None or c[0] in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
                continue
            tb = nb.nnv_transformed_bytes(model.plan, i, c[0], c[1])
            one = harness.dev_bytes(tb)
            L = layers[i]
            rb = 4 * L["K"] * L["C"] * L["R"] * L["S"]
            nb.nnv_transform_weights(model.plan, i, c[0], c[1], model.d_weights[model.w_off[i]:model.w_off[i] + rb], one,
                                     torch.cuda.current_stream())
            torch.cuda.synchronize()
            assert torch.equal(out[offs[i]:offs[i] + tb], one[:tb]), (i, c)


def test_cached_bypass_gives_identical_result():
    """Reading cached post-transform weights and skipping the transform changes nothing in the output."""
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=4)
    ch = _choices(model, [nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    y_raw, _ = model.cold_run(x, ch, depth=2)
    ch_c = [None if c is None else (c[0], c[1], 1 if c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else 0) for c in ch]
    model.build_cached_blob(ch_c)
    y_c, tm = model.cold_run(x, ch_c, depth=2, want_timings=True)
    assert np.array_equal(y_raw.view(np.uint32), y_c.view(np.uint32))
    for i, c in enumerate(ch_c):
        if c is not None and c[2]:
            assert tm[i]["xform_bytes"] == 0
            assert tm[i]["h2d_bytes"] >= nb.nnv_transformed_bytes(model.plan, i, c[0], c[1])


def test_profile_then_select_matches_oracle_selection():
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=5)
    costs = model.profile(x, reps=3)
    n_expected = sum(len(osel.math_modes(v)) for L in layers if L["op"] == 0 for v in osel.eligible(L))
    assert len(costs) == n_expected
    assert all(c["exec_ns"] > 0 and c["h2d_raw_ns"] > 0 for c in costs)
    for allow in (0, 1):
        got = nb.nnv_select_kernels(model.plan, costs, allow)
        assert got == osel.select_kernels(layers, costs, allow)
    # the selected plan runs and matches the oracle
    ch = nb.nnv_select_kernels(model.plan, costs, 0)
    acts = omodel.run_model(layers, ws, bs, x)
    y, _ = model.cold_run(x, ch, depth=2)
    assert rel_l2(y[0], acts[-1]) <= 2e-2


def test_arena_too_small_and_bad_depth():
    layers = wl.cfg1()
    model, ws, bs, x = _model(layers)
    ch = [(nb.VAR_IM2COL, 1, 0)]
    need = model.ensure_arena(ch, 1)
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_cold_run(model.plan, ch, model.h_weights, model.w_bytes, None, 0, model.h_input, model.h_output,
                        model.arena, need - 1024, model.streams[0], model.streams[1], model.streams[2], 1)
    assert e.value.status == 4
    with pytest.raises(nb.NnvError) as e:
        nb.nnv_cold_run(model.plan, ch, model.h_weights, model.w_bytes, None, 0, model.h_input, model.h_output,
                        model.arena, need, model.streams[0], model.streams[1], model.streams[2], -1)
    assert e.value.status == 1


def test_residual_branch_layers_on_the_side_stream():
    """ResNet-18-shaped: the 1x1 downsample convs run on the plan's side stream beside the main branch.  Same
    result bit for bit as with everything on the execution stream, and every consumer of a side layer
    starts after that layer has ended."""
    import os
    layers = wl.cfg2_resnet18()
    model, ws, bs, x = _model(layers)
    ch = _choices(model, [nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    side = [i for i, L in enumerate(layers) if L["op"] == wl.OP_CONV and any(M["in1"] == i for M in layers)
            and not any(M["in0"] == i for M in layers)]
    assert len(side) == 3
    y_side, tm = model.cold_run(x, ch, depth=0, want_timings=True)
    for i in side:
        for j, M in enumerate(layers):
            if M["in1"] == i:
                assert tm[j]["exec_start_ns"] >= tm[i]["exec_end_ns"], (i, j)
        assert tm[i]["exec_start_ns"] >= tm[layers[i]["in0"]]["exec_end_ns"]
    nb.nnv_tuning_set("side=0")
    try:
        y_main, _ = model.cold_run(x, ch, depth=0, want_timings=True)
    finally:
        nb.nnv_tuning_set(None)
    assert np.array_equal(y_side, y_main)
    y_graph, _ = model.cold_run(x, ch, depth=0)
    assert np.array_equal(y_graph, y_side)


def test_merged_copies_at_depth_zero():
    """ResNet-18-shaped, depth 0: consecutive layers whose host and device ranges line up are read by one copy.
    Same result bit for bit as with one copy per layer; layers of one chunk report the same copy interval, the
    byte counts stay per layer, and no layer executes before its chunk has landed."""
    import os
    layers = wl.cfg2_resnet18()
    model, ws, bs, x = _model(layers)
    ch = _choices(model, [nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    y_merged, tm = model.cold_run(x, ch, depth=0, want_timings=True)
    convs = [i for i, L in enumerate(layers) if L["op"] == wl.OP_CONV]
    intervals = {(tm[i]["h2d_start_ns"], tm[i]["h2d_end_ns"]) for i in convs}
    assert len(intervals) < len(convs)                     # some layers share a copy
    for i in convs:
        L = layers[i]
        assert tm[i]["h2d_bytes"] == 4 * L["K"] * L["C"] * L["R"] * L["S"]
        assert tm[i]["exec_start_ns"] >= tm[i]["h2d_end_ns"]
    nb.nnv_tuning_set("merge=0")
    try:
        y_single, tm1 = model.cold_run(x, ch, depth=0, want_timings=True)
    finally:
        nb.nnv_tuning_set(None)
    assert len({(tm1[i]["h2d_start_ns"], tm1[i]["h2d_end_ns"]) for i in convs}) == len(convs)
    assert np.array_equal(y_merged, y_single)


def test_kernel_stamps_measure_without_changing_the_result():
    """A plan with kernel_stamps = 1: the tensor-core and transform kernels write device-clock stamps; the
    result is bit for bit that of a plan without them, every stamped duration is positive and none is longer
    than the whole run, and layers executed by the fp32 kernels report none."""
    layers = wl.cfg2_resnet18()
    ws, bs = wl.make_weights(layers)
    x = wl.make_input(layers)
    plain = harness.model_from_workload(layers, ws, bs, wl.weight_blob, use_graphs=0)
    stamped = harness.model_from_workload(layers, ws, bs, wl.weight_blob, use_graphs=0, kernel_stamps=1)
    ch = _choices(plain, [nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    ch[0] = (nb.VAR_DIRECT, nb.MATH_FP32, 0)
    y0, _ = plain.cold_run(x, ch, depth=0)
    with pytest.raises(nb.NnvError):
        nb.nnv_kernel_times(plain.plan)
    for depth in (0, 2):
        y1, tm = stamped.cold_run(x, ch, depth=depth, want_timings=True)
        assert np.array_equal(y0.view(np.uint32), y1.view(np.uint32))
        xf, ex = nb.nnv_kernel_times(stamped.plan)
        total = max(t["exec_end_ns"] for t in tm)
        convs = [i for i, L in enumerate(layers) if L["op"] == wl.OP_CONV]
        assert ex[0] == 0                                      # the direct kernel is no tensor-core launch
        assert depth == 0 or xf[0] == 0                        # (at depth 0 layer 0 books the grouped transform of its chunk)
        for i in convs[1:]:
            assert 0 < ex[i] < total, (i, ex[i], total)
            # the stamps lie inside the event interval around the layer (1 us of slack for the two clocks)
            assert ex[i] <= tm[i]["exec_end_ns"] - tm[i]["exec_start_ns"] + 1000, (i, ex[i], tm[i])
        assert sum(1 for i in convs if xf[i] > 0) >= 1 and all(v < total for v in xf)
        if depth:                                              # one transform launch per layer
            assert all(xf[i] > 0 for i in convs[1:])
        # the same stamps as a timeline: same durations, the earliest start is 0, a layer's GEMM starts after the
        # transform that produced its weights has ended, and the main branch executes in layer order
        spans = nb.nnv_kernel_spans(stamped.plan)
        assert [b - a for (a, b), _ in spans] == xf and [d - c for _, (c, d) in spans] == ex
        starts = [a for (a, b), _ in spans if b] + [c for _, (c, d) in spans if d]
        assert min(starts) == 0
        last_xf_end = 0
        for i in convs:
            (a, b), (c, d) = spans[i]
            last_xf_end = b if b else last_xf_end              # a grouped launch is booked on its first layer
            if i == convs[0]:
                continue                                       # (executed by the fp32 kernel: no stamp)
            assert c >= last_xf_end > 0, (i, spans[i], last_xf_end)
            if depth:
                assert c >= b > a, (i, spans[i])


def test_zero_copy_arm_is_bitwise_the_raw_arm():
    """The third preparation arm: the transform kernels read the raw weights in place in pinned host memory.  Same
    kernels, same arithmetic, same bytes out: the result equals the copy-then-transform run bit for bit at every
    depth, on the scheduled queues and fed from a model file; only biases are still copied; layers without a
    transform cannot take the arm."""
    layers = wl.tiny_net()
    model, ws, bs, x = _model(layers, seed=4)
    raw = _choices(model, [nb.VAR_WINO_F4, nb.VAR_GEMM1X1, nb.VAR_IM2COL], nb.MATH_TF32)
    zc = [None if c is None else (c[0], c[1], nb.ARM_ZERO_COPY if c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else 0) for c in raw]
    assert any(c is not None and c[2] == nb.ARM_ZERO_COPY for c in zc)
    y_raw, _ = model.cold_run(x, raw, depth=2)
    for depth in (0, 1, 3):
        y, tm = model.cold_run(x, zc, depth=depth, want_timings=True)
        assert np.array_equal(y.view(np.uint32), y_raw.view(np.uint32)), depth
        for i, L in enumerate(layers):
            if zc[i] is None:
                continue
            if zc[i][2] == nb.ARM_ZERO_COPY:
                assert tm[i]["choice"][2] == nb.ARM_ZERO_COPY
                assert tm[i]["h2d_bytes"] == (4 * L["K"] if L["has_bias"] else 0)        # no weight copy
                assert tm[i]["xform_bytes"] > 0 and tm[i]["exec_start_ns"] >= tm[i]["xform_end_ns"]
            else:
                assert tm[i]["h2d_bytes"] >= 4 * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"]
    q = [(-1 if c is None else (i % 3)) for i, c in enumerate(zc)]
    q[next(i for i, c in enumerate(zc) if c is not None)] = 0
    y_q, _ = model.cold_run_queues(x, zc, q, 2)
    assert np.array_equal(y_q.view(np.uint32), y_raw.view(np.uint32))
    bad = list(zc)
    dw = next((i for i, c in enumerate(raw) if c is not None and c[0] in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE)), None)
    if dw is not None:
        bad[dw] = (raw[dw][0], raw[dw][1], nb.ARM_ZERO_COPY)
        with pytest.raises(nb.NnvError):
            model.cold_run(x, bad, depth=0)
    # a larger model: ResNet-18-shaped, mixed arms picked by the selection on the profiled table
    layers = wl.cfg2_resnet18()
    model, ws, bs, x = _model(layers)
    costs = model.profile(x, reps=3)
    assert all(c["zc_ns"] > 0 for c in costs if c["variant"] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE))
    mixed = nb.nnv_select_kernels(model.plan, costs, 2)
    same_raw = [None if c is None else (c[0], c[1], 0) for c in mixed]
    y_m, _ = model.cold_run(x, mixed, depth=0)
    y_r, _ = model.cold_run(x, same_raw, depth=0)
    assert np.array_equal(y_m.view(np.uint32), y_r.view(np.uint32))
    print("zero-copy layers chosen:", sum(1 for c in mixed if c is not None and c[2] == nb.ARM_ZERO_COPY), "of",
          sum(1 for c in mixed if c is not None))
