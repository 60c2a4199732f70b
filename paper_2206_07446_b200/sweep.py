"""Per-kernel timing sweeps through the C ABI (CUDA events, L2 flushed between repetitions).

  python -m paper_2206_07446_b200.sweep transform --m 4 --C 512 --K 512      (--m 0: GEMM repack)
  python -m paper_2206_07446_b200.sweep transform-sweep
  python -m paper_2206_07446_b200.sweep conv --variant wino_f4 --C 64 --K 64 --H 56
  python -m paper_2206_07446_b200.sweep conv-sweep
  python -m paper_2206_07446_b200.sweep transform-all --config cfg2_resnet18 --prefer wino_f4

Each line of output is one JSON record with the algorithmic bytes / flops of the operation, the
median duration and the achieved rate.  Weights and inputs are seeded random tensors created on
the device; nothing here checks results (the tests do).
"""
import argparse
import json
import statistics

import torch

from . import binding as nb

WINO = {2: nb.VAR_WINO_F2, 4: nb.VAR_WINO_F4, 6: nb.VAR_WINO_F6}
FLUSH_BYTES = 256 << 20


def _layer(C, K, R, stride, H, W, groups=1):
    return dict(op=0, C=C, K=K, R=R, S=R, stride=stride, pad=R // 2, groups=groups, H=H, W=W, in0=-1, in1=-1,
                act=1, has_bias=0)


def _buf(nbytes):
    t = torch.empty(max(256, int(nbytes)), dtype=torch.uint8, device="cuda")
    assert t.data_ptr() % 256 == 0
    return t


def _rand(nfloats, scale=1.0):
    return (torch.rand(max(64, int(nfloats)), device="cuda", dtype=torch.float32) * 2 - 1) * scale


def _time(fn, reps, flush):
    st = torch.cuda.current_stream()
    ts = []
    for r in range(reps + 2):
        if flush is not None:
            flush.fill_(r & 0xFF)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        fn(st)
        e1.record(st)
        e1.synchronize()
        if r >= 2:
            ts.append(e0.elapsed_time(e1) * 1e3)            # us
    return statistics.median(ts), min(ts)


def time_transform(variant, math, C, K, R=3, reps=20, flush=None):
    L = _layer(C, K, R, 1, 8, 8)
    if R == 1:
        L["pad"] = 0
    plan = nb.Plan([L], [0], [0])
    raw_bytes = 4 * K * C * R * R
    out_bytes = nb.nnv_transformed_bytes(plan, 0, variant, math)
    d_raw = _rand(K * C * R * R, 0.05)
    d_out = _buf(out_bytes)
    med, best = _time(lambda st: nb.nnv_transform_weights(plan, 0, variant, math, d_raw, d_out, st), reps, flush)
    return dict(op="transform", variant=nb.VARIANT_NAMES[variant], math=nb.MATH_NAMES[math], C=C, K=K, R=R,
                bytes=raw_bytes + out_bytes, us=med, us_min=best, gbs=(raw_bytes + out_bytes) / med / 1e3)


def time_conv(variant, math, C, K, R, stride, H, W, groups=1, reps=20, flush=None):
    L = _layer(C, K, R, stride, H, W, groups)
    if R == 1:
        L["pad"] = 0
    plan = nb.Plan([L], [0], [0])
    oh = (H + 2 * L["pad"] - R) // stride + 1
    ow = (W + 2 * L["pad"] - R) // stride + 1
    cg = C // groups
    d_raw = _rand(K * cg * R * R, 0.05)
    if variant in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
        d_wt = d_raw
    else:
        d_wt = _buf(nb.nnv_transformed_bytes(plan, 0, variant, math))
        nb.nnv_transform_weights(plan, 0, variant, math, d_raw, d_wt, torch.cuda.current_stream())
    d_in = _rand(C * H * W)
    d_out = _buf(4 * oh * ow * K)
    wsb = nb.nnv_exec_workspace_bytes(plan, 0, variant, math)
    d_ws = _buf(wsb) if wsb else None
    med, best = _time(lambda st: nb.nnv_conv_exec(plan, 0, variant, math, d_in, None, d_wt, None, d_out, d_ws, wsb, st),
                      reps, flush)
    flops = 2.0 * oh * ow * K * cg * R * R
    return dict(op="conv", variant=nb.VARIANT_NAMES[variant], math=nb.MATH_NAMES[math], C=C, K=K, R=R, stride=stride,
                H=H, W=W, groups=groups, direct_flops=flops, us=med, us_min=best, direct_tflops=flops / med / 1e6)


def time_transform_all(config, prefer, math, reps=20, flush=None):
    """Every layer's weight transform of one configuration in a single nnv_transform_all launch
    (run from the repository root: the layer shapes come from the top-level `workloads` module).
    Layers take the first eligible variant of `prefer`, then gemm1x1 / im2col."""
    import workloads as wl
    layers = wl.CONFIGS[config]()
    w_off, b_off, w_bytes = _offsets(layers)
    plan = nb.Plan(layers, w_off, b_off)
    choices = []
    for i, L in enumerate(layers):
        if L["op"] != nb.OP_CONV:
            choices.append(None)
            continue
        el = nb.nnv_eligible(plan, i)
        v = next((c for c in prefer + [nb.VAR_GEMM1X1, nb.VAR_IM2COL] if c in el), None)
        if v is None:
            v = nb.VAR_DEPTHWISE if nb.VAR_DEPTHWISE in el else el[0]
        m = nb.MATH_FP32 if v in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else (nb.MATH_TF32 if v in (nb.VAR_WINO_F4, nb.VAR_WINO_F6) else math)
        choices.append((v, m, 0))
    d_w = _rand(w_bytes // 4 + 64, 0.05)
    offs, total = nb.nnv_transformed_layout(plan, choices)
    d_out = _buf(total)
    med, best = _time(lambda st: nb.nnv_transform_all(plan, choices, d_w, w_bytes, d_out, total, st), reps, flush)
    raw = sum(4 * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"] for L, c in zip(layers, choices)
              if c is not None and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE))
    out = sum(nb.nnv_transformed_bytes(plan, i, c[0], c[1]) for i, c in enumerate(choices)
              if c is not None and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE))
    # the same bytes moved by a plain device copy, timed the same way: the ceiling of this measurement
    half = (raw + out) // 2
    a, b = _buf(half), _buf(half)
    cmed, _ = _time(lambda st: b.copy_(a, non_blocking=True), reps, flush)
    return dict(op="transform-all", config=config, prefer=[nb.VARIANT_NAMES[v] for v in prefer], math=nb.MATH_NAMES[math],
                bytes=raw + out, us=med, us_min=best, gbs=(raw + out) / med / 1e3, copy_same_bytes_us=cmed,
                copy_gbs=2 * half / cmed / 1e3)


def _offsets(layers):
    """Byte offsets of each layer's weights in a dense blob (256-byte aligned), no biases."""
    w_off, pos = [], 0
    for L in layers:
        w_off.append(pos)
        if L["op"] == nb.OP_CONV:
            pos += (4 * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"] + 255) // 256 * 256
    return w_off, [0] * len(layers), pos


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["transform", "transform-sweep", "conv", "conv-sweep", "transform-all"])
    ap.add_argument("--config", default="cfg2_resnet18")
    ap.add_argument("--prefer", default="", help="comma-separated variants tried first per layer (transform-all)")
    ap.add_argument("--m", type=int, default=4)
    ap.add_argument("--variant", default="wino_f4", choices=nb.VARIANT_NAMES)
    ap.add_argument("--math", default="tf32", choices=nb.MATH_NAMES)
    ap.add_argument("--C", type=int, default=512)
    ap.add_argument("--K", type=int, default=512)
    ap.add_argument("--R", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--H", type=int, default=56)
    ap.add_argument("--groups", type=int, default=1)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--no-flush", action="store_true")
    a = ap.parse_args()
    flush = None if a.no_flush else torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    math = nb.MATH_NAMES.index(a.math)
    if a.what == "transform":
        v = WINO[a.m] if (a.R == 3 and a.m in WINO) else nb.VAR_IM2COL      # --m 0: the repack of a 3x3 layer
        print(json.dumps(time_transform(v, math, a.C, a.K, a.R, a.reps, flush)))
    elif a.what == "transform-sweep":
        for m in (2, 4, 6):
            for n in (64, 128, 256, 512, 1024, 2048):
                print(json.dumps(time_transform(WINO[m], nb.MATH_TF32, n, n, 3, a.reps, flush)), flush=True)
        for n in (64, 256, 512, 1024):
            print(json.dumps(time_transform(nb.VAR_IM2COL, nb.MATH_TF32, n, n, 3, a.reps, flush)), flush=True)
            print(json.dumps(time_transform(nb.VAR_IM2COL, nb.MATH_BF16, n, n, 3, a.reps, flush)), flush=True)
    elif a.what == "transform-all":
        prefer = [nb.VARIANT_NAMES.index(v) for v in a.prefer.split(",") if v]
        print(json.dumps(time_transform_all(a.config, prefer, math, a.reps, flush)))
    elif a.what == "conv":
        v = nb.VARIANT_NAMES.index(a.variant)
        print(json.dumps(time_conv(v, math, a.C, a.K, a.R, a.stride, a.H, a.H, a.groups, a.reps, flush)))
    else:
        shapes = [(64, 64, 3, 1, 56), (128, 128, 3, 1, 28), (256, 256, 3, 1, 14), (512, 512, 3, 1, 7),
                  (64, 64, 3, 1, 224), (128, 128, 3, 1, 112), (256, 256, 3, 1, 56), (512, 512, 3, 1, 28),
                  (256, 256, 3, 1, 112), (256, 256, 3, 1, 224), (512, 512, 3, 1, 112)]   # beyond the configurations: the asymptote
        for (C, K, R, s, H) in shapes:
            for v, m in ((nb.VAR_DIRECT, 0), (nb.VAR_IM2COL, 1), (nb.VAR_IM2COL, 2), (nb.VAR_WINO_F2, 1),
                         (nb.VAR_WINO_F2, 2), (nb.VAR_WINO_F4, 1), (nb.VAR_WINO_F6, 1)):
                print(json.dumps(time_conv(v, m, C, K, R, s, H, H, 1, a.reps, flush)), flush=True)
        for (C, K, H) in [(64, 256, 56), (256, 64, 56), (512, 2048, 7), (2048, 512, 7), (320, 1280, 7), (16, 96, 112)]:
            for m in (1, 2):
                print(json.dumps(time_conv(nb.VAR_GEMM1X1, m, C, K, 1, 1, H, H, 1, a.reps, flush)), flush=True)
        for (C, s, H) in [(96, 2, 112), (384, 1, 14), (960, 1, 7)]:
            print(json.dumps(time_conv(nb.VAR_DEPTHWISE, 0, C, C, 3, s, H, H, C, a.reps, flush)), flush=True)


if __name__ == "__main__":
    main()
