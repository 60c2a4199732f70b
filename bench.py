#!/usr/bin/env python
"""Benchmark of the cold-start convolution path on B200.

One step = one cold inference of the workload at batch 1, as the paper's Section 2 lists its stages:
every conv layer's RAW fp32 weights are read (pinned host memory -> HBM), transformed on the device
(Winograd filter transform or GEMM repack) and the layer is executed, pipelined over streams.  The
kernels come from the per-layer selection on the profiled cost table with the cached-weights bypass
switched OFF, and every call is enqueued eagerly (no recorded graph: a cold inference happens once).

  value   cold ms of that step with the model input / output in device memory (nnv_cold_run_dio):
          weights H2D + transform + execution inside the timed region, CUDA events
  e2e     the same step through nnv_cold_run with HOST input and output (their copies inside too)
  arms    beside them: the bypass arm (selection may take cached post-transform weights), the
          graph-replayed variant of the headline, and the device-resident pass (no read stage)
  roofline*  kernel durations come from the per-layer events of the TIMED headline steps

`python bench.py` (1 GPU) or under torch.distributed.run with --gpus N (independent replicas; the path
does not shard).  `--impl reference` times the CPU oracle instead.  `--kernel ...` times one kernel
(or a sweep of shapes) through the C ABI instead of a whole step.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads as wl  # noqa: E402

# DRAM bytes per tensor-core GEMM launch (dram__bytes_read.sum + dram__bytes_write.sum, averaged over the
# launches of one step) from an ncu capture of this command; the file under profiles/ gives the command.
# An entry is dropped (traffic = null) whenever the kernel changes after the capture.
NCU_GEMM_TRAFFIC_BYTES = {("cfg4_resnet50", "tf32"): 3380086}   # profiles/gemm_cfg4_dram_traffic.md

METRIC = "cold_inference_ms_batch1"
UNIT = "ms"
DEFAULT_CONFIG = "cfg4_resnet50"       # the largest configuration by bytes over the host link (94 MB raw weights)
FLUSH_BYTES = 256 << 20


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=list(wl.CONFIGS))
    ap.add_argument("--cold-depth", type=int, default=0, help="pipeline depth of the cold runs (staging slots; 0 = no limit)")
    ap.add_argument("--depth", type=int, default=3, help="pipeline depth of the device-resident pass")
    ap.add_argument("--math", default="tf32", choices=["tf32", "bf16"])
    ap.add_argument("--cpu-passes", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--arm-steps", type=int, default=20, help="timed steps of each side arm (bypass, graph replay, resident)")
    ap.add_argument("--depth-steps", type=int, default=10, help="timed steps per pipeline depth of the depth sweep (0 = skip)")
    ap.add_argument("--queues", type=int, default=2, help="preparation queues for the Algorithm 1 run (0 = skip)")
    ap.add_argument("--continuous-reps", type=int, default=10, help="cold + warm sequences for the kernel-switching report (0 = skip)")
    ap.add_argument("--file-reps", type=int, default=5, help="cold runs fed from a model file on local storage (0 = skip)")
    ap.add_argument("--also", default="cfg2_resnet18,cfg5_vgg16", help="other workloads measured beside --config (headline, e2e and rooflines only)")
    ap.add_argument("--minimal", action="store_true", help="headline + e2e + rooflines only (no side arms or sections)")
    ap.add_argument("--save-costs", default=None, help="write the profiled cost table (JSON) to this file")
    ap.add_argument("--load-costs", default=None, help="use a cost table saved earlier instead of profiling (e.g. under a profiler)")
    # single-kernel timing through the C ABI
    ap.add_argument("--kernel", default=None, choices=["transform", "transform-sweep", "conv", "conv-sweep", "transform-all"])
    ap.add_argument("--prefer", default="", help="comma-separated variants tried first per layer (--kernel transform-all)")
    ap.add_argument("--m", type=int, default=4, help="Winograd tile size of --kernel transform (0 = the GEMM repack)")
    ap.add_argument("--variant", default="im2col")
    ap.add_argument("--C", type=int, default=512)
    ap.add_argument("--K", type=int, default=512)
    ap.add_argument("--R", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--H", type=int, default=56)
    ap.add_argument("--W", type=int, default=0, help="image width of --kernel conv (0 = H)")
    ap.add_argument("--groups", type=int, default=1)
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--tuning", default=None, help="nnv_tuning_set specification applied before anything runs")
    return ap.parse_args()


def config_dict(args):
    """The workload description; identical for both arms (`--impl ours` and `--impl reference`)."""
    return {"workload": args.config, "batch": 1, "math": args.math,
            "weights": "raw fp32, He-normal, seed 0; every step reads, transforms and executes all of them",
            "l2": "GPU arm: flushed between steps by a 256 MiB device write"}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline and --impl reference)
def oracle_pass(layers, ws, bs, x):
    """One whole cold pass of the oracle: literal filter transform / naive pack per layer, then the
    fp64 direct-convolution chain.  Returns seconds."""
    from oracle import model as omodel
    from oracle import pack as opack
    from oracle import winograd as owin
    t0 = time.perf_counter()
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV or L["groups"] != 1:
            continue
        if L["R"] == 3 and L["S"] == 3 and L["stride"] == 1:
            owin.filter_transform(ws[i], 4)
        else:
            opack.pack_weights(ws[i])
    omodel.run_model(layers, ws, bs, x)
    return time.perf_counter() - t0


def cpu_threads():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


REFERENCE_BUDGET_S = 120.0        # wall-clock the reference arm may spend on its timed steps


def oracle_layer_pass(layers, ws, bs, acts_in, idx):
    """The oracle's cold work for the conv layers `idx` only (transform / pack + fp64 direct convolution),
    each fed the activation a full pass produced; returns seconds."""
    from oracle import model as omodel
    from oracle import pack as opack
    from oracle import winograd as owin
    t0 = time.perf_counter()
    for i in idx:
        L = layers[i]
        if L["groups"] == 1:
            if L["R"] == 3 and L["S"] == 3 and L["stride"] == 1:
                owin.filter_transform(ws[i], 4)
            else:
                opack.pack_weights(ws[i])
        src, add = acts_in[i]
        omodel.run_layer(L, src, ws[i], bs[i], add)
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import conv as oconv
    from oracle import model as omodel
    oconv.build()
    os.environ.setdefault("OMP_NUM_THREADS", str(cpu_threads()))
    layers = wl.CONFIGS[args.config]()
    ws, bs = wl.make_weights(layers)
    x = wl.make_input(layers)
    oracle_pass(layers, ws, bs, x)
    t_full = min(oracle_pass(layers, ws, bs, x) for _ in range(2))
    if args.steps * t_full <= REFERENCE_BUDGET_S:
        for _ in range(min(args.warmup, 2)):
            oracle_pass(layers, ws, bs, x)
        ts = [oracle_pass(layers, ws, bs, x) for _ in range(args.steps)]
        ms = 1e3 * sum(ts) / len(ts)
        sample = "whole %s workload per step: F(4,3) literal filter transform / naive pack of every conv layer + fp64 direct-conv chain" % args.config
    else:
        # Bounded sample: every `stride`-th conv layer per step, fed the activations of one full pass; the
        # step time is scaled by the share those layers have in a full pass's time (measured, not assumed).
        acts = omodel.run_model(layers, ws, bs, x)
        feed = {}
        convs = [i for i, L in enumerate(layers) if L["op"] == wl.OP_CONV]
        for i in convs:
            L = layers[i]
            src = x[0] if L["in0"] < 0 else acts[L["in0"]].astype(np.float32)
            add = None if L["in1"] < 0 else acts[L["in1"]].astype(np.float32)
            feed[i] = (src, add)
        stride = int(np.ceil(args.steps * t_full / REFERENCE_BUDGET_S))
        idx = convs[::stride] or convs[:1]
        t_all = min(oracle_layer_pass(layers, ws, bs, feed, convs) for _ in range(2))
        t_idx = min(oracle_layer_pass(layers, ws, bs, feed, idx) for _ in range(2))
        share = t_idx / t_all
        for _ in range(min(args.warmup, 2)):
            oracle_layer_pass(layers, ws, bs, feed, idx)
        ts = [oracle_layer_pass(layers, ws, bs, feed, idx) for _ in range(args.steps)]
        ms = 1e3 * (sum(ts) / len(ts)) / share
        sample = ("every %d-th conv layer of %s per step (%d of %d layers, %.1f %% of a full pass's time, which is %.0f ms), "
                  "scaled to the whole workload" % (stride, args.config, len(idx), len(convs), 100 * share, 1e3 * t_full))
    line = {
        "impl": "reference", "metric": METRIC, "value": ms, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": config_dict(args),
        "cpu_baseline": {"value": ms, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": ms, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.uuid = uuid
        self.proc = None
        self.path = None

    def start(self):
        f = tempfile.NamedTemporaryFile(prefix="nnv_clocks_", suffix=".csv", delete=False)
        self.path = f.name
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", self.uuid, "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=f, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        f.close()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        try:
            rows = [r.strip().split(",") for r in open(self.path) if r.strip()]
            os.unlink(self.path)
        except OSError:
            rows = []
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for nme, v in zip(names, r[4:8]):
                if v.strip().lower() == "active":
                    reasons.add(nme)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def count_launches(layers, choices, plan, nb):
    """Kernels of this library launched by one pass (layout conversion in, per-layer kernels, out)."""
    n = 2
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            n += 1
            continue
        v, m, cached = choices[i]
        if v in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
            n += 1
            continue
        if not cached:
            n += 1                                           # transform
        if v in (nb.VAR_WINO_F2, nb.VAR_WINO_F4, nb.VAR_WINO_F6):
            n += 3
        else:
            n += 1 + (1 if nb.nnv_exec_workspace_bytes(plan, i, v, m) else 0)
    return n


def raw_bytes(L):
    return 4 * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"]


def h2d_bytes(layers, choices, plan, nb, with_input_bytes):
    """Bytes that cross the host link per cold step: weights (raw or cached), biases, and the input image."""
    total = with_input_bytes
    for i, c in enumerate(choices):
        if c is None:
            continue
        L = layers[i]
        total += nb.nnv_transformed_bytes(plan, i, c[0], c[1]) if c[2] else raw_bytes(L)
        total += 4 * L["K"] if L["has_bias"] else 0
    return int(total)


def names(choices, nb):
    return [None if c is None else [nb.VARIANT_NAMES[c[0]], nb.MATH_NAMES[c[1]], c[2]] for c in choices]


def gemm_bytes(L):
    """Algorithmic bytes of one GEMM-executed layer: X once + packed weights + Y (fp32 words)."""
    oh, ow = wl.out_hw(L)
    qp = -(-(L["R"] * L["S"] * L["C"]) // 8) * 8
    return 4 * (L["C"] * L["H"] * L["W"] + L["K"] * qp + oh * ow * L["K"])


class Ranks:
    """The only cross-rank traffic of the benchmark: a barrier around the timed steps and the maximum of a timing over
    the ranks.  The path itself does not shard (every rank runs its own replica), so nothing else is exchanged.
    backend "nccl" reduces on the rank's GPU, "gloo" on the host (CPU tests)."""

    def __init__(self, backend=None, device=None):
        import torch.distributed as dist
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.device = device
        self.dist = dist
        if self.world > 1:
            if backend == "nccl":
                dist.init_process_group("nccl", device_id=device)
            else:
                dist.init_process_group(backend)

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()

    def reduce_max(self, v):
        if self.world == 1:
            return v
        import torch
        t = torch.tensor([v], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def run_ours(args):
    import torch
    from paper_2206_07446_b200 import binding as nb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    ranks = Ranks("nccl", torch.device("cuda", local))
    if args.tuning:
        nb.nnv_tuning_set(args.tuning)
    line = measure(args, args.config, args.steps, args.warmup, args.minimal, rank, world, local, ranks)
    # the other single-GPU configurations, headline numbers and rooflines only, beside the main workload
    others = {}
    for name in [c for c in args.also.split(",") if c and c != "none" and c != args.config]:
        o = measure(args, name, args.arm_steps, 3, True, rank, world, local, ranks)
        others[name] = {k: o[k] for k in ("value", "unit", "steps", "e2e", "roofline", "roofline_transform", "transform_all", "run", "per_layer", "pipeline_depth_ms")}
        others[name]["e2e"] = {k: o["e2e"][k] for k in ("value", "h2d_bytes_per_step", "host_link")}
    line["other_workloads"] = others
    if rank == 0:
        print(json.dumps(line))
    ranks.close()


def measure(args, config, steps, warmup, minimal, rank, world, local, ranks):
    """All measurements of one workload; returns the JSON line as a dict."""
    import torch
    from paper_2206_07446_b200 import binding as nb
    from paper_2206_07446_b200 import harness

    class _A:                                                  # the arguments with this call's workload and step counts
        pass
    a2 = _A()
    a2.__dict__.update(vars(args))
    a2.config, a2.steps, a2.warmup, a2.minimal = config, steps, warmup, minimal
    args = a2

    layers = wl.CONFIGS[args.config]()
    ws, bs = wl.make_weights(layers)
    x = wl.make_input(layers)
    # the headline is eager; a second plan over the same blob replays recorded graphs for the side arms
    model = harness.model_from_workload(layers, ws, bs, wl.weight_blob, use_graphs=0, kernel_stamps=1)
    plan_g = model.second_plan(use_graphs=1)
    math = nb.MATH_BF16 if args.math == "bf16" else nb.MATH_TF32

    # offline decision stage: profile every candidate kernel, select per layer by cold cost
    if args.load_costs:
        costs = json.load(open(args.load_costs))
    else:
        costs = model.profile(x, reps=5)
    if args.save_costs and rank == 0:
        json.dump(costs, open(args.save_costs, "w"))
    # math modes are accuracy classes: the BF16 class (output rel-L2 <= 1e-2) admits every kernel of the TF32 class (<= 1e-3) too
    admitted = (nb.MATH_FP32, nb.MATH_TF32) if math == nb.MATH_TF32 else (nb.MATH_FP32, nb.MATH_TF32, nb.MATH_BF16)
    costs = nb.CostTable([c for c in costs if c["math"] in admitted])
    choices_raw = nb.nnv_select_kernels(model.plan, costs, 0)        # headline: every layer reads RAW weights and transforms them
    choices_byp = nb.nnv_select_kernels(model.plan, costs, 1)        # bypass arm: cached post-transform weights allowed
    costs_res = nb.CostTable([dict(c, h2d_raw_ns=0, h2d_cached_ns=0) for c in costs])
    choices_res = nb.nnv_select_kernels(model.plan, costs_res, 0)    # no read stage: transform + exec only
    model.to_device()
    model.d_input.copy_(torch.from_numpy(x))
    model.h_input.copy_(torch.from_numpy(x))
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    s_copy, s_xform, s_exec = model.streams
    nev = max(args.steps, args.arm_steps)
    ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(nev)]
    ev1 = [torch.cuda.Event(enable_timing=True) for _ in range(nev)]

    def barrier():
        ranks.barrier()
        torch.cuda.synchronize()

    reduce_max = ranks.reduce_max

    last_ms = []                                              # per-step times of the most recent timed region

    def timed_region(step_fn, steps, warmup):
        """W untimed + K timed steps between barriers; mean ms per step (max over ranks)."""
        for k in range(warmup):
            step_fn(k, False)
        barrier()
        out = [step_fn(k, True) for k in range(steps)]
        barrier()
        ms = [ev0[k].elapsed_time(ev1[k]) for k in range(steps)]
        last_ms[:] = ms
        return reduce_max(sum(ms) / len(ms)), out

    def begin(k, timed, streams):
        model.arena.fill_(0xFF)                               # poison weights, transformed weights, scratch and activations: a
        flush.fill_(k & 0xFF)                                 # skipped operation cannot go unnoticed; then evict L2
        torch.cuda.synchronize()
        if timed:
            ev0[k].record(s_exec)
            for s in streams:
                s.wait_event(ev0[k])

    uuid = str(torch.cuda.get_device_properties(local).uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid)
    model.arena = None
    need = max(model.ensure_arena(c, d) for c, d in ((choices_raw, args.cold_depth), (choices_byp, args.cold_depth), (choices_res, args.depth)))
    model.arena.fill_(0xFF)
    if any(c is not None and c[2] for c in choices_byp):
        model.build_cached_blob(choices_byp)

    ch_raw_c = nb.choices_array(model.plan, choices_raw)      # marshalled once: ~1 us of Python per layer stays out of the steps
    ch_byp_c = nb.choices_array(model.plan, choices_byp)
    ch_res_c = nb.choices_array(model.plan, choices_res)

    # ---- headline: raw weights from pinned host memory, transform, execute; input / output on the device ----
    def step_value(k, timed):
        begin(k, timed, (s_copy, s_xform))
        ch = ch_raw_c                                         # decided offline (the paper's decision stage runs once per model and device)
        nb.nnv_cold_run_dio(model.plan, ch, model.h_weights, model.w_bytes, None, 0, model.d_input, model.d_output,
                            model.arena, model.arena.numel(), s_copy, s_xform, s_exec, args.cold_depth)
        if timed:
            ev1[k].record(s_exec)
            return nb.nnv_kernel_times(model.plan)            # the kernels' own device-clock stamps of this step

    sampler.start()
    torch.cuda.cudart().cudaProfilerStart()                  # a profiler attached with "profile from start off" sees the timed steps only
    value, step_timings = timed_region(step_value, args.steps, args.warmup)
    value_median = reduce_max(statistics.median(last_ms))
    y_gpu = model.d_output.cpu().numpy()

    # ---- e2e: the same step through nnv_cold_run, input and output in pinned host memory ---------------------
    wall, enq = [], []

    def step_e2e(k, timed):
        begin(k, timed, (s_copy, s_xform))
        t0 = time.perf_counter()
        ch = ch_raw_c
        nb.nnv_cold_run(model.plan, ch, model.h_weights, model.w_bytes, None, 0, model.h_input, model.h_output,
                        model.arena, model.arena.numel(), s_copy, s_xform, s_exec, args.cold_depth)
        if timed:
            ev1[k].record(s_exec)
            wall.append(time.perf_counter() - t0)
            enq.append(nb.nnv_last_enqueue_ns(model.plan))

    e2e, _ = timed_region(step_e2e, args.steps, args.warmup)
    torch.cuda.cudart().cudaProfilerStop()
    y_e2e = model.h_output.numpy().copy()
    e2e_wall = reduce_max(1e3 * sum(wall) / len(wall))

    # ---- the same step at every pipeline depth (staging slots; 1 = read, transform, execute one layer after the other) ----
    depth_ms = {}
    if args.depth_steps > 0:
        for d in (1, 2, 3, 4, 0):
            need_d = model.ensure_arena(choices_raw, d)

            def step_depth(k, timed, d=d, need_d=need_d):
                begin(k, timed, (s_copy, s_xform))
                nb.nnv_cold_run(model.plan, ch_raw_c, model.h_weights, model.w_bytes, None, 0, model.h_input, model.h_output,
                                model.arena, need_d, s_copy, s_xform, s_exec, d)
                if timed:
                    ev1[k].record(s_exec)

            depth_ms["unbounded" if d == 0 else str(d)] = timed_region(step_depth, min(args.depth_steps, nev), 3)[0]
        model.ensure_arena(choices_raw, args.cold_depth)

    arms = {}
    if not args.minimal:
        # ---- bypass arm (the paper's Section 3.1.2): selection may read cached post-transform weights ----
        def step_bypass(k, timed):
            begin(k, timed, (s_copy, s_xform))
            ch = ch_byp_c
            nb.nnv_cold_run(model.plan, ch, model.h_weights, model.w_bytes, model.h_cached, model.c_bytes, model.h_input,
                            model.h_output, model.arena, model.arena.numel(), s_copy, s_xform, s_exec, args.cold_depth)
            if timed:
                ev1[k].record(s_exec)

        ms, _ = timed_region(step_bypass, args.arm_steps, 3)
        arms["bypass_allowed"] = {"e2e_ms": ms, "what": "nnv_cold_run, eager, selection with allow_cached = 1",
                                  "cached_layers": sum(1 for c in choices_byp if c is not None and c[2]),
                                  "transform_launches": sum(1 for c in choices_byp if c is not None and not c[2] and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE)),
                                  "h2d_bytes_per_step": h2d_bytes(layers, choices_byp, model.plan, nb, x.nbytes)}

        # ---- zero-copy arm: the transform kernels read the raw weights in place in pinned host memory ----
        choices_zc = nb.nnv_select_kernels(model.plan, costs, 2)
        choices_zc_all = [None if c is None else (c[0], c[1], nb.ARM_ZERO_COPY if c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else 0)
                          for c in choices_raw]
        for name, chz in (("zero_copy_allowed", choices_zc), ("zero_copy_every_layer", choices_zc_all)):
            need = max(need, model.ensure_arena(chz, args.cold_depth))

            def step_zc(k, timed, chz=nb.choices_array(model.plan, chz)):
                begin(k, timed, (s_copy, s_xform))
                nb.nnv_cold_run(model.plan, chz, model.h_weights, model.w_bytes, None, 0, model.h_input, model.h_output,
                                model.arena, model.arena.numel(), s_copy, s_xform, s_exec, args.cold_depth)
                if timed:
                    ev1[k].record(s_exec)

            ms, _ = timed_region(step_zc, args.arm_steps, 3)
            arms[name] = {"e2e_ms": ms, "zero_copy_layers": sum(1 for c in chz if c is not None and c[2] == nb.ARM_ZERO_COPY),
                          "what": "nnv_cold_run, eager; " + ("selection with the zero-copy arm allowed (allow_cached = 2)" if name == "zero_copy_allowed"
                                                             else "the headline's kernels, every transform reading host memory in place")}
        # per layer, isolated: copy then transform against the fused zero-copy preparation (profiled costs)
        by_size = {}
        for c in costs:
            if c["zc_ns"] and choices_raw[c["layer"]] is not None and (c["variant"], c["math"]) == tuple(choices_raw[c["layer"]][:2]):
                by_size.setdefault(raw_bytes(layers[c["layer"]]), []).append((c["h2d_raw_ns"] + c["xform_ns"], c["zc_ns"]))
        arms["zero_copy_by_layer_size"] = [{"raw_bytes": b, "layers": len(v), "copy_then_transform_us": statistics.mean(a for a, _ in v) / 1e3,
                                            "zero_copy_us": statistics.mean(z for _, z in v) / 1e3} for b, v in sorted(by_size.items())]

        # ---- the headline step replayed from a recorded CUDA graph ----
        def step_graph(k, timed):
            begin(k, timed, (s_copy, s_xform))
            ch = ch_raw_c
            nb.nnv_cold_run(plan_g, ch, model.h_weights, model.w_bytes, None, 0, model.h_input, model.h_output,
                            model.arena, model.arena.numel(), s_copy, s_xform, s_exec, args.cold_depth)
            if timed:
                ev1[k].record(s_exec)

        ms, _ = timed_region(step_graph, args.arm_steps, 3)
        arms["graph_replay"] = {"e2e_ms": ms, "what": "nnv_cold_run with raw weights, replayed from a CUDA graph recorded by an earlier identical call"}

        # ---- weights already resident in HBM: transform + execution only ----
        def step_resident(k, timed):
            begin(k, timed, (s_xform,))
            ch = ch_res_c
            nb.nnv_resident_run(plan_g, ch, model.d_weights, model.w_bytes, None, 0, model.d_input, model.d_output,
                                model.arena, model.arena.numel(), s_xform, s_exec, args.depth)
            if timed:
                ev1[k].record(s_exec)

        ms, _ = timed_region(step_resident, args.arm_steps, 3)
        arms["resident"] = {"ms": ms, "what": "nnv_resident_run (no read stage), graph replay, pipeline depth %d" % args.depth}

    # ---- Algorithm 1: schedule (with calibration under overlap), then the same end-to-end step on its queues
    alg1 = None
    y_s = None
    if args.queues > 0 and not args.minimal:
        ch_s, q_s, t_pred, _ = model.schedule(x, costs, args.queues, allow_cached=0, rounds=2, eps_pct=1, combo_limit=4096)
        need_s = model.ensure_arena(ch_s, 0)
        st_s = model.prep_streams(args.queues)

        def step_sched(k, timed):
            begin(k, timed, st_s[1:])
            nb.nnv_cold_run_queues(model.plan, ch_s, q_s, args.queues, model.h_weights, model.w_bytes, None, 0,
                                   model.h_input, model.h_output, model.arena, model.arena.numel(), st_s)
            if timed:
                ev1[k].record(s_exec)

        ms, _ = timed_region(step_sched, args.arm_steps, 3)
        iso = {(c["layer"], c["variant"], c["math"]): c for c in costs}
        chosen = [iso[(i,) + c[:2]] for i, c in enumerate(ch_s) if c is not None]
        alg1 = {"n_little": args.queues, "e2e_ms": ms, "predicted_ms": t_pred / 1e6,
                "model": "shared host link (nnv_schedule_link); reads keep their isolated costs, transform and execution are rescaled by the calibration run",
                "isolated_sums_ms": {"read": sum(c["h2d_raw_ns"] for c in chosen) / 1e6, "transform": sum(c["xform_ns"] for c in chosen) / 1e6,
                                     "exec": sum(c["exec_ns"] for c in chosen) / 1e6},
                "calibration_factors": getattr(model, "calibration", None),
                "preps_on_queue0": sum(1 for q in q_s if q == 0),
                "choices_differing_from_per_layer_argmin": sum(1 for a, b in zip(ch_s, choices_raw) if a != b),
                "parity_rel_l2_end_to_end": None}
        y_s = model.h_output.numpy().copy()
        need = max(need, need_s)
        model.arena.fill_(0xFF)

    # ---- continuous mode (the paper's Section 3.5): cold inference with K_cold that leaves K_warm prepared,
    # then warm inferences; latency of the 1st, 2nd and later inferences, end to end from host buffers
    cont = None
    y_w = None
    if args.continuous_reps > 0 and not args.minimal:
        warm = nb.nnv_select_warm(model.plan, costs)
        need_c = max(model.ensure_arena(choices_raw, 0), model.ensure_arena(warm, 0))
        wbytes = nb.nnv_warm_bytes(model.plan, warm, model.w_bytes)
        d_warm = harness.dev_bytes(wbytes)
        seq = [[], [], [], []]
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
        for k in range(args.continuous_reps + 2):
            flush.fill_(k & 0xFF)
            torch.cuda.synchronize()
            evs[0].record(s_exec)
            s_copy.wait_event(evs[0])
            s_xform.wait_event(evs[0])
            nb.nnv_cold_run_continuous(model.plan, choices_raw, warm, model.h_weights, model.w_bytes, None, 0,
                                       model.h_input, model.h_output, model.arena, model.arena.numel(), d_warm, wbytes, s_copy, s_xform, s_exec)
            evs[1].record(s_exec)
            for j in range(3):
                nb.nnv_warm_run(model.plan, warm, d_warm, wbytes, model.w_bytes, model.h_input, model.h_output, model.arena,
                                need_c, s_xform, s_exec)
                evs[2 + j].record(s_exec)
            torch.cuda.synchronize()
            if k >= 2:
                for j in range(4):
                    seq[j].append(evs[j].elapsed_time(evs[j + 1]))
        y_w = model.h_output.numpy().copy()
        cont = {"first_cold_ms": reduce_max(statistics.mean(seq[0])), "second_ms": reduce_max(statistics.mean(seq[1])),
                "third_ms": reduce_max(statistics.mean(seq[2])), "fourth_ms": reduce_max(statistics.mean(seq[3])),
                "switched_layers": len(nb.nnv_switch_set(model.plan, choices_raw, warm)), "warm_buffer_bytes": int(wbytes),
                "parity_rel_l2_end_to_end": None}
        del d_warm
        need = max(need, need_c)
        model.arena.fill_(0xFF)

    # ---- storage stage: the same end-to-end step with the weights read from a model file (page cache
    # dropped before every run), the paper's "weights reading" in front of copy / transform / execution
    storage = None
    if args.file_reps > 0 and not args.minimal:
        path = os.path.join(tempfile.gettempdir(), "nnv_bench_%d_%d.nnv" % (os.getpid(), rank))
        try:
            model.write_model_file(path, choices_byp)
            cache = nb.CacheFile(path)
            ts, rd_ns, rd_b = [], [], []
            for k in range(args.file_reps + 2):
                flush.fill_(k & 0xFF)
                torch.cuda.synchronize()
                cache.drop_pages()
                evs2 = [torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)]
                evs2[0].record(s_exec)
                s_copy.wait_event(evs2[0])
                s_xform.wait_event(evs2[0])
                _, _, ns, nbytes = model.cold_run_file(None, choices_raw, cache, depth=args.cold_depth, drop_pages=False)
                evs2[1].record(s_exec)
                evs2[1].synchronize()
                if k >= 2:
                    ts.append(evs2[0].elapsed_time(evs2[1])); rd_ns.append(ns); rd_b.append(nbytes)
            storage = {"e2e_from_file_ms": reduce_max(statistics.mean(ts)), "file_bytes": int(cache.file_bytes),
                       "raw_weight_bytes": int(sum(raw_bytes(L) for L in layers if L["op"] == wl.OP_CONV)),
                       "cached_blob_bytes": int(cache.c_bytes),
                       "bytes_read_per_step": int(rd_b[-1]), "reader_gbs": rd_b[-1] / statistics.mean(rd_ns),
                       "reader_threads": 4, "page_cache": "posix_fadvise DONTNEED before every run (best effort)"}
            cache.close()
        finally:
            if os.path.exists(path):
                os.unlink(path)
        model.arena.fill_(0xFF)

    # host link: one bulk pinned copy of the same number of bytes, as the floor of the end-to-end number
    link_ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    link_ms = []
    nlink = min(model.w_bytes, model.d_weights.numel())
    for _ in range(5):
        with torch.cuda.stream(s_copy):
            link_ev[0].record(s_copy)
            model.d_weights[:nlink].copy_(model.h_weights[:nlink], non_blocking=True)
            link_ev[1].record(s_copy)
        link_ev[1].synchronize()
        link_ms.append(link_ev[0].elapsed_time(link_ev[1]))
    link_gbs = nlink / (min(link_ms) * 1e-3) / 1e9

    # the whole model's weights transformed by one multi-layer launch (the decision stage's job, also
    # what builds the cached blob): algorithmic bytes = raw read + transformed written
    xall = None
    offs_all, total_all = nb.nnv_transformed_layout(model.plan, choices_raw)
    if total_all:
        out_all = harness.dev_bytes(total_all, fill=None)
        ta = []
        for k in range(7):
            flush.fill_(k & 0xFF)
            s_xform.wait_stream(torch.cuda.current_stream())
            link_ev[0].record(s_xform)
            nb.nnv_transform_all(model.plan, choices_raw, model.d_weights, model.w_bytes, out_all, total_all, s_xform)
            link_ev[1].record(s_xform)
            link_ev[1].synchronize()
            ta.append(link_ev[0].elapsed_time(link_ev[1]))
        has_xf = [i for i, c in enumerate(choices_raw) if c is not None and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE)]
        raw_all = sum(raw_bytes(layers[i]) for i in has_xf)
        tr_all = sum(nb.nnv_transformed_bytes(model.plan, i, choices_raw[i][0], choices_raw[i][1]) for i in has_xf)
        med = sorted(ta)[len(ta) // 2]
        xall = {"kernel": "multi_transform_kernel (nnv_transform_all, one launch per transform group for the whole model)", "bound": "hbm",
                "bytes": raw_all + tr_all, "us": med * 1e3, "achieved": (raw_all + tr_all) / (med * 1e-3) / 1e9,
                "peak": None, "unit": "GB/s"}
        del out_all
    clocks = sampler.stop()
    peaks = load_peaks()

    # ---- rooflines: kernel durations are the kernels' own device-clock stamps (first block in, last block
    # out) taken INSIDE the timed headline steps; event pairs around 5 us kernels add microseconds of their own
    # and serialise the streams (the same step with per-layer events takes 1.8x as long)
    xf, ex = {}, {}                                              # layer -> [ns] over the timed steps
    for xs, es in step_timings:
        for i in range(len(layers)):
            if xs[i]:
                xf.setdefault(i, []).append(xs[i])
            if es[i]:
                ex.setdefault(i, []).append(es[i])
    avg = statistics.mean

    def layer_flops(i):
        L = layers[i]
        oh, ow = wl.out_hw(L)
        return 2 * oh * ow * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"]

    tf32_peak = peaks["bf16_tflops"] * 0.5
    tens_peak = peaks["bf16_tflops"] if math == nb.MATH_BF16 else tf32_peak
    # the tensor-core launches that carry a layer's convolution (implicit GEMM, 3x3 halo kernel, direct-operand 1x1, the
    # weights-on-rows kernel together with its split reduction; the stem's GEMM after its explicit im2col)
    single = [i for i in ex if choices_raw[i][0] in (nb.VAR_IM2COL, nb.VAR_GEMM1X1)]
    roof = None
    if single:
        gfl = sum(layer_flops(i) for i in single)
        gby = sum(gemm_bytes(layers[i]) for i in single)
        gns = sum(avg(ex[i]) for i in single)
        big = max(single, key=layer_flops)
        t_tensor = gfl / (tens_peak * 1e3)                       # ns at the tensor peak
        t_hbm = gby / peaks["hbm_gbs"]                            # ns at the HBM peak (the weights arrive cold)
        tens = {"bound": "tensor", "achieved": gfl / gns / 1e3, "peak": tens_peak, "unit": "TFLOP/s", "frac": gfl / gns / 1e3 / tens_peak}
        hbm = {"bound": "hbm", "achieved": gby / gns, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gby / gns / peaks["hbm_gbs"]}
        roof = dict(hbm if t_hbm >= t_tensor else tens)           # the binding roofline of these launches
        roof.update({"kernel": "gemm_tc_kernel / gemm_sp_kernel (+ splitk_reduce_kernel) / conv3x3_tc_kernel: the tcgen05 GEMM of every im2col / 1x1 layer",
                     "traffic": NCU_GEMM_TRAFFIC_BYTES.get((args.config, args.math)),
                     "durations": "device-clock stamps written by the kernels themselves inside the timed steps (CUDA events time the step)",
                     "peak_source": peaks["source"] + (" HBM copy" if t_hbm >= t_tensor else " bf16 burst" + ("" if math == nb.MATH_BF16 else " x 0.5 (tf32:bf16 nominal ratio)")),
                     "other_roofline": tens if t_hbm >= t_tensor else hbm,
                     "launches_per_step": len(single), "flops_per_step": gfl, "bytes_per_step": gby,
                     "sum_us_per_step": gns / 1e3, "avg_launch_us": gns / len(single) / 1e3,
                     "largest_launch": {"layer": big, "flops": layer_flops(big), "bytes": gemm_bytes(layers[big]),
                                        "us": avg(ex[big]) / 1e3, "tflops": layer_flops(big) / avg(ex[big]) / 1e3}})
    # the weight-transform kernels: filter transform and repack, HBM-bound; a grouped launch is booked on its first layer
    xroof = None
    if xf:
        xbytes = sum(raw_bytes(layers[i]) + nb.nnv_transformed_bytes(model.plan, i, c[0], c[1]) for i, c in enumerate(choices_raw)
                     if c is not None and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE))
        tns = sum(avg(v) for v in xf.values())
        xroof = {"kernel": "multi_transform_kernel (filter transform + repack), the grouped launches of the timed headline steps",
                 "bound": "hbm", "achieved": xbytes / tns, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": xbytes / tns / peaks["hbm_gbs"],
                 "traffic": None, "peak_source": peaks["source"], "launches_per_step": len(xf), "bytes_per_step": xbytes,
                 "sum_us_per_step": tns / 1e3, "avg_launch_us": tns / len(xf) / 1e3,
                 "durations": "device-clock stamps written by the kernels themselves inside the timed steps"}
    # per layer: the tensor-core kernel's duration inside the timed steps against the layer's own roofline
    per_layer = []
    for i in sorted(ex):
        L = layers[i]
        c = choices_raw[i]
        fl, by, us = layer_flops(i), gemm_bytes(L), avg(ex[i]) / 1e3
        t_min_us = max(fl / (tens_peak * 1e6), by / (peaks["hbm_gbs"] * 1e3))
        per_layer.append({"layer": i, "shape": "%dx%d C=%d K=%d R=%d s=%d" % (L["H"], L["W"], L["C"], L["K"], L["R"], L["stride"]),
                          "kernel": nb.VARIANT_NAMES[c[0]], "whole_conv": i in single, "us": round(us, 2),
                          "roofline_us": round(t_min_us, 2), "bound": "tensor" if fl / (tens_peak * 1e6) >= by / (peaks["hbm_gbs"] * 1e3) else "hbm",
                          "frac": round(t_min_us / us, 4)})
    # kernels that are not tensor-core GEMMs, each on the workload's layers that can run it (isolated launches, L2 flushed)
    krows = None if args.minimal else other_kernel_rooflines(layers, model, nb, torch, flush, peaks)

    flops = sum(layer_flops(i) for i in ex)
    exec_ns = sum(avg(v) for v in ex.values())
    xform_ns = sum(avg(v) for v in xf.values())
    n_xf = sum(1 for c in choices_raw if c is not None and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE))
    per_step_launches = count_launches(layers, choices_raw, model.plan, nb)

    h2d_value = h2d_bytes(layers, choices_raw, model.plan, nb, 0)
    h2d_e2e = h2d_bytes(layers, choices_raw, model.plan, nb, x.nbytes)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": value, "ms_per_step_median": value_median, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "tf32" if math == nb.MATH_TF32 else "bf16", "data": "synthetic",
        "config": config_dict(args),
        "run": {"what": "nnv_cold_run_dio: raw weights H2D + transform + execution, eager (no CUDA graph), selection with allow_cached = 0",
                "pipeline_depth": args.cold_depth, "replicas": world, "weights_bytes": int(model.w_bytes),
                "h2d_bytes_per_step": h2d_value, "transform_launches_per_step": n_xf,
                "cached_layers": sum(1 for c in choices_raw if c is not None and c[2])},
        "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": h2d_e2e,
                "d2h_bytes_per_step": int(model.h_output.numel() * 4), "host_wall_ms": e2e_wall,
                "host_enqueue_ms": statistics.mean(enq) / 1e6,
                "what": "nnv_cold_run: as `value`, plus the input image from and the output to pinned host memory",
                "host_link": {"bound": "pcie", "bulk_copy_gbs": link_gbs, "floor_ms": h2d_e2e / link_gbs / 1e6,
                              "frac_of_floor": (h2d_e2e / link_gbs / 1e6) / e2e if e2e > 0 else None}},
        "gpu_launches": 2 * per_step_launches * args.steps,
        "clocks": clocks,
        "roofline": roof,
        "roofline_transform": xroof,
        "transform_all": xall,
        "kernel_rooflines": krows,
        "per_layer": per_layer,
        "pipeline_depth_ms": {"what": "e2e of the headline's kernels at each pipeline depth (staging slots); the headline runs unbounded", **depth_ms} if depth_ms else None,
        "arms": arms,
        "algorithm1": alg1,
        "continuous": cont,
        "storage": storage,
        "breakdown": {"sum_xform_kernel_us": xform_ns / 1e3, "sum_tensor_core_kernel_us": exec_ns / 1e3,
                      "tensor_core_tflops": flops / exec_ns / 1e3 if exec_ns else None,
                      "choices": names(choices_raw, nb), "choices_bypass_arm": names(choices_byp, nb),
                      "choices_resident_arm": names(choices_res, nb)},
    }
    if xall:
        xall["peak"] = peaks["hbm_gbs"]
        xall["frac"] = xall["achieved"] / peaks["hbm_gbs"]

    if rank == 0 and world == 1 and not args.no_cpu_baseline and not args.minimal:
        from oracle import conv as oconv
        from oracle import model as omodel
        oconv.build()
        os.environ.setdefault("OMP_NUM_THREADS", str(cpu_threads()))
        oracle_pass(layers, ws, bs, x)
        ts = [oracle_pass(layers, ws, bs, x) for _ in range(args.cpu_passes)]
        line["cpu_baseline"] = {"value": 1e3 * sum(ts) / len(ts), "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": "whole %s workload, %d passes: literal filter transform / naive pack + fp64 direct-conv chain"
                                          % (args.config, args.cpu_passes)}
        ref = omodel.run_model(layers, ws, bs, x)[-1]
        den = float(np.sqrt(np.sum(ref * ref)))
        line["parity_rel_l2_end_to_end"] = float(np.sqrt(np.sum((y_gpu[0] - ref) ** 2)) / den)
        line["e2e"]["parity_rel_l2_end_to_end"] = float(np.sqrt(np.sum((y_e2e[0] - ref) ** 2)) / den)
        if alg1:
            alg1["parity_rel_l2_end_to_end"] = float(np.sqrt(np.sum((y_s[0] - ref) ** 2)) / den)
        if cont:
            cont["parity_rel_l2_end_to_end"] = float(np.sqrt(np.sum((y_w[0] - ref) ** 2)) / den)
    return line


# ------------------------------------------------------------------------------------------------
# Single kernels through the C ABI (CUDA events, L2 flushed between repetitions).  Weights and inputs are
# seeded random tensors created on the device; nothing here checks results (the tests do).
def _layer(C, K, R, stride, H, W, groups=1):
    return dict(op=0, C=C, K=K, R=R, S=R, stride=stride, pad=R // 2 if R > 1 else 0, groups=groups, H=H, W=W, in0=-1, in1=-1,
                act=1, has_bias=0)


def _buf(torch, nbytes):
    t = torch.empty(max(256, int(nbytes)), dtype=torch.uint8, device="cuda")
    assert t.data_ptr() % 256 == 0
    return t


def _rand(torch, nfloats, scale=1.0):
    return (torch.rand(max(64, int(nfloats)), device="cuda", dtype=torch.float32) * 2 - 1) * scale


def _time(torch, fn, reps, flush):
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


def _time_rotating(torch, fns, launches, reps):
    """Per-launch time of `launches` back-to-back launches between ONE pair of events, cycling through `fns` (the same
    kernel on different buffer sets whose total exceeds the L2): the events' own few microseconds are shared by all
    launches and every launch finds its data in DRAM."""
    st = torch.cuda.current_stream()
    ts = []
    for r in range(reps + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for i in range(launches):
            fns[i % len(fns)](st)
        e1.record(st)
        e1.synchronize()
        if r >= 2:
            ts.append(e0.elapsed_time(e1) * 1e3 / launches)  # us
    return statistics.median(ts)


def time_transform(torch, nb, variant, math, C, K, R=3, reps=20, flush=None):
    L = _layer(C, K, R, 1, 8, 8)
    plan = nb.Plan([L], [0], [0])
    rawb = 4 * K * C * R * R
    outb = nb.nnv_transformed_bytes(plan, 0, variant, math)
    d_raw = _rand(torch, K * C * R * R, 0.05)
    d_out = _buf(torch, outb)
    med, best = _time(torch, lambda st: nb.nnv_transform_weights(plan, 0, variant, math, d_raw, d_out, st), reps, flush)
    out = dict(op="transform", variant=nb.VARIANT_NAMES[variant], math=nb.MATH_NAMES[math], C=C, K=K, R=R,
               bytes=rawb + outb, us=med, us_min=best, gbs=(rawb + outb) / med / 1e3)
    # the kernel's own duration (device-clock stamps, no launch or event overhead): the layer as a one-layer model
    # whose resident run transforms the weights before it executes
    from paper_2206_07446_b200 import harness
    w = np.zeros((K, C, R, R), np.float32)
    m1 = harness.model_from_workload([L], [w], [None], wl.weight_blob, use_graphs=0, kernel_stamps=1)
    ch = [(variant, math, 0)]
    need = m1.ensure_arena(ch, 1)
    d_io_in, d_io_out = _rand(torch, C * 64), _buf(torch, 4 * 64 * K)
    ks = []
    for r in range(reps + 2):
        if flush is not None:
            flush.fill_(r & 0xFF)
        nb.nnv_resident_run(m1.plan, ch, d_raw, m1.w_bytes, None, 0, d_io_in, d_io_out, m1.arena, need, m1.streams[1], m1.streams[2], 1)
        ks.append(nb.nnv_kernel_times(m1.plan)[0][0] / 1e3)
    out["kernel_us"] = statistics.median(ks[2:])
    out["kernel_gbs"] = (rawb + outb) / out["kernel_us"] / 1e3 if out["kernel_us"] else None
    return out


def time_conv(torch, nb, variant, math, C, K, R, stride, H, W, groups=1, reps=20, flush=None):
    L = _layer(C, K, R, stride, H, W, groups)
    plan = nb.Plan([L], [0], [0])
    oh, ow = wl.out_hw(L)
    cg = C // groups
    d_raw = _rand(torch, K * cg * R * R, 0.05)
    if variant in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
        d_wt = d_raw
    else:
        d_wt = _buf(torch, nb.nnv_transformed_bytes(plan, 0, variant, math))
        nb.nnv_transform_weights(plan, 0, variant, math, d_raw, d_wt, torch.cuda.current_stream())
    d_in = _rand(torch, C * H * W)
    d_out = _buf(torch, 4 * oh * ow * K)
    wsb = nb.nnv_exec_workspace_bytes(plan, 0, variant, math)
    d_ws = _buf(torch, wsb) if wsb else None
    med, best = _time(torch, lambda st: nb.nnv_conv_exec(plan, 0, variant, math, d_in, None, d_wt, None, d_out, d_ws, wsb, st),
                      reps, flush)
    flops = 2.0 * oh * ow * K * cg * R * R
    out = dict(op="conv", variant=nb.VARIANT_NAMES[variant], math=nb.MATH_NAMES[math], C=C, K=K, R=R, stride=stride,
               H=H, W=W, groups=groups, direct_flops=flops, us=med, us_min=best, direct_tflops=flops / med / 1e6)
    if variant not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE):
        # the tensor-core kernel's own duration (device-clock stamps, no launch or event overhead): the layer as a
        # one-layer model through nnv_resident_run with its transformed weights passed as the cached blob
        from paper_2206_07446_b200 import harness
        w = np.zeros((K, cg, R, R), np.float32)
        m1 = harness.model_from_workload([L], [w], [None], wl.weight_blob, use_graphs=0, kernel_stamps=1)
        ch = [(variant, math, 1)]
        need = m1.ensure_arena(ch, 1)
        d_w = _buf(torch, m1.w_bytes)
        d_io_in, d_io_out = _rand(torch, C * H * W), _buf(torch, 4 * oh * ow * K)
        ks = []
        for r in range(reps + 2):
            if flush is not None:
                flush.fill_(r & 0xFF)
            nb.nnv_resident_run(m1.plan, ch, d_w, m1.w_bytes, d_wt, d_wt.numel(), d_io_in, d_io_out, m1.arena, need,
                                m1.streams[1], m1.streams[2], 1)
            ks.append(nb.nnv_kernel_times(m1.plan)[1][0] / 1e3)
        out["kernel_us"] = statistics.median(ks[2:])
        out["kernel_tflops"] = flops / out["kernel_us"] / 1e6 if out["kernel_us"] else None
    return out


def _offsets(layers):
    """Byte offsets of each layer's weights in a dense blob (256-byte aligned), no biases."""
    w_off, pos = [], 0
    for L in layers:
        w_off.append(pos)
        if L["op"] == wl.OP_CONV:
            pos += (raw_bytes(L) + 255) // 256 * 256
    return w_off, [0] * len(layers), pos


def time_transform_all(torch, nb, config, prefer, math, reps=20, flush=None):
    """Every layer's weight transform of one configuration by nnv_transform_all.  Layers take the first
    eligible variant of `prefer`, then gemm1x1 / im2col."""
    layers = wl.CONFIGS[config]()
    w_off, b_off, w_bytes = _offsets(layers)
    plan = nb.Plan(layers, w_off, b_off)
    choices = []
    for i, L in enumerate(layers):
        if L["op"] != wl.OP_CONV:
            choices.append(None)
            continue
        el = nb.nnv_eligible(plan, i)
        v = next((c for c in prefer + [nb.VAR_GEMM1X1, nb.VAR_IM2COL] if c in el), None)
        if v is None:
            v = nb.VAR_DEPTHWISE if nb.VAR_DEPTHWISE in el else el[0]
        m = nb.MATH_FP32 if v in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else (nb.MATH_TF32 if v in (nb.VAR_WINO_F4, nb.VAR_WINO_F6) else math)
        choices.append((v, m, 0))
    d_w = _rand(torch, w_bytes // 4 + 64, 0.05)
    offs, total = nb.nnv_transformed_layout(plan, choices)
    d_out = _buf(torch, total)
    med, best = _time(torch, lambda st: nb.nnv_transform_all(plan, choices, d_w, w_bytes, d_out, total, st), reps, flush)
    has = [i for i, c in enumerate(choices) if c is not None and c[0] not in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE)]
    raw = sum(raw_bytes(layers[i]) for i in has)
    out = sum(nb.nnv_transformed_bytes(plan, i, choices[i][0], choices[i][1]) for i in has)
    # the same bytes moved by a plain device copy, timed the same way: the ceiling of this measurement
    half = (raw + out) // 2
    a, b = _buf(torch, half), _buf(torch, half)
    cmed, _ = _time(torch, lambda st: b.copy_(a, non_blocking=True), reps, flush)
    return dict(op="transform-all", config=config, prefer=[nb.VARIANT_NAMES[v] for v in prefer], math=nb.MATH_NAMES[math],
                bytes=raw + out, us=med, us_min=best, gbs=(raw + out) / med / 1e3, copy_same_bytes_us=cmed,
                copy_gbs=2 * half / cmed / 1e3)


def other_kernel_rooflines(layers, model, nb, torch, flush, peaks):
    """Roofline rows for the kernels that are not tensor-core GEMMs, each timed alone (CUDA events, L2 flushed)
    on the layers of the workload that can run it: depthwise and direct convolution through nnv_conv_exec.
    Peaks: HBM = the measured copy bandwidth; FP32 = 2 flop x 128 lanes x 148 SMs x the maximum SM clock."""
    props = torch.cuda.get_device_properties(torch.cuda.current_device())
    sms = props.multi_processor_count
    clk_ghz = 1.965
    fp32_peak = 2 * 128 * sms * clk_ghz / 1e3                   # TFLOP/s
    rows = []
    dw = [L for L in layers if L["op"] == wl.OP_CONV and L["groups"] > 1]
    if dw:
        L = max(dw, key=lambda L: L["C"] * L["H"] * L["W"])
        r = time_conv(torch, nb, nb.VAR_DEPTHWISE, nb.MATH_FP32, L["C"], L["K"], L["R"], L["stride"], L["H"], L["W"], L["groups"], 10, flush)
        oh, ow = wl.out_hw(L)
        by = 4 * (L["C"] * L["H"] * L["W"] + L["C"] * oh * ow + L["C"] * L["R"] * L["S"])
        rows.append({"kernel": "depthwise_kernel", "bound": "hbm", "layer": "%dx%d C=%d stride %d" % (L["H"], L["W"], L["C"], L["stride"]),
                     "bytes": by, "us": r["us"], "achieved": by / r["us"] / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": by / r["us"] / 1e3 / peaks["hbm_gbs"]})
    w3 = [L for L in layers if L["op"] == wl.OP_CONV and L["groups"] == 1 and L["R"] == 3 and L["S"] == 3 and L["stride"] == 1]
    if w3:
        # the Winograd data transforms on the largest 3x3 / stride-1 layer, F(4x4,3x3): V and M through HBM
        L = dict(max(w3, key=lambda L: L["C"] * L["H"] * L["W"]), in0=-1, in1=-1, has_bias=0)
        plan = nb.Plan([L], [0], [0])
        v = nb.VAR_WINO_F4
        T, vb, mb = nb.nnv_wino_sizes(plan, 0, v, nb.MATH_TF32)
        oh, ow = wl.out_hw(L)
        d_in, d_V, d_M = _rand(torch, L["C"] * L["H"] * L["W"]), _buf(torch, vb), _rand(torch, mb // 4)
        d_out = _buf(torch, 4 * oh * ow * L["K"])
        us_in, _ = _time(torch, lambda st: nb.nnv_wino_input_transform(plan, 0, v, nb.MATH_TF32, d_in, d_V, st), 10, flush)
        us_out, _ = _time(torch, lambda st: nb.nnv_wino_output_transform(plan, 0, v, d_M, None, None, d_out, st), 10, flush)
        shape = "%dx%d C=%d K=%d, F(4x4,3x3), %d tiles" % (L["H"], L["W"], L["C"], L["K"], T)
        for name, by, us in (("wino_input_kernel", 4 * L["C"] * L["H"] * L["W"] + vb, us_in),
                             ("wino_output_kernel", mb + 4 * oh * ow * L["K"], us_out)):
            rows.append({"kernel": name, "bound": "hbm", "layer": shape, "bytes": by, "us": us, "achieved": by / us / 1e3,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": by / us / 1e3 / peaks["hbm_gbs"]})
    # The same kernels on an instance large enough for a bandwidth figure (the layers of the workloads above are 1-13 MB:
    # a few microseconds of launch ramp and tail around 0.2-2 us of data): 64 channels on 224 x 224, F(4x4,3x3) data
    # transforms and a 3x3 depthwise layer, eight launches per event pair over four buffer sets (> L2 in total).
    Lb = dict(op=0, C=64, K=64, R=3, S=3, stride=1, pad=1, groups=1, H=224, W=224, in0=-1, in1=-1, act=1, has_bias=0)
    planb = nb.Plan([Lb], [0], [0])
    T, vb, mb = nb.nnv_wino_sizes(planb, 0, nb.VAR_WINO_F4, nb.MATH_TF32)
    sets = [(_rand(torch, 64 * 224 * 224), _buf(torch, vb), _rand(torch, mb // 4), _buf(torch, 4 * 224 * 224 * 64)) for _ in range(4)]
    us_in = _time_rotating(torch, [lambda st, b=b: nb.nnv_wino_input_transform(planb, 0, nb.VAR_WINO_F4, nb.MATH_TF32, b[0], b[1], st) for b in sets], 8, 5)
    us_out = _time_rotating(torch, [lambda st, b=b: nb.nnv_wino_output_transform(planb, 0, nb.VAR_WINO_F4, b[2], None, None, b[3], st) for b in sets], 8, 5)
    for name, by, us in (("wino_input_kernel", 4 * 64 * 224 * 224 + vb, us_in), ("wino_output_kernel", mb + 4 * 224 * 224 * 64, us_out)):
        rows.append({"kernel": name, "bound": "hbm", "layer": "large instance: 224x224 C=64 K=64, F(4x4,3x3), %d tiles; 8 launches per event pair over 4 buffer sets" % T,
                     "bytes": by, "us": us, "achieved": by / us / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": by / us / 1e3 / peaks["hbm_gbs"]})
    Ld = dict(op=0, C=64, K=64, R=3, S=3, stride=1, pad=1, groups=64, H=224, W=224, in0=-1, in1=-1, act=1, has_bias=0)
    pland = nb.Plan([Ld], [0], [0])
    wd = _rand(torch, 64 * 9, 0.3)
    dsets = [(_rand(torch, 64 * 224 * 224), _buf(torch, 4 * 224 * 224 * 64)) for _ in range(6)]
    us_dw = _time_rotating(torch, [lambda st, b=b: nb.nnv_conv_exec(pland, 0, nb.VAR_DEPTHWISE, nb.MATH_FP32, b[0], None, wd, None, b[1], None, 0, st) for b in dsets], 12, 5)
    by = 4 * (2 * 64 * 224 * 224 + 64 * 9)
    rows.append({"kernel": "depthwise3x3_v4_kernel", "bound": "hbm", "layer": "large instance: 224x224 C=64 3x3 stride 1; 12 launches per event pair over 6 buffer sets",
                 "bytes": by, "us": us_dw, "achieved": by / us_dw / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": by / us_dw / 1e3 / peaks["hbm_gbs"]})
    dense = [L for L in layers if L["op"] == wl.OP_CONV and L["groups"] == 1]
    if dense:
        L = max(dense, key=lambda L: wl.out_hw(L)[0] * wl.out_hw(L)[1] * L["K"] * L["C"] * L["R"] * L["S"])
        r = time_conv(torch, nb, nb.VAR_DIRECT, nb.MATH_FP32, L["C"], L["K"], L["R"], L["stride"], L["H"], L["W"], 1, 5, flush)
        rows.append({"kernel": "direct_conv_kernel", "bound": "alu", "layer": "%dx%d C=%d K=%d R=%d stride %d" % (L["H"], L["W"], L["C"], L["K"], L["R"], L["stride"]),
                     "flops": r["direct_flops"], "us": r["us"], "achieved": r["direct_tflops"], "peak": fp32_peak, "unit": "TFLOP/s",
                     "frac": r["direct_tflops"] / fp32_peak,
                     "peak_derivation": "2 flop x 128 FP32 lanes x %d SMs x %.3f GHz (clocks.max.sm)" % (sms, clk_ghz)})
    return rows


def run_kernel(args):
    import torch
    from paper_2206_07446_b200 import binding as nb
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    if args.tuning:
        nb.nnv_tuning_set(args.tuning)
    wino = {2: nb.VAR_WINO_F2, 4: nb.VAR_WINO_F4, 6: nb.VAR_WINO_F6}
    flush = None if args.no_flush else torch.empty(FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    math = nb.MATH_NAMES.index(args.math)
    a = args
    if a.kernel == "transform":
        v = wino[a.m] if (a.R == 3 and a.m in wino) else (nb.VAR_GEMM1X1 if a.R == 1 else nb.VAR_IM2COL)
        print(json.dumps(time_transform(torch, nb, v, math, a.C, a.K, a.R, a.reps, flush)))
    elif a.kernel == "transform-sweep":
        for m in (2, 4, 6):
            for n in (64, 128, 256, 512, 1024, 2048):
                print(json.dumps(time_transform(torch, nb, wino[m], nb.MATH_TF32, n, n, 3, a.reps, flush)), flush=True)
        for n in (64, 256, 512, 1024):
            print(json.dumps(time_transform(torch, nb, nb.VAR_IM2COL, nb.MATH_TF32, n, n, 3, a.reps, flush)), flush=True)
            print(json.dumps(time_transform(torch, nb, nb.VAR_IM2COL, nb.MATH_BF16, n, n, 3, a.reps, flush)), flush=True)
    elif a.kernel == "transform-all":
        prefer = [nb.VARIANT_NAMES.index(v) for v in a.prefer.split(",") if v]
        print(json.dumps(time_transform_all(torch, nb, a.config, prefer, math, a.reps, flush)))
    elif a.kernel == "conv":
        v = nb.VARIANT_NAMES.index(a.variant)
        m = nb.MATH_FP32 if v in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else math
        print(json.dumps(time_conv(torch, nb, v, m, a.C, a.K, a.R, a.stride, a.H, a.W or a.H, a.groups, a.reps, flush)))
    else:
        shapes = [(64, 64, 3, 1, 56), (128, 128, 3, 1, 28), (256, 256, 3, 1, 14), (512, 512, 3, 1, 7),
                  (64, 64, 3, 1, 224), (128, 128, 3, 1, 112), (256, 256, 3, 1, 56), (512, 512, 3, 1, 28),
                  (256, 256, 3, 1, 112), (256, 256, 3, 1, 224), (512, 512, 3, 1, 112)]   # beyond the configurations: the asymptote
        for (C, K, R, s, H) in shapes:
            for v, m in ((nb.VAR_DIRECT, 0), (nb.VAR_IM2COL, 1), (nb.VAR_IM2COL, 2), (nb.VAR_WINO_F2, 1),
                         (nb.VAR_WINO_F2, 2), (nb.VAR_WINO_F4, 1), (nb.VAR_WINO_F6, 1)):
                print(json.dumps(time_conv(torch, nb, v, m, C, K, R, s, H, H, 1, a.reps, flush)), flush=True)
        for (C, K, H) in [(64, 256, 56), (256, 64, 56), (512, 2048, 7), (2048, 512, 7), (320, 1280, 7), (16, 96, 112),
                          (256, 1024, 14), (1024, 256, 14), (128, 512, 28), (512, 128, 28)]:
            for m in (1, 2):
                print(json.dumps(time_conv(torch, nb, nb.VAR_GEMM1X1, m, C, K, 1, 1, H, H, 1, a.reps, flush)), flush=True)
        for (C, s, H) in [(96, 2, 112), (384, 1, 14), (960, 1, 7)]:
            print(json.dumps(time_conv(torch, nb, nb.VAR_DEPTHWISE, 0, C, C, 3, s, H, H, C, a.reps, flush)), flush=True)


def main():
    args = parse()
    if args.kernel:
        run_kernel(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
