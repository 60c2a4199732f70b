"""Thin PyTorch harness around the C ABI: owns device memory, pinned host blobs and streams.

PyTorch is used for allocation and stream handles only; every step of the path
runs inside libnnv.so.
"""
import numpy as np
import torch

from . import binding as nb


def _pinned_bytes(arr_u8):
    t = torch.empty(max(1, arr_u8.size), dtype=torch.uint8).pin_memory()
    if arr_u8.size:
        t[:arr_u8.size].copy_(torch.from_numpy(arr_u8))
    return t


def dev_bytes(nbytes, fill=0xFF):
    """256-byte aligned device buffer (torch's allocator returns >= 512-byte alignment), poisoned."""
    t = torch.empty(max(256, int(nbytes)), dtype=torch.uint8, device="cuda")
    assert t.data_ptr() % 256 == 0
    if fill is not None:
        t.fill_(fill)
    return t


class Model:
    """A plan plus its host-side weight blob, ready for cold runs."""

    def __init__(self, layers, blob_u8, w_off, b_off, max_depth=4, use_graphs=1, kernel_stamps=0):
        self.layers = layers
        self.plan = nb.Plan(layers, w_off, b_off, opts=dict(default_math=nb.MATH_TF32, allow_cached=1,
                                                            max_depth=max_depth, kernel_stamps=kernel_stamps,
                                                            use_graphs=use_graphs))
        self.h_weights = _pinned_bytes(np.ascontiguousarray(blob_u8))
        self.w_bytes = int(blob_u8.size)
        self.w_off, self.b_off = list(w_off), list(b_off)
        # copy, transform, execute; execution is latency-critical, so its blocks get scheduled ahead of
        # the bandwidth-heavy transforms that run beside it
        self.streams = [torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream(priority=-1)]
        L0, Ln = layers[0], layers[-1]
        self.h_input = torch.empty((1, L0["C"], L0["H"], L0["W"]), dtype=torch.float32).pin_memory()
        oh, ow = self.out_hw(len(layers) - 1)
        self.h_output = torch.empty((1, Ln["K"], oh, ow), dtype=torch.float32).pin_memory()
        self.arena = None
        self.h_cached = None
        self.c_bytes = 0

    def second_plan(self, use_graphs):
        """Another plan over the same layers and weight blob (e.g. one that replays recorded graphs beside an eager one)."""
        return nb.Plan(self.layers, self.w_off, self.b_off, opts=dict(default_math=nb.MATH_TF32, allow_cached=1, max_depth=4,
                                                                      kernel_stamps=0, use_graphs=use_graphs))

    def out_hw(self, i):
        L = self.layers[i]
        if L["op"] == nb.OP_GAVGPOOL:
            return 1, 1
        return ((L["H"] + 2 * L["pad"] - L["R"]) // L["stride"] + 1,
                (L["W"] + 2 * L["pad"] - L["S"]) // L["stride"] + 1)

    def default_choices(self, prefer=None, math=nb.MATH_TF32):
        """First eligible variant per conv layer, or the first of `prefer` that is eligible."""
        out = []
        for i, L in enumerate(self.layers):
            if L["op"] != nb.OP_CONV:
                out.append(None)
                continue
            el = nb.nnv_eligible(self.plan, i)
            v = None
            for cand in (prefer or []):
                if cand in el:
                    v = cand
                    break
            if v is None:
                v = nb.VAR_DEPTHWISE if nb.VAR_DEPTHWISE in el else el[0]
            m = nb.MATH_FP32 if v in (nb.VAR_DIRECT, nb.VAR_DEPTHWISE) else math
            out.append((v, m, 0))
        return out

    def ensure_arena(self, choices, depth):
        need = nb.nnv_arena_bytes(self.plan, choices, depth)
        if self.arena is None or self.arena.numel() < need:
            self.arena = dev_bytes(need)
        return need

    def build_cached_blob(self, choices):
        """Transform the weights of every layer chosen with cached=1 on the device and keep the
        result in pinned host memory, laid out as nnv_cached_layout() says."""
        offs, total = nb.nnv_cached_layout(self.plan, choices)
        host = torch.zeros(max(1, total), dtype=torch.uint8).pin_memory()
        for i, c in enumerate(choices):
            if c is None or not c[2]:
                continue
            L = self.layers[i]
            rbytes = 4 * L["K"] * (L["C"] // L["groups"]) * L["R"] * L["S"]
            raw = dev_bytes(rbytes)
            raw[:rbytes].copy_(self.h_weights[self.w_off[i]:self.w_off[i] + rbytes])
            tb = nb.nnv_transformed_bytes(self.plan, i, c[0], c[1])
            out = dev_bytes(tb)
            nb.nnv_transform_weights(self.plan, i, c[0], c[1], raw, out, torch.cuda.current_stream())
            torch.cuda.synchronize()
            host[offs[i]:offs[i] + tb].copy_(out[:tb])
        self.h_cached, self.c_bytes = host, total
        return offs, total

    def cold_run(self, x_nchw, choices, depth=2, want_timings=False, poison=True):
        """One cold inference through nnv_cold_run; returns (output NCHW numpy, timings)."""
        self.h_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.h_input.shape))
        need = self.ensure_arena(choices, depth)
        if poison:
            self.arena.fill_(0xFF)
            torch.cuda.synchronize()
        tm = nb.nnv_cold_run(self.plan, choices, self.h_weights, self.w_bytes, self.h_cached, self.c_bytes,
                             self.h_input, self.h_output, self.arena, need,
                             self.streams[0], self.streams[1], self.streams[2], depth, want_timings)
        return self.h_output.numpy().copy(), tm

    def prep_streams(self, n_little):
        """Execution stream + n_little preparation streams for nnv_cold_run_queues (created once)."""
        extra = getattr(self, "_prep_streams", [])
        while len(extra) < n_little:
            extra.append(torch.cuda.Stream())
        self._prep_streams = extra
        return [self.streams[2]] + extra[:n_little]

    def cold_run_queues(self, x_nchw, choices, queue_of, n_little, want_timings=False, poison=True):
        """One cold inference on the queues Algorithm 1 produced (nnv_cold_run_queues)."""
        self.h_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.h_input.shape))
        need = self.ensure_arena(choices, 0)
        if poison:
            self.arena.fill_(0xFF)
            torch.cuda.synchronize()
        tm = nb.nnv_cold_run_queues(self.plan, choices, queue_of, n_little, self.h_weights, self.w_bytes,
                                    self.h_cached, self.c_bytes, self.h_input, self.h_output, self.arena, need,
                                    self.prep_streams(n_little), want_timings)
        return self.h_output.numpy().copy(), tm

    def schedule(self, x_nchw, costs, n_little, allow_cached=1, rounds=2, eps_pct=1, big_pct=100, combo_limit=4096, link=True):
        """Algorithm 1 with its profiling step repeated under load: schedule from the cost table, run the
        schedule once with per-operation timings, let the library rescale the table by how much slower each kind
        of operation ran beside the others than alone (nnv_calibrate_costs), schedule again; `rounds` times.
        This method only sequences library calls.  link=True evaluates schedules with the shared-link latency
        (nnv_schedule_link) and keeps the isolated read costs (the link model adds the reads' waiting itself).  Returns (choices, queue_of, predicted ns, calibrated costs)."""
        table = costs
        eps = nb.nnv_schedule_eps(self.plan, costs, allow_cached, eps_pct)
        out = None
        self.calibration = None
        for r in range(rounds + 1):
            out = nb.nnv_schedule(self.plan, table, allow_cached, n_little, eps, big_pct, combo_limit, link=link)
            if r == rounds:
                break
            choices, queue_of, _ = out
            if any(c is not None and c[2] for c in choices):
                self.build_cached_blob(choices)
            self.cold_run_queues(x_nchw, choices, queue_of, n_little, poison=False)          # warm
            # three timed runs, per operation the median duration: one stalled run on a shared GPU must not set the factors
            runs = [self.cold_run_queues(x_nchw, choices, queue_of, n_little, want_timings=True, poison=False)[1] for _ in range(3)]
            tm = []
            for per_layer in zip(*runs):
                t = dict(per_layer[0])
                for op in ("h2d", "xform", "exec"):
                    t[op + "_start_ns"] = 0
                    t[op + "_end_ns"] = sorted(r[op + "_end_ns"] - r[op + "_start_ns"] for r in per_layer)[1]
                tm.append(t)
            rows, fac = nb.nnv_calibrate_costs(self.plan, costs, choices, tm, kinds=6 if link else 7)
            self.calibration = {k: (f[0] / f[1] if f[1] else None) for k, f in zip(("h2d", "xform", "exec"), fac)}
            table = nb.CostTable(rows)
        return out[0], out[1], out[2], table

    def cold_run_continuous(self, x_nchw, cold, warm, want_timings=False):
        """Cold inference with kernels `cold` that leaves the kernels `warm` prepared in a device buffer
        (nnv_cold_run_continuous); returns (output NCHW numpy, timings)."""
        self.h_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.h_input.shape))
        need = self.ensure_arena(cold, 0)
        need = max(need, self.ensure_arena(warm, 0))
        self.warm_bytes = nb.nnv_warm_bytes(self.plan, warm, self.w_bytes)
        if getattr(self, "d_warm", None) is None or self.d_warm.numel() < self.warm_bytes:
            self.d_warm = dev_bytes(self.warm_bytes)
        torch.cuda.synchronize()
        tm = nb.nnv_cold_run_continuous(self.plan, cold, warm, self.h_weights, self.w_bytes, self.h_cached, self.c_bytes,
                                        self.h_input, self.h_output, self.arena, self.arena.numel(), self.d_warm, self.warm_bytes,
                                        self.streams[0], self.streams[1], self.streams[2], want_timings)
        return self.h_output.numpy().copy(), tm

    def warm_run(self, x_nchw, warm, want_timings=False):
        """One warm inference from the buffer a continuous cold run left behind (nnv_warm_run)."""
        if x_nchw is not None:
            self.h_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.h_input.shape))
        tm = nb.nnv_warm_run(self.plan, warm, self.d_warm, self.warm_bytes, self.w_bytes, self.h_input, self.h_output,
                             self.arena, self.arena.numel(), self.streams[1], self.streams[2], want_timings)
        return self.h_output.numpy().copy(), tm

    def write_model_file(self, path, choices, queue_of=None, n_little=0):
        """Store the plan, the raw weights and (for choices with cached = 1) the cached blob in a model file."""
        if any(c is not None and c[2] for c in choices):
            self.build_cached_blob(choices)
        nb.nnv_cache_write(path, self.plan, choices, queue_of, n_little, self.h_weights, self.w_bytes,
                           self.h_cached if self.c_bytes else None, self.c_bytes)

    def cold_run_file(self, x_nchw, choices, cache, depth=2, want_timings=False, drop_pages=True):
        """One cold inference whose weights come from an open model file (nnv_cold_run_file) through pinned
        staging buffers of this object; returns (output NCHW numpy, timings, reader ns, bytes read)."""
        if x_nchw is not None:
            self.h_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.h_input.shape))
        if getattr(self, "h_stage_w", None) is None or self.h_stage_w.numel() < cache.w_bytes:
            self.h_stage_w = torch.empty(max(1, cache.w_bytes), dtype=torch.uint8).pin_memory()
        if getattr(self, "h_stage_c", None) is None or self.h_stage_c.numel() < max(1, cache.c_bytes):
            self.h_stage_c = torch.empty(max(1, cache.c_bytes), dtype=torch.uint8).pin_memory()
        need = self.ensure_arena(choices, depth)
        if drop_pages:
            cache.drop_pages()
        tm, ns, nbytes = nb.nnv_cold_run_file(self.plan, choices, cache, self.h_stage_w, self.h_stage_w.numel(),
                                              self.h_stage_c if cache.c_bytes else None, self.h_stage_c.numel() if cache.c_bytes else 0,
                                              self.h_input, self.h_output, self.arena, need,
                                              self.streams[0], self.streams[1], self.streams[2], depth, want_timings)
        return self.h_output.numpy().copy(), tm, ns, nbytes

    def to_device(self):
        """Device copies of the weight blob, the cached blob (if built) and I/O buffers for nnv_resident_run."""
        self.d_weights = dev_bytes(self.w_bytes, fill=None)
        self.d_weights[:self.w_bytes].copy_(self.h_weights[:self.w_bytes])
        self.d_cached = None
        if self.h_cached is not None and self.c_bytes:
            self.d_cached = dev_bytes(self.c_bytes, fill=None)
            self.d_cached[:self.c_bytes].copy_(self.h_cached[:self.c_bytes])
        self.d_input = torch.empty(self.h_input.shape, dtype=torch.float32, device="cuda")
        self.d_output = torch.empty(self.h_output.shape, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()

    def resident_run(self, x_nchw, choices, depth=2, want_timings=False, poison=True):
        """One pass with weights and input already in HBM (nnv_resident_run); returns (NCHW numpy, timings)."""
        if getattr(self, "d_weights", None) is None:
            self.to_device()
        if x_nchw is not None:
            self.d_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.d_input.shape))
        need = self.ensure_arena(choices, depth)
        if poison:
            self.arena.fill_(0xFF)
        torch.cuda.synchronize()
        tm = nb.nnv_resident_run(self.plan, choices, self.d_weights, self.w_bytes, self.d_cached, self.c_bytes,
                                 self.d_input, self.d_output, self.arena, need,
                                 self.streams[1], self.streams[2], depth, want_timings)
        return self.d_output.cpu().numpy(), tm

    def layer_output(self, i):
        """NCHW numpy copy of layer i's activation left in the arena by the last cold run."""
        ptr, nbytes = nb.nnv_layer_output(self.plan, i)
        off = ptr - self.arena.data_ptr()
        L = self.layers[i]
        oh, ow = self.out_hw(i)
        t = self.arena[off:off + nbytes].view(torch.float32).reshape(oh, ow, L["K"])
        return t.permute(2, 0, 1).contiguous().cpu().numpy()

    def profile(self, x_nchw, reps=5):
        self.h_input.copy_(torch.from_numpy(np.ascontiguousarray(x_nchw, dtype=np.float32)).reshape(self.h_input.shape))
        need = nb.nnv_profile_arena_bytes(self.plan)
        arena = dev_bytes(need, fill=None)
        costs = nb.nnv_profile(self.plan, self.h_weights, self.w_bytes, self.h_input, arena, need,
                               torch.cuda.current_stream(), reps)
        del arena
        return costs


def model_from_workload(layers, weights, biases, blob_fn, max_depth=4, use_graphs=1, kernel_stamps=0):
    """Build a Model from a layer list and per-layer numpy weights using `blob_fn`
    (workloads.weight_blob) to lay out the host blob."""
    blob, w_off, b_off = blob_fn(layers, weights, biases)
    return Model(layers, blob, w_off, b_off, max_depth=max_depth, use_graphs=use_graphs, kernel_stamps=kernel_stamps)
