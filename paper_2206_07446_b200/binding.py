"""ctypes binding of libnnv.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see
include/nnv.h) and does nothing but convert Python values to C arguments and
raise on a non-zero status.  Device buffers are torch tensors (or raw integer
addresses); streams are torch.cuda.Stream objects (or raw handles).  There is
no CPU fallback: importing this module fails if the library has not been built.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnnv.so")

OP_CONV, OP_MAXPOOL, OP_GAVGPOOL = 0, 1, 2
VAR_DIRECT, VAR_IM2COL, VAR_GEMM1X1, VAR_DEPTHWISE, VAR_WINO_F2, VAR_WINO_F4, VAR_WINO_F6 = range(7)
VARIANT_NAMES = ["direct", "im2col", "gemm1x1", "depthwise", "wino_f2", "wino_f4", "wino_f6"]
MATH_FP32, MATH_TF32, MATH_BF16 = 0, 1, 2
ARM_RAW, ARM_CACHED, ARM_ZERO_COPY = 0, 1, 2           # the `cached` field of a choice: how the weights are prepared
MATH_NAMES = ["fp32", "tf32", "bf16"]
STATUS_NAMES = ["OK", "INVALID_ARG", "UNSUPPORTED", "STATE", "WORKSPACE_TOO_SMALL", "CUDA", "TIMEOUT"]


class NnvError(RuntimeError):
    def __init__(self, status, message):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__("nnv: %s: %s" % (name, message))


class LayerDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("op", "C", "K", "R", "S", "stride", "pad", "groups", "H", "W", "in0", "in1", "act", "has_bias")] + \
               [("w_off", ctypes.c_uint64), ("b_off", ctypes.c_uint64)]


class PlanOpts(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("default_math", "allow_cached", "max_depth", "kernel_stamps", "use_graphs")]


class Cost(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("layer", "variant", "math", "reserved")] + \
               [(n, ctypes.c_uint64) for n in ("h2d_raw_ns", "xform_ns", "h2d_cached_ns", "exec_ns", "zc_ns")]


class Choice(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("variant", "math", "cached")]


class Timing(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint64) for n in
                ("h2d_start_ns", "h2d_end_ns", "xform_start_ns", "xform_end_ns", "exec_start_ns", "exec_end_ns",
                 "h2d_bytes", "xform_bytes", "exec_flops")] + [("choice", Choice), ("reserved", ctypes.c_int32)]


if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libnnv.so is not built (%s). Run `python -m paper_2206_07446_b200.build` "
        "(needs nvcc with sm_100a support); there is no fallback path." % LIB_PATH)
_lib = ctypes.CDLL(LIB_PATH)

_vp, _i32, _u64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64
_P = ctypes.POINTER
_SIGS = {
    "nnv_plan_create": [_P(LayerDesc), _i32, _P(PlanOpts), _P(_vp)],
    "nnv_plan_destroy": [_vp],
    "nnv_tuning_set": [ctypes.c_char_p],
    "nnv_eligible": [_vp, _i32, _P(_i32), _i32, _P(_i32)],
    "nnv_transformed_bytes": [_vp, _i32, _i32, _i32, _P(_u64)],
    "nnv_exec_workspace_bytes": [_vp, _i32, _i32, _i32, _P(_u64)],
    "nnv_arena_bytes": [_vp, _P(Choice), _i32, _P(_u64)],
    "nnv_cached_layout": [_vp, _P(Choice), _P(_u64), _P(_u64)],
    "nnv_filter_candidates": [_vp, _i32, _P(Cost), _i32, _i32, _P(Choice), _i32, _P(_i32)],
    "nnv_select_kernels": [_vp, _P(Cost), _i32, _i32, _P(Choice)],
    "nnv_select_warm": [_vp, _P(Cost), _i32, _P(Choice)],
    "nnv_switch_set": [_vp, _P(Choice), _P(Choice), _P(_i32), _i32, _P(_i32)],
    "nnv_simulate": [_vp, _P(_u64), _P(_u64), _P(_u64), _P(_i32), _i32, _P(_u64)],
    "nnv_schedule_queues": [_vp, _P(_u64), _P(_u64), _P(_u64), _i32, _u64, _P(_i32), _P(_u64)],
    "nnv_schedule": [_vp, _P(Cost), _i32, _i32, _P(_u64), _i32, _u64, _i32, _u64, _P(Choice), _P(_i32), _P(_u64)],
    "nnv_simulate_link": [_vp, _P(_u64), _P(_u64), _P(_u64), _P(_u64), _P(_i32), _i32, _P(_u64)],
    "nnv_schedule_link": [_vp, _P(Cost), _i32, _i32, _P(_u64), _i32, _u64, _i32, _u64, _P(Choice), _P(_i32), _P(_u64)],
    "nnv_schedule_eps": [_vp, _P(Cost), _i32, _i32, _i32, _P(_u64)],
    "nnv_calibrate_costs": [_vp, _P(Cost), _i32, _P(Choice), _P(Timing), _i32, _P(Cost), _P(_u64)],
    "nnv_transform_weights": [_vp, _i32, _i32, _i32, _vp, _vp, _vp],
    "nnv_transformed_layout": [_vp, _P(Choice), _P(_u64), _P(_u64)],
    "nnv_transform_all": [_vp, _P(Choice), _vp, _u64, _vp, _u64, _vp],
    "nnv_conv_exec": [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _u64, _vp],
    "nnv_conv_exec_static": [_vp, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp],
    "nnv_wino_sizes": [_vp, _i32, _i32, _i32, _P(_i32), _P(_u64), _P(_u64)],
    "nnv_wino_input_transform": [_vp, _i32, _i32, _i32, _vp, _vp, _vp],
    "nnv_wino_output_transform": [_vp, _i32, _i32, _vp, _vp, _vp, _vp, _vp],
    "nnv_pool_exec": [_vp, _i32, _vp, _vp, _vp],
    "nnv_chw_to_hwc": [_vp, _vp, _i32, _i32, _i32, _vp],
    "nnv_hwc_to_chw": [_vp, _vp, _i32, _i32, _i32, _vp],
    "nnv_cold_run": [_vp, _P(Choice), _vp, _u64, _vp, _u64, _vp, _vp, _vp, _u64, _vp, _vp, _vp, _i32, _P(Timing)],
    "nnv_cold_run_dio": [_vp, _P(Choice), _vp, _u64, _vp, _u64, _vp, _vp, _vp, _u64, _vp, _vp, _vp, _i32, _P(Timing)],
    "nnv_cold_run_queues": [_vp, _P(Choice), _P(_i32), _i32, _vp, _u64, _vp, _u64, _vp, _vp, _vp, _u64, _P(_vp), _P(Timing)],
    "nnv_resident_run": [_vp, _P(Choice), _vp, _u64, _vp, _u64, _vp, _vp, _vp, _u64, _vp, _vp, _i32, _P(Timing)],
    "nnv_warm_bytes": [_vp, _P(Choice), _u64, _P(_u64)],
    "nnv_cold_run_continuous": [_vp, _P(Choice), _P(Choice), _vp, _u64, _vp, _u64, _vp, _vp, _vp, _u64, _vp, _u64, _vp, _vp, _vp,
                                _P(Timing)],
    "nnv_warm_run": [_vp, _P(Choice), _vp, _u64, _u64, _vp, _vp, _vp, _u64, _vp, _vp, _P(Timing)],
    "nnv_cache_write": [ctypes.c_char_p, _vp, _P(Choice), _P(_i32), _i32, _vp, _u64, _vp, _u64],
    "nnv_cache_open": [ctypes.c_char_p, _P(_vp)],
    "nnv_cache_close": [_vp],
    "nnv_cache_info": [_vp, _P(_i32), _P(_u64), _P(_u64), _P(_i32), _P(_u64)],
    "nnv_cache_read_plan": [_vp, _P(LayerDesc), _P(Choice), _P(_i32), _i32],
    "nnv_cache_read_blobs": [_vp, _vp, _u64, _vp, _u64],
    "nnv_cache_drop_pages": [_vp],
    "nnv_cold_run_file": [_vp, _P(Choice), _vp, _vp, _u64, _vp, _u64, _vp, _vp, _vp, _u64, _vp, _vp, _vp, _i32, _P(Timing),
                          _P(_u64), _P(_u64)],
    "nnv_layer_output": [_vp, _i32, _P(_vp), _P(_u64)],
    "nnv_last_enqueue_ns": [_vp, _P(_u64)],
    "nnv_kernel_times": [_vp, _P(_u64), _P(_u64)],
    "nnv_kernel_spans": [_vp, _P(_u64), _P(_u64)],
    "nnv_profile_arena_bytes": [_vp, _P(_u64)],
    "nnv_profile": [_vp, _vp, _u64, _vp, _vp, _u64, _vp, _i32, _P(Cost), _i32, _P(_i32)],
    "nnv_device_status": [_P(_i32)],
}
for _name, _args in _SIGS.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes = _args
    _fn.restype = ctypes.c_int
_lib.nnv_last_error.restype = ctypes.c_char_p
_lib.nnv_last_error.argtypes = []
_lib.nnv_version.restype = ctypes.c_int32
_lib.nnv_version.argtypes = []


def _check(status):
    if status != 0:
        raise NnvError(status, _lib.nnv_last_error().decode("utf-8", "replace"))


def _ptr(x):
    """Address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError("cannot take the address of %r" % type(x))


def _stream(s):
    if s is None:
        return None
    if isinstance(s, int):
        return s
    return s.cuda_stream


def nnv_version():
    return int(_lib.nnv_version())


def nnv_last_error():
    return _lib.nnv_last_error().decode("utf-8", "replace")


class Plan:
    """Owns an nnv_plan_t*.  `layers` is a list of dicts with the descriptor's field names."""

    def __init__(self, layers, w_off=None, b_off=None, opts=None):
        n = len(layers)
        arr = (LayerDesc * n)()
        for i, L in enumerate(layers):
            for f, _ in LayerDesc._fields_:
                if f in ("w_off", "b_off"):
                    continue
                setattr(arr[i], f, int(L[f]))
            arr[i].w_off = int(w_off[i]) if w_off is not None else int(L.get("w_off", 0))
            arr[i].b_off = int(b_off[i]) if b_off is not None else int(L.get("b_off", 0))
        o = None
        if opts is not None:
            o = ctypes.pointer(PlanOpts(**opts))
        h = _vp()
        _check(_lib.nnv_plan_create(arr, n, o, ctypes.byref(h)))
        self.handle = h
        self.n = n
        self.layers = [dict(L) for L in layers]

    def close(self):
        if getattr(self, "handle", None):
            _lib.nnv_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def nnv_plan_create(layers, w_off=None, b_off=None, opts=None):
    return Plan(layers, w_off, b_off, opts)


def nnv_plan_destroy(plan):
    plan.close()


def nnv_tuning_set(spec=None):
    """Process-wide tuning overrides, "key=value;key=value"; None or "" restores the defaults."""
    _check(_lib.nnv_tuning_set(None if spec is None else spec.encode("ascii")))


def nnv_eligible(plan, layer):
    out = (_i32 * 8)()
    n = _i32(0)
    _check(_lib.nnv_eligible(plan.handle, layer, out, 8, ctypes.byref(n)))
    return [int(out[i]) for i in range(n.value)]


def nnv_transformed_bytes(plan, layer, variant, math):
    b = _u64(0)
    _check(_lib.nnv_transformed_bytes(plan.handle, layer, variant, math, ctypes.byref(b)))
    return int(b.value)


def nnv_exec_workspace_bytes(plan, layer, variant, math):
    b = _u64(0)
    _check(_lib.nnv_exec_workspace_bytes(plan.handle, layer, variant, math, ctypes.byref(b)))
    return int(b.value)


def _choices_array(plan, choices):
    if isinstance(choices, ctypes.Array):                 # already marshalled (choices_array): latency-critical callers
        return choices
    arr = (Choice * plan.n)()
    for i, c in enumerate(choices):
        if c is None:
            arr[i] = Choice(-1, -1, 0)
        else:
            arr[i] = Choice(int(c[0]), int(c[1]), int(c[2]))
    return arr


def choices_array(plan, choices):
    """The per-layer choices as the C array the run calls take; building it once keeps ~1 us per layer of Python
    out of every call that passes it."""
    return _choices_array(plan, choices)


def nnv_arena_bytes(plan, choices, depth):
    b = _u64(0)
    _check(_lib.nnv_arena_bytes(plan.handle, _choices_array(plan, choices), depth, ctypes.byref(b)))
    return int(b.value)


def nnv_cached_layout(plan, choices):
    offs = (_u64 * plan.n)()
    total = _u64(0)
    _check(_lib.nnv_cached_layout(plan.handle, _choices_array(plan, choices), offs, ctypes.byref(total)))
    return [int(o) for o in offs], int(total.value)


class CostTable:
    """A cost table already laid out as the C array of nnv_cost_t, so that calls that take one (selection,
    scheduling) cost what the library call costs and not the conversion from Python dicts."""

    def __init__(self, costs):
        self.rows = [dict(c) for c in costs]
        self.array = _costs_array(self.rows)

    def __len__(self):
        return len(self.rows)

    def __iter__(self):
        return iter(self.rows)


def _costs_array(costs):
    if isinstance(costs, CostTable):
        return costs.array
    arr = (Cost * max(1, len(costs)))()
    for i, c in enumerate(costs):
        arr[i] = Cost(int(c["layer"]), int(c["variant"]), int(c["math"]), 0, int(c["h2d_raw_ns"]),
                      int(c["xform_ns"]), int(c["h2d_cached_ns"]), int(c["exec_ns"]), int(c.get("zc_ns", 0)))
    return arr


def nnv_filter_candidates(plan, layer, costs, allow_cached):
    out = (Choice * 64)()
    n = _i32(0)
    _check(_lib.nnv_filter_candidates(plan.handle, layer, _costs_array(costs), len(costs), int(allow_cached),
                                      out, 64, ctypes.byref(n)))
    return [(out[i].variant, out[i].math, out[i].cached) for i in range(n.value)]


def nnv_select_kernels(plan, costs, allow_cached):
    out = (Choice * plan.n)()
    _check(_lib.nnv_select_kernels(plan.handle, _costs_array(costs), len(costs), int(allow_cached), out))
    return [None if out[i].variant < 0 else (out[i].variant, out[i].math, out[i].cached) for i in range(plan.n)]


def nnv_select_warm(plan, costs):
    """K_warm: per conv layer the kernel with the least execution time, as (variant, math, prepared)."""
    out = (Choice * plan.n)()
    _check(_lib.nnv_select_warm(plan.handle, _costs_array(costs), len(costs), out))
    return [None if out[i].variant < 0 else (out[i].variant, out[i].math, out[i].cached) for i in range(plan.n)]


def nnv_switch_set(plan, cold, warm):
    """Layers of K_warm - K_cold."""
    out = (_i32 * max(1, plan.n))()
    n = _i32(0)
    _check(_lib.nnv_switch_set(plan.handle, _choices_array(plan, cold), _choices_array(plan, warm), out, plan.n,
                               ctypes.byref(n)))
    return [int(out[i]) for i in range(n.value)]


def _u64_array(plan, values):
    if len(values) != plan.n:
        raise ValueError("one entry per layer expected")
    return (_u64 * plan.n)(*[int(v) for v in values])


def nnv_simulate(plan, prep_little_ns, prep_big_ns, exec_ns, queue_of, n_little):
    if len(queue_of) != plan.n:
        raise ValueError("one entry per layer expected")
    t = _u64(0)
    _check(_lib.nnv_simulate(plan.handle, _u64_array(plan, prep_little_ns), _u64_array(plan, prep_big_ns),
                             _u64_array(plan, exec_ns), (_i32 * plan.n)(*[int(q) for q in queue_of]), n_little,
                             ctypes.byref(t)))
    return int(t.value)


def nnv_schedule_queues(plan, prep_little_ns, prep_big_ns, exec_ns, n_little, eps_ns=0):
    q = (_i32 * plan.n)()
    t = _u64(0)
    _check(_lib.nnv_schedule_queues(plan.handle, _u64_array(plan, prep_little_ns), _u64_array(plan, prep_big_ns),
                                    _u64_array(plan, exec_ns), n_little, int(eps_ns), q, ctypes.byref(t)))
    return [int(v) for v in q], int(t.value)


def nnv_simulate_link(plan, read_ns, xform_little_ns, xform_big_ns, exec_ns, queue_of, n_little):
    if len(queue_of) != plan.n:
        raise ValueError("one entry per layer expected")
    t = _u64(0)
    _check(_lib.nnv_simulate_link(plan.handle, _u64_array(plan, read_ns), _u64_array(plan, xform_little_ns),
                                  _u64_array(plan, xform_big_ns), _u64_array(plan, exec_ns),
                                  (_i32 * plan.n)(*[int(q) for q in queue_of]), n_little, ctypes.byref(t)))
    return int(t.value)


def nnv_schedule_eps(plan, costs, allow_cached, eps_pct):
    e = _u64(0)
    _check(_lib.nnv_schedule_eps(plan.handle, _costs_array(costs), len(costs), int(allow_cached), int(eps_pct), ctypes.byref(e)))
    return int(e.value)


def _timings_array(plan, timings):
    arr = (Timing * plan.n)()
    for i, t in enumerate(timings):
        for f, _ in Timing._fields_:
            if f in ("choice", "reserved"):
                continue
            setattr(arr[i], f, int(t.get(f, 0)))
    return arr


def nnv_calibrate_costs(plan, costs, choices, timings, kinds=7):
    """kinds: bit mask of the kinds to rescale (1 read, 2 transform, 4 execution).
    Returns (rescaled cost rows as dicts, [(num, den) for read, transform, execution])."""
    n = len(costs)
    out = (Cost * max(1, n))()
    fac = (_u64 * 6)()
    _check(_lib.nnv_calibrate_costs(plan.handle, _costs_array(costs), n, _choices_array(plan, choices),
                                    _timings_array(plan, timings), int(kinds), out, fac))
    rows = [{f: int(getattr(out[i], f)) for f, _ in Cost._fields_ if f != "reserved"} for i in range(n)]
    return rows, [(int(fac[2 * k]), int(fac[2 * k + 1])) for k in range(3)]


def nnv_schedule(plan, costs, allow_cached, n_little, eps_ns=0, big_pct=100, combo_limit=4096, pool_ns=None, link=False):
    """Algorithm 1; link=True evaluates every combination with the shared-link latency (nnv_schedule_link)."""
    out = (Choice * plan.n)()
    q = (_i32 * plan.n)()
    t = _u64(0)
    pool = _u64_array(plan, pool_ns) if pool_ns is not None else None
    fn = _lib.nnv_schedule_link if link else _lib.nnv_schedule
    _check(fn(plan.handle, _costs_array(costs), len(costs), int(allow_cached), pool, n_little,
              int(eps_ns), int(big_pct), int(combo_limit), out, q, ctypes.byref(t)))
    choices = [None if out[i].variant < 0 else (out[i].variant, out[i].math, out[i].cached) for i in range(plan.n)]
    return choices, [int(v) for v in q], int(t.value)


def nnv_transform_weights(plan, layer, variant, math, d_raw, d_out, stream=None):
    _check(_lib.nnv_transform_weights(plan.handle, layer, variant, math, _ptr(d_raw), _ptr(d_out), _stream(stream)))


def nnv_transformed_layout(plan, choices):
    offs = (_u64 * plan.n)()
    total = _u64(0)
    _check(_lib.nnv_transformed_layout(plan.handle, _choices_array(plan, choices), offs, ctypes.byref(total)))
    return [int(o) for o in offs], int(total.value)


def nnv_transform_all(plan, choices, d_weights, w_bytes, d_out, out_bytes, stream=None):
    _check(_lib.nnv_transform_all(plan.handle, _choices_array(plan, choices), _ptr(d_weights), int(w_bytes),
                                  _ptr(d_out), int(out_bytes), _stream(stream)))


def nnv_conv_exec(plan, layer, variant, math, d_in, d_addend, d_wt, d_bias, d_out, d_ws, ws_bytes, stream=None):
    _check(_lib.nnv_conv_exec(plan.handle, layer, variant, math, _ptr(d_in), _ptr(d_addend), _ptr(d_wt),
                              _ptr(d_bias), _ptr(d_out), _ptr(d_ws), int(ws_bytes), _stream(stream)))


STATIC_SCRATCH_BYTES = 16 << 20


def nnv_conv_exec_static(plan, layer, variant, math, d_in, d_addend, d_wt, d_bias, d_out, stream=None):
    """nnv_conv_exec for callers without device scratch of their own: the scratch is a fixed array
    inside the library (STATIC_SCRATCH_BYTES); nothing is allocated by this call."""
    _check(_lib.nnv_conv_exec_static(plan.handle, layer, variant, math, _ptr(d_in), _ptr(d_addend), _ptr(d_wt),
                                     _ptr(d_bias), _ptr(d_out), _stream(stream)))


def nnv_wino_sizes(plan, layer, variant, math):
    """(tiles, bytes of V, bytes of M) of a Winograd variant of a layer."""
    t, vb, mb = _i32(0), _u64(0), _u64(0)
    _check(_lib.nnv_wino_sizes(plan.handle, layer, variant, math, ctypes.byref(t), ctypes.byref(vb), ctypes.byref(mb)))
    return int(t.value), int(vb.value), int(mb.value)


def nnv_wino_input_transform(plan, layer, variant, math, d_in, d_V, stream=None):
    _check(_lib.nnv_wino_input_transform(plan.handle, layer, variant, math, _ptr(d_in), _ptr(d_V), _stream(stream)))


def nnv_wino_output_transform(plan, layer, variant, d_M, d_addend, d_bias, d_out, stream=None):
    _check(_lib.nnv_wino_output_transform(plan.handle, layer, variant, _ptr(d_M), _ptr(d_addend), _ptr(d_bias), _ptr(d_out),
                                          _stream(stream)))


def nnv_pool_exec(plan, layer, d_in, d_out, stream=None):
    _check(_lib.nnv_pool_exec(plan.handle, layer, _ptr(d_in), _ptr(d_out), _stream(stream)))


def nnv_chw_to_hwc(d_in, d_out, C, H, W, stream=None):
    _check(_lib.nnv_chw_to_hwc(_ptr(d_in), _ptr(d_out), C, H, W, _stream(stream)))


def nnv_hwc_to_chw(d_in, d_out, C, H, W, stream=None):
    _check(_lib.nnv_hwc_to_chw(_ptr(d_in), _ptr(d_out), C, H, W, _stream(stream)))


def nnv_cold_run(plan, choices, h_weights, w_bytes, h_cached, c_bytes, h_input, h_output, d_arena, arena_bytes,
                 s_copy, s_xform, s_exec, depth, want_timings=False):
    """Returns the list of per-layer timing dicts when want_timings, else None."""
    tarr = (Timing * plan.n)() if want_timings else None
    _check(_lib.nnv_cold_run(plan.handle, _choices_array(plan, choices), _ptr(h_weights), int(w_bytes),
                             _ptr(h_cached), int(c_bytes), _ptr(h_input), _ptr(h_output), _ptr(d_arena),
                             int(arena_bytes), _stream(s_copy), _stream(s_xform), _stream(s_exec), int(depth), tarr))
    return _timings_list(tarr)


def nnv_cold_run_dio(plan, choices, h_weights, w_bytes, h_cached, c_bytes, d_input, d_output, d_arena, arena_bytes,
                     s_copy, s_xform, s_exec, depth, want_timings=False):
    """nnv_cold_run with the model input / output in device memory; weights still come from pinned host memory."""
    tarr = (Timing * plan.n)() if want_timings else None
    _check(_lib.nnv_cold_run_dio(plan.handle, _choices_array(plan, choices), _ptr(h_weights), int(w_bytes),
                                 _ptr(h_cached), int(c_bytes), _ptr(d_input), _ptr(d_output), _ptr(d_arena),
                                 int(arena_bytes), _stream(s_copy), _stream(s_xform), _stream(s_exec), int(depth), tarr))
    return _timings_list(tarr)


def nnv_cold_run_queues(plan, choices, queue_of, n_little, h_weights, w_bytes, h_cached, c_bytes, h_input, h_output,
                        d_arena, arena_bytes, streams, want_timings=False):
    """streams: n_little + 1 streams, [0] = execution.  Returns per-layer timing dicts when want_timings."""
    if len(queue_of) != plan.n or len(streams) != n_little + 1:
        raise ValueError("queue_of needs one entry per layer and streams n_little + 1 entries")
    tarr = (Timing * plan.n)() if want_timings else None
    sarr = (_vp * (n_little + 1))(*[_stream(s) for s in streams])
    _check(_lib.nnv_cold_run_queues(plan.handle, _choices_array(plan, choices),
                                    (_i32 * plan.n)(*[int(q) for q in queue_of]), int(n_little), _ptr(h_weights),
                                    int(w_bytes), _ptr(h_cached), int(c_bytes), _ptr(h_input), _ptr(h_output),
                                    _ptr(d_arena), int(arena_bytes), sarr, tarr))
    return _timings_list(tarr)


def nnv_warm_bytes(plan, warm, w_bytes):
    b = _u64(0)
    _check(_lib.nnv_warm_bytes(plan.handle, _choices_array(plan, warm), int(w_bytes), ctypes.byref(b)))
    return int(b.value)


def nnv_cold_run_continuous(plan, cold, warm, h_weights, w_bytes, h_cached, c_bytes, h_input, h_output, d_arena,
                            arena_bytes, d_warm, warm_bytes, s_copy, s_xform, s_exec, want_timings=False):
    tarr = (Timing * plan.n)() if want_timings else None
    _check(_lib.nnv_cold_run_continuous(plan.handle, _choices_array(plan, cold), _choices_array(plan, warm),
                                        _ptr(h_weights), int(w_bytes), _ptr(h_cached), int(c_bytes), _ptr(h_input),
                                        _ptr(h_output), _ptr(d_arena), int(arena_bytes), _ptr(d_warm), int(warm_bytes),
                                        _stream(s_copy), _stream(s_xform), _stream(s_exec), tarr))
    return _timings_list(tarr)


def nnv_warm_run(plan, warm, d_warm, warm_bytes, w_bytes, h_input, h_output, d_arena, arena_bytes, s_xform, s_exec,
                 want_timings=False):
    tarr = (Timing * plan.n)() if want_timings else None
    _check(_lib.nnv_warm_run(plan.handle, _choices_array(plan, warm), _ptr(d_warm), int(warm_bytes), int(w_bytes),
                             _ptr(h_input), _ptr(h_output), _ptr(d_arena), int(arena_bytes), _stream(s_xform),
                             _stream(s_exec), tarr))
    return _timings_list(tarr)


def nnv_cache_write(path, plan, choices, queue_of, n_little, h_weights, w_bytes, h_cached, c_bytes):
    q = None if queue_of is None else (_i32 * plan.n)(*[int(v) for v in queue_of])
    _check(_lib.nnv_cache_write(os.fsencode(path), plan.handle, _choices_array(plan, choices), q, int(n_little),
                                _ptr(h_weights), int(w_bytes), _ptr(h_cached), int(c_bytes)))


class CacheFile:
    """An open model file (nnv_cache_t*)."""

    def __init__(self, path):
        h = _vp()
        _check(_lib.nnv_cache_open(os.fsencode(path), ctypes.byref(h)))
        self.handle = h
        n, w, c, nl, fb = _i32(0), _u64(0), _u64(0), _i32(0), _u64(0)
        _check(_lib.nnv_cache_info(h, ctypes.byref(n), ctypes.byref(w), ctypes.byref(c), ctypes.byref(nl), ctypes.byref(fb)))
        self.n_layers, self.w_bytes, self.c_bytes, self.n_little, self.file_bytes = n.value, w.value, c.value, nl.value, fb.value

    def read_plan(self):
        """(layer dicts, choices, queue_of) as stored."""
        n = self.n_layers
        layers, choices, queues = (LayerDesc * n)(), (Choice * n)(), (_i32 * n)()
        _check(_lib.nnv_cache_read_plan(self.handle, layers, choices, queues, n))
        ls = [{f: int(getattr(layers[i], f)) for f, _ in LayerDesc._fields_} for i in range(n)]
        cs = [None if choices[i].variant < 0 else (choices[i].variant, choices[i].math, choices[i].cached) for i in range(n)]
        return ls, cs, [int(q) for q in queues]

    def read_blobs(self, h_weights, h_cached=None):
        _check(_lib.nnv_cache_read_blobs(self.handle, _ptr(h_weights), int(self.w_bytes), _ptr(h_cached),
                                         int(self.c_bytes if h_cached is not None else 0)))

    def drop_pages(self):
        _check(_lib.nnv_cache_drop_pages(self.handle))

    def close(self):
        if self.handle:
            _lib.nnv_cache_close(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def nnv_cold_run_file(plan, choices, cache, h_stage_weights, stage_w_bytes, h_stage_cached, stage_c_bytes, h_input, h_output,
                      d_arena, arena_bytes, s_copy, s_xform, s_exec, depth, want_timings=False):
    """Returns (timings or None, reader nanoseconds, bytes read from the file)."""
    tarr = (Timing * plan.n)() if want_timings else None
    ns, nbytes = _u64(0), _u64(0)
    _check(_lib.nnv_cold_run_file(plan.handle, _choices_array(plan, choices), cache.handle, _ptr(h_stage_weights),
                                  int(stage_w_bytes), _ptr(h_stage_cached), int(stage_c_bytes), _ptr(h_input), _ptr(h_output),
                                  _ptr(d_arena), int(arena_bytes), _stream(s_copy), _stream(s_xform), _stream(s_exec),
                                  int(depth), tarr, ctypes.byref(ns), ctypes.byref(nbytes)))
    return _timings_list(tarr), int(ns.value), int(nbytes.value)


def _timings_list(tarr):
    if tarr is None:
        return None
    out = []
    for t in tarr:
        d = {f: int(getattr(t, f)) for f, _ in Timing._fields_ if f not in ("choice", "reserved")}
        d["choice"] = (t.choice.variant, t.choice.math, t.choice.cached)
        out.append(d)
    return out


def nnv_resident_run(plan, choices, d_weights, w_bytes, d_cached, c_bytes, d_input, d_output, d_arena, arena_bytes,
                     s_xform, s_exec, depth, want_timings=False):
    tarr = (Timing * plan.n)() if want_timings else None
    _check(_lib.nnv_resident_run(plan.handle, _choices_array(plan, choices), _ptr(d_weights), int(w_bytes),
                                 _ptr(d_cached), int(c_bytes), _ptr(d_input), _ptr(d_output), _ptr(d_arena),
                                 int(arena_bytes), _stream(s_xform), _stream(s_exec), int(depth), tarr))
    return _timings_list(tarr)


def nnv_layer_output(plan, layer):
    p = _vp()
    b = _u64(0)
    _check(_lib.nnv_layer_output(plan.handle, layer, ctypes.byref(p), ctypes.byref(b)))
    return int(p.value), int(b.value)


def nnv_kernel_times(plan):
    """(xform_ns, exec_ns) per layer from the kernels' own device-clock stamps of the last run (plan option kernel_stamps)."""
    xf, ex = (_u64 * plan.n)(), (_u64 * plan.n)()
    _check(_lib.nnv_kernel_times(plan.handle, xf, ex))
    return [int(v) for v in xf], [int(v) for v in ex]


def nnv_kernel_spans(plan):
    """Per layer ((xform_start, xform_end), (exec_start, exec_end)) in ns from the run's earliest stamped kernel start."""
    xf, ex = (_u64 * (2 * plan.n))(), (_u64 * (2 * plan.n))()
    _check(_lib.nnv_kernel_spans(plan.handle, xf, ex))
    return [((int(xf[2 * i]), int(xf[2 * i + 1])), (int(ex[2 * i]), int(ex[2 * i + 1]))) for i in range(plan.n)]


def nnv_last_enqueue_ns(plan):
    b = _u64(0)
    _check(_lib.nnv_last_enqueue_ns(plan.handle, ctypes.byref(b)))
    return int(b.value)


def nnv_profile_arena_bytes(plan):
    b = _u64(0)
    _check(_lib.nnv_profile_arena_bytes(plan.handle, ctypes.byref(b)))
    return int(b.value)


def nnv_profile(plan, h_weights, w_bytes, h_input, d_arena, arena_bytes, stream, reps):
    cap = plan.n * 16
    out = (Cost * cap)()
    n = _i32(0)
    _check(_lib.nnv_profile(plan.handle, _ptr(h_weights), int(w_bytes), _ptr(h_input), _ptr(d_arena),
                            int(arena_bytes), _stream(stream), int(reps), out, cap, ctypes.byref(n)))
    return [{f: int(getattr(out[i], f)) for f, _ in Cost._fields_ if f != "reserved"} for i in range(n.value)]


def nnv_device_status():
    c = _i32(0)
    _check(_lib.nnv_device_status(ctypes.byref(c)))
    return int(c.value)


EXPORTED_SYMBOLS = sorted(list(_SIGS.keys()) + ["nnv_last_error", "nnv_version"])
