"""ctypes binding of ``libkimad.so`` (C ABI in ``include/kimad.h``), same names as the C calls.

Argument marshalling only: every step of the compression pass runs in the CUDA library.  PyTorch
appears here for device memory and streams.  There is no CPU fallback: if the library is missing
the import of a symbol fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

KIMAD_OK = 0
KIMAD_STATUS_INFEASIBLE = 1
KIMAD_STATUS_PLATEAU = 2
KIMAD_ERR_INVALID_ARG = -1
KIMAD_ERR_WORKSPACE = -2
KIMAD_ERR_CAPACITY = -3
KIMAD_ERR_NONFINITE = -4
KIMAD_ERR_TIMEOUT = -5
KIMAD_ERR_CUDA = -6
KIMAD_ERR_NOMEM = -7
KIMAD_ERR_TOO_LARGE = -8
KIMAD_BUILTIN_SCRATCH_BYTES = 32 << 20


class kimad_options(C.Structure):
    _fields_ = [("D", C.c_uint32), ("value_dtype", C.c_uint32), ("check_finite", C.c_uint32),
                ("infeasible_policy", C.c_uint32), ("max_packed_elems", C.c_uint64), ("worker_stride", C.c_uint64),
                ("curve_mode", C.c_uint32), ("policy", C.c_uint32), ("cost_model", C.c_uint32)]


class kimad_stats(C.Structure):
    _fields_ = [("budget_bytes", C.c_uint64), ("used_bytes", C.c_uint64), ("n_selected", C.c_uint64),
                ("total_err", C.c_float), ("status", C.c_int32)]


class kimad_packed(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("val", C.c_void_p), ("offs", C.c_void_p), ("k", C.c_void_p),
                ("j", C.c_void_p), ("stats", C.c_void_p), ("dense", C.c_void_p)]


STATS_DTYPE = np.dtype([("budget_bytes", "<u8"), ("used_bytes", "<u8"), ("n_selected", "<u8"),
                        ("total_err", "<f4"), ("status", "<i4")])

_lib = None


class KimadError(RuntimeError):
    def __init__(self, code, what):
        self.code = code
        super().__init__(f"{what}: {kimad_strerror(code)} ({code})")


def lib_path() -> str:
    """The ordinary build, or the checked build when the environment has KIMAD_CHECKED=1."""
    return _build.CHECKED_LIB_PATH if os.environ.get("KIMAD_CHECKED") == "1" else _build.LIB_PATH


def load():
    """Loads the compiled library; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2312_08053_b200.build` "
                           "(nvcc, sm_100a); there is no fallback implementation")
    L = C.CDLL(path)
    vp, u32, u64, dbl = C.c_void_p, C.c_uint32, C.c_uint64, C.c_double
    L.kimad_create.restype = C.c_int
    L.kimad_create.argtypes = [C.POINTER(vp), C.POINTER(u64), u32, u32, C.POINTER(dbl), u32,
                               C.POINTER(kimad_options)]
    L.kimad_destroy.restype = None
    L.kimad_destroy.argtypes = [vp]
    L.kimad_workspace_bytes.restype = C.c_size_t
    L.kimad_workspace_bytes.argtypes = [vp]
    L.kimad_set_workspace.restype = C.c_int
    L.kimad_set_workspace.argtypes = [vp, vp, C.c_size_t]
    step_args = [vp, vp, vp, C.POINTER(dbl), dbl, C.POINTER(kimad_packed), vp]
    L.kimad_step.restype = C.c_int
    L.kimad_step.argtypes = step_args
    L.kimad_step_builtin_scratch.restype = C.c_int
    L.kimad_step_builtin_scratch.argtypes = step_args
    L.kimad_debug_step_with_err.restype = C.c_int
    L.kimad_debug_step_with_err.argtypes = step_args + [vp]
    L.kimad_debug_step_with_j.restype = C.c_int
    L.kimad_debug_step_with_j.argtypes = step_args + [vp]
    L.kimad_apply_packed.restype = C.c_int
    L.kimad_apply_packed.argtypes = [vp, C.POINTER(kimad_packed), vp, vp]
    L.kimad_aggregate.restype = C.c_int
    L.kimad_aggregate.argtypes = [vp, vp, u64, u32, u64, C.POINTER(C.c_float), C.c_float, vp]
    L.kimad_get_k.restype = C.c_int
    L.kimad_get_k.argtypes = [vp, vp, vp]
    L.kimad_get_k_table.restype = C.c_int
    L.kimad_get_k_table.argtypes = [vp, vp]
    L.kimad_plan_budget.restype = C.c_int
    L.kimad_plan_budget.argtypes = [vp, dbl, dbl, C.POINTER(u64), vp]
    L.kimad_debug_get_curve.restype = C.c_int
    L.kimad_debug_get_curve.argtypes = [vp, vp, vp, vp, vp]
    L.kimad_debug_get_selection.restype = C.c_int
    L.kimad_debug_get_selection.argtypes = [vp, vp, vp]
    L.kimad_debug_enable_stage_timing.restype = C.c_int
    L.kimad_debug_enable_stage_timing.argtypes = [vp, C.c_int]
    L.kimad_debug_stage_times.restype = C.c_int
    L.kimad_debug_stage_times.argtypes = [vp, vp]
    L.kimad_debug_set_schedule.restype = C.c_int
    L.kimad_debug_set_schedule.argtypes = [vp, C.c_int]
    L.kimad_debug_trace_step.restype = C.c_int
    L.kimad_debug_trace_step.argtypes = [vp, vp, vp, C.POINTER(dbl), dbl, vp, vp, C.c_char_p, C.c_size_t]
    L.kimad_debug_get_band_meta.restype = C.c_int
    L.kimad_debug_get_band_meta.argtypes = [vp, vp]
    L.kimad_debug_exact_path_layers.restype = C.c_int
    L.kimad_debug_exact_path_layers.argtypes = [vp, C.POINTER(u64)]
    L.kimad_debug_check.restype = C.c_int
    L.kimad_debug_check.argtypes = [vp, C.POINTER(u32), C.POINTER(u32)]
    L.kimad_launch_count.restype = u64
    L.kimad_launch_count.argtypes = [vp]
    L.kimad_monitor_create.restype = C.c_int
    L.kimad_monitor_create.argtypes = [C.POINTER(vp), u32, dbl]
    L.kimad_monitor_destroy.restype = None
    L.kimad_monitor_destroy.argtypes = [vp]
    L.kimad_monitor_observe.restype = C.c_int
    L.kimad_monitor_observe.argtypes = [vp, u64, dbl]
    L.kimad_monitor_estimate.restype = dbl
    L.kimad_monitor_estimate.argtypes = [vp]
    L.kimad_strerror.restype = C.c_char_p
    L.kimad_strerror.argtypes = [C.c_int]
    _lib = L
    return L


def kimad_strerror(code: int) -> str:
    return load().kimad_strerror(int(code)).decode()


def _check(code, what):
    if code < 0:
        raise KimadError(code, what)
    return code


class Ctx:
    """Owning handle of a ``kimad_ctx*`` plus the shapes needed to size buffers."""

    def __init__(self, handle, L, W, K, N, opts: kimad_options):
        self.handle, self.L, self.W, self.K, self.N = handle, L, W, K, N
        self.D = opts.D or 1000
        self.value_dtype = opts.value_dtype
        self.cap = opts.max_packed_elems or N
        self.stride = opts.worker_stride or N
        self._keep = []  # tensors the context points into (workspace)

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and _lib is not None:
            _lib.kimad_destroy(h)


def kimad_create(layer_sizes, n_workers, ratio_grid, D=0, value_dtype=0, check_finite=0, max_packed_elems=0,
                 worker_stride=0, curve_mode=0, policy=0, cost_model=0) -> Ctx:
    ls = np.ascontiguousarray(layer_sizes, dtype=np.uint64)
    rg = np.ascontiguousarray(ratio_grid, dtype=np.float64)
    opts = kimad_options(D, value_dtype, check_finite, 0, max_packed_elems, worker_stride, curve_mode, policy, cost_model)
    h = C.c_void_p()
    _check(load().kimad_create(C.byref(h), ls.ctypes.data_as(C.POINTER(C.c_uint64)), ls.size, n_workers,
                               rg.ctypes.data_as(C.POINTER(C.c_double)), rg.size, C.byref(opts)), "kimad_create")
    return Ctx(h, int(ls.size), int(n_workers), int(rg.size), int(ls.sum()), opts)


def kimad_destroy(ctx: Ctx) -> None:
    h, ctx.handle = ctx.handle, None
    if h:
        load().kimad_destroy(h)


def kimad_workspace_bytes(ctx: Ctx) -> int:
    return int(load().kimad_workspace_bytes(ctx.handle))


def kimad_set_workspace(ctx: Ctx, workspace) -> None:
    """``workspace``: a CUDA uint8 tensor of at least kimad_workspace_bytes(ctx) bytes (kept alive by ctx)."""
    _check(load().kimad_set_workspace(ctx.handle, workspace.data_ptr(), workspace.numel() * workspace.element_size()),
           "kimad_set_workspace")
    ctx._keep = [workspace]


class Packed:
    """Device output buffers of one step (torch tensors) and the matching ``kimad_packed`` struct."""

    def __init__(self, ctx: Ctx, device="cuda"):
        import torch

        W, L, cap = ctx.W, ctx.L, ctx.cap
        self.idx = torch.zeros((W, cap), dtype=torch.int32, device=device)
        self.val = torch.zeros((W, cap), dtype=torch.float32 if ctx.value_dtype == 0 else torch.bfloat16, device=device)
        self.offs = torch.zeros((W, L + 1), dtype=torch.int64, device=device)
        self.k = torch.zeros((W, L), dtype=torch.int32, device=device)
        self.j = torch.zeros((W, L), dtype=torch.int32, device=device)
        self.stats = torch.zeros((W, STATS_DTYPE.itemsize), dtype=torch.uint8, device=device)
        self.dense = torch.zeros((W, L), dtype=torch.int32, device=device)
        self.c = kimad_packed(self.idx.data_ptr(), self.val.data_ptr(), self.offs.data_ptr(), self.k.data_ptr(),
                              self.j.data_ptr(), self.stats.data_ptr(), self.dense.data_ptr())

    def stats_host(self) -> np.ndarray:
        return self.stats.cpu().numpy().view(STATS_DTYPE).reshape(-1)


def _stream_ptr(stream):
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def kimad_apply_packed(ctx: Ctx, msg: "Packed", est, stream=None) -> int:
    """est: CUDA float32 tensor [W][ctx.stride], the receiver's copies of the senders' estimators (in place)."""
    return _check(load().kimad_apply_packed(ctx.handle, C.byref(msg.c), est.data_ptr(), _stream_ptr(stream)),
                  "kimad_apply_packed")


def kimad_aggregate(x, est, weights, gamma, stream=None) -> int:
    """x: CUDA float32 [n] (in place); est: CUDA float32 [W][stride]; weights: W host floats."""
    w = np.ascontiguousarray(weights, dtype=np.float32)
    return _check(load().kimad_aggregate(x.data_ptr(), est.data_ptr(), est.stride(0), w.size, x.numel(),
                                         w.ctypes.data_as(C.POINTER(C.c_float)), C.c_float(gamma),
                                         _stream_ptr(stream)), "kimad_aggregate")


def _bw(ctx, bandwidth):
    bw = np.ascontiguousarray(bandwidth, dtype=np.float64).reshape(-1)
    assert bw.size == ctx.W, "one bandwidth per worker"
    return bw


def kimad_step(ctx: Ctx, grads, state, bandwidth_bytes_per_s, t_target_s, out: Packed, stream=None) -> None:
    bw = _bw(ctx, bandwidth_bytes_per_s)
    _check(load().kimad_step(ctx.handle, grads.data_ptr(), state.data_ptr(), bw.ctypes.data_as(C.POINTER(C.c_double)),
                             float(t_target_s), C.byref(out.c), _stream_ptr(stream)), "kimad_step")


def kimad_step_builtin_scratch(ctx: Ctx, grads, state, bandwidth_bytes_per_s, t_target_s, out: Packed, stream=None) -> None:
    """kimad_step with the scratch in the library's built-in device array: for callers that cannot allocate
    device memory.  No workspace has to be attached to ``ctx``; raises KimadError(KIMAD_ERR_TOO_LARGE) when the
    context needs more than KIMAD_BUILTIN_SCRATCH_BYTES."""
    bw = _bw(ctx, bandwidth_bytes_per_s)
    _check(load().kimad_step_builtin_scratch(ctx.handle, grads.data_ptr(), state.data_ptr(),
                                             bw.ctypes.data_as(C.POINTER(C.c_double)), float(t_target_s),
                                             C.byref(out.c), _stream_ptr(stream)), "kimad_step_builtin_scratch")


def kimad_debug_step_with_err(ctx: Ctx, grads, state, bandwidth_bytes_per_s, t_target_s, out: Packed, err_dev,
                              stream=None) -> None:
    bw = _bw(ctx, bandwidth_bytes_per_s)
    _check(load().kimad_debug_step_with_err(ctx.handle, grads.data_ptr(), state.data_ptr(),
                                            bw.ctypes.data_as(C.POINTER(C.c_double)), float(t_target_s),
                                            C.byref(out.c), _stream_ptr(stream), err_dev.data_ptr()),
           "kimad_debug_step_with_err")


def kimad_debug_step_with_j(ctx: Ctx, grads, state, bandwidth_bytes_per_s, t_target_s, out: Packed, j_dev,
                            stream=None) -> None:
    bw = _bw(ctx, bandwidth_bytes_per_s)
    _check(load().kimad_debug_step_with_j(ctx.handle, grads.data_ptr(), state.data_ptr(),
                                          bw.ctypes.data_as(C.POINTER(C.c_double)), float(t_target_s),
                                          C.byref(out.c), _stream_ptr(stream), j_dev.data_ptr()),
           "kimad_debug_step_with_j")


def kimad_get_k(ctx: Ctx, stream=None):
    """Returns (status, k[W][L]) of the last step after synchronising the stream."""
    k = np.zeros((ctx.W, ctx.L), dtype=np.uint32)
    st = load().kimad_get_k(ctx.handle, k.ctypes.data, _stream_ptr(stream))
    return int(st), k


def kimad_get_k_table(ctx: Ctx) -> np.ndarray:
    kt = np.zeros((ctx.L, ctx.K), dtype=np.uint64)
    _check(load().kimad_get_k_table(ctx.handle, kt.ctypes.data), "kimad_get_k_table")
    return kt


def kimad_plan_budget(ctx: Ctx, bandwidth_bytes_per_s: float, t_target_s: float):
    """Returns (status, budget_bytes, cells[L][K] or None)."""
    c = C.c_uint64(0)
    cells = np.zeros((ctx.L, ctx.K), dtype=np.uint64)
    st = _check(load().kimad_plan_budget(ctx.handle, float(bandwidth_bytes_per_s), float(t_target_s), C.byref(c),
                                         cells.ctypes.data), "kimad_plan_budget")
    return st, int(c.value), (cells if st == 0 else None)


def kimad_debug_get_curve(ctx: Ctx):
    """Returns (err f32, tau u32, keep_eq u32, shift u32), each [W][L][K], of the last step."""
    shape = (ctx.W, ctx.L, ctx.K)
    err = np.zeros(shape, np.float32)
    tau = np.zeros(shape, np.uint32)
    keq = np.zeros(shape, np.uint32)
    shift = np.zeros(shape, np.uint32)
    _check(load().kimad_debug_get_curve(ctx.handle, err.ctypes.data, tau.ctypes.data, keq.ctypes.data,
                                        shift.ctypes.data), "kimad_debug_get_curve")
    return err, tau, keq, shift


def kimad_debug_get_selection(ctx: Ctx):
    """Returns (tau u32, keep_eq u32), each [W][L]: exact threshold of the chosen candidate of every layer."""
    tau = np.zeros((ctx.W, ctx.L), np.uint32)
    keq = np.zeros((ctx.W, ctx.L), np.uint32)
    _check(load().kimad_debug_get_selection(ctx.handle, tau.ctypes.data, keq.ctypes.data),
           "kimad_debug_get_selection")
    return tau, keq


STAGE_NAMES = ["sample", "sweep", "curve", "exact_fallback", "dp", "select_count", "select_scan", "select_write"]


def kimad_debug_enable_stage_timing(ctx: Ctx, enable: bool) -> None:
    _check(load().kimad_debug_enable_stage_timing(ctx.handle, int(bool(enable))), "kimad_debug_enable_stage_timing")


def kimad_debug_set_schedule(ctx: Ctx, mode: int) -> None:
    """0: two worker groups for large steps, 1: whenever W >= 2, 2: one group."""
    _check(load().kimad_debug_set_schedule(ctx.handle, int(mode)), "kimad_debug_set_schedule")


def kimad_debug_trace_step(ctx: Ctx, grads, state, bandwidth_bytes_per_s, t_target_s, out: "Packed", stream=None) -> str:
    """One step with CUDA events around every launch; returns the timeline, one line per launch."""
    bw = _bw(ctx, bandwidth_bytes_per_s)
    buf = C.create_string_buffer(1 << 16)
    _check(load().kimad_debug_trace_step(ctx.handle, grads.data_ptr(), state.data_ptr(),
                                         bw.ctypes.data_as(C.POINTER(C.c_double)), float(t_target_s), C.byref(out.c),
                                         _stream_ptr(stream), buf, len(buf)), "kimad_debug_trace_step")
    return buf.value.decode()


def kimad_debug_stage_times(ctx: Ctx) -> np.ndarray:
    """Stage durations (ms) of the last step, order as STAGE_NAMES."""
    ms = np.zeros(len(STAGE_NAMES), np.float32)
    _check(load().kimad_debug_stage_times(ctx.handle, ms.ctypes.data), "kimad_debug_stage_times")
    return ms


def kimad_debug_get_band_meta(ctx: Ctx, n_regular: int) -> np.ndarray:
    """u32 [W][n_regular][4]: bins, entries of the cell table in use, flag, detail (see kimad.h)."""
    out = np.zeros((ctx.W, n_regular, 4), np.uint32)
    _check(load().kimad_debug_get_band_meta(ctx.handle, out.ctypes.data), "kimad_debug_get_band_meta")
    return out


def kimad_debug_exact_path_layers(ctx: Ctx, detail: bool = False):
    """Layers handed to the exact radix path so far; with detail also the count per reason
    (forced, bands too wide, threshold outside band, bound too loose even after refinement), the number of
    layers refined, and per candidate how often its first bound was loose."""
    n = (C.c_uint64 * (6 + ctx.K))()
    _check(load().kimad_debug_exact_path_layers(ctx.handle, n), "kimad_debug_exact_path_layers")
    return [int(x) for x in n] if detail else int(n[0])


def kimad_debug_check(ctx: Ctx):
    """Returns (checked build?, failed-check bits, damaged canaries) -- see kimad.h."""
    w, b = C.c_uint32(0), C.c_uint32(0)
    rc = _check(load().kimad_debug_check(ctx.handle, C.byref(w), C.byref(b)), "kimad_debug_check")
    return bool(rc), int(w.value), int(b.value)


def kimad_launch_count(ctx: Ctx) -> int:
    return int(load().kimad_launch_count(ctx.handle))


def new_context(layer_sizes, n_workers, ratio_grid, device="cuda", **opts):
    """Convenience: create a context, allocate its workspace with torch and attach it."""
    import torch

    ctx = kimad_create(layer_sizes, n_workers, ratio_grid, **opts)
    ws = torch.empty(kimad_workspace_bytes(ctx) + 256, dtype=torch.uint8, device=device)
    off = (-ws.data_ptr()) % 256
    kimad_set_workspace(ctx, ws[off:])
    ctx._keep.append(ws)
    return ctx


class Monitor:
    """Owning handle of a ``kimad_monitor*`` (bandwidth estimate from the history of finished transfers)."""

    def __init__(self, window: int = 8, alpha: float = 1.0):
        h = C.c_void_p()
        _check(load().kimad_monitor_create(C.byref(h), int(window), float(alpha)), "kimad_monitor_create")
        self.handle = h

    def __del__(self):
        h, self.handle = getattr(self, "handle", None), None
        if h and _lib is not None:
            _lib.kimad_monitor_destroy(h)


def kimad_monitor_create(window: int = 8, alpha: float = 1.0) -> Monitor:
    return Monitor(window, alpha)


def kimad_monitor_observe(m: Monitor, n_bytes: int, seconds: float) -> None:
    _check(load().kimad_monitor_observe(m.handle, int(n_bytes), float(seconds)), "kimad_monitor_observe")


def kimad_monitor_estimate(m: Monitor) -> float:
    return float(load().kimad_monitor_estimate(m.handle))


def kimad_monitor_destroy(m: Monitor) -> None:
    h, m.handle = m.handle, None
    if h:
        load().kimad_monitor_destroy(h)
