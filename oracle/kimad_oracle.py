"""ctypes front end of the CPU oracle (``kimad_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline / reference legs.  The CUDA package never imports it and
it never imports the CUDA package.

Each function marshals numpy arrays into the C routine of the same name; all of
the method's arithmetic lives in the C file, which cites the passage of the paper
each step follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kimad_oracle.c")
_LIB = os.path.join(_HERE, "libkimad_oracle.so")

STATUS_OK = 0
STATUS_INFEASIBLE = 1
STATUS_PLATEAU = 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no FMA contraction) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True, capture_output=True)
    return _LIB


class _Stats(C.Structure):
    _fields_ = [("budget_bytes", C.c_uint64), ("used_bytes", C.c_uint64), ("n_selected", C.c_uint64),
                ("total_err", C.c_float), ("status", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ko_bf16_rne.restype = C.c_uint16
        _lib.ko_bf16_rne.argtypes = [C.c_float]
        _lib.ko_budget_bytes.restype = C.c_uint64
        _lib.ko_budget_bytes.argtypes = [C.c_double, C.c_double]
        _lib.ko_get_threads.restype = C.c_int
    return _lib


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None else None


def _chk(rc, what):
    if rc < 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")
    return rc


def set_threads(n: int) -> None:
    lib().ko_set_threads(C.c_int(int(n)))


def get_threads() -> int:
    return int(lib().ko_get_threads())


def diff(grad: np.ndarray, g: np.ndarray) -> np.ndarray:
    grad = np.ascontiguousarray(grad, dtype=np.float32)
    g = np.ascontiguousarray(g, dtype=np.float32)
    assert grad.shape == g.shape
    d = np.empty_like(grad)
    lib().ko_diff(_p(grad, C.c_float), _p(g, C.c_float), _p(d, C.c_float), C.c_uint64(grad.size))
    return d


def k_table(layer_sizes, ratios) -> np.ndarray:
    ls = np.ascontiguousarray(layer_sizes, dtype=np.uint64)
    r = np.ascontiguousarray(ratios, dtype=np.float64)
    out = np.zeros((ls.size, r.size), dtype=np.uint64)
    _chk(lib().ko_k_table(_p(ls, C.c_uint64), C.c_uint32(ls.size), _p(r, C.c_double), C.c_uint32(r.size),
                          _p(out, C.c_uint64)), "k_table")
    return out


@dataclass
class Curve:
    err: np.ndarray      # float32 [K]
    tau: np.ndarray      # uint32 [K]  threshold key
    keep_eq: np.ndarray  # uint32 [K]  entries equal to tau that are kept
    n_gt: np.ndarray     # uint32 [K]
    n_eq: np.ndarray     # uint32 [K]


def layer_curve(d: np.ndarray, k_row) -> Curve:
    d = np.ascontiguousarray(d, dtype=np.float32)
    k = np.ascontiguousarray(k_row, dtype=np.uint64)
    K = k.size
    err = np.zeros(K, np.float32)
    tau, keq, ngt, neq = (np.zeros(K, np.uint32) for _ in range(4))
    _chk(lib().ko_layer_curve(_p(d, C.c_float), C.c_uint64(d.size), _p(k, C.c_uint64), C.c_uint32(K),
                              _p(err, C.c_float), _p(tau, C.c_uint32), _p(keq, C.c_uint32), _p(ngt, C.c_uint32),
                              _p(neq, C.c_uint32)), "layer_curve")
    return Curve(err, tau, keq, ngt, neq)


def _val_dtype(value_dtype):
    return np.float32 if value_dtype == 0 else np.uint16


def select_pack(d: np.ndarray, k: int, value_dtype: int = 0):
    d = np.ascontiguousarray(d, dtype=np.float32)
    idx = np.zeros(int(k), np.uint32)
    val = np.zeros(int(k), _val_dtype(value_dtype))
    _chk(lib().ko_select_pack(_p(d, C.c_float), C.c_uint64(d.size), C.c_uint64(int(k)), C.c_uint32(value_dtype),
                              _p(idx, C.c_uint32), val.ctypes.data_as(C.c_void_p)), "select_pack")
    return idx, val


def state_update(g: np.ndarray, idx: np.ndarray, val: np.ndarray, value_dtype: int = 0) -> np.ndarray:
    g = np.array(g, dtype=np.float32, copy=True)
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    val = np.ascontiguousarray(val, dtype=_val_dtype(value_dtype))
    lib().ko_state_update(_p(g, C.c_float), _p(idx, C.c_uint32), val.ctypes.data_as(C.c_void_p),
                          C.c_uint64(idx.size), C.c_uint32(value_dtype))
    return g


def bf16_rne(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    f = lib().ko_bf16_rne
    return np.array([f(C.c_float(float(v))) for v in x.ravel()], dtype=np.uint16).reshape(x.shape)


def budget_bytes(bandwidth_bytes_per_s: float, t_target_s: float) -> int:
    return int(lib().ko_budget_bytes(C.c_double(bandwidth_bytes_per_s), C.c_double(t_target_s)))


def units(ktab: np.ndarray, value_dtype: int, c: int, D: int):
    ktab = np.ascontiguousarray(ktab, dtype=np.uint64)
    L, K = ktab.shape
    out = np.zeros((L, K), np.uint64)
    st = _chk(lib().ko_units(_p(ktab, C.c_uint64), C.c_uint32(L), C.c_uint32(K), C.c_uint32(value_dtype),
                             C.c_uint64(int(c)), C.c_uint32(D), _p(out, C.c_uint64)), "units")
    return st, out


def dp(err: np.ndarray, units_tab: np.ndarray, D: int):
    """Returns (status, j[L], best_value, best_cell)."""
    err = np.ascontiguousarray(err, dtype=np.float32)
    u = np.ascontiguousarray(units_tab, dtype=np.uint64)
    L, K = err.shape
    assert u.shape == (L, K)
    j = np.zeros(L, np.uint32)
    bv = C.c_float(0)
    bc = C.c_uint32(0)
    st = _chk(lib().ko_dp(_p(err, C.c_float), _p(u, C.c_uint64), C.c_uint32(L), C.c_uint32(K), C.c_uint32(D),
                          _p(j, C.c_uint32), C.byref(bv), C.byref(bc)), "dp")
    return st, j, np.float32(bv.value), int(bc.value)


@dataclass
class StepResult:
    err: np.ndarray       # float32 [W][L][K]
    tau: np.ndarray       # uint32  [W][L][K]
    keep_eq: np.ndarray   # uint32  [W][L][K]
    j: np.ndarray         # uint32  [W][L]
    k: np.ndarray         # uint32  [W][L]
    idx: np.ndarray       # uint32  [W][cap]
    val: np.ndarray       # float32 or uint16 (bf16 bits) [W][cap]
    offs: np.ndarray      # uint64  [W][L+1]
    budget_bytes: np.ndarray
    used_bytes: np.ndarray
    n_selected: np.ndarray
    total_err: np.ndarray
    status: np.ndarray
    state: np.ndarray     # float32 [W][stride], the updated estimator
    dense: np.ndarray = None  # uint32 [W][L]: 1 where the chosen candidate is sent densely (cost model 1)


def uniform(ktab: np.ndarray, value_dtype: int, c: int):
    """O9: (status, j) of Kimad with one grid ratio for all layers under a budget of c bytes."""
    kt = np.ascontiguousarray(ktab, dtype=np.uint64)
    L, K = kt.shape
    j = C.c_uint32(0)
    rc = lib().ko_uniform(_p(kt, C.c_uint64), C.c_uint32(L), C.c_uint32(K), C.c_uint32(value_dtype), C.c_uint64(int(c)),
                          C.byref(j))
    if rc < 0:
        _chk(rc, "uniform")
    return rc, int(j.value)


def fit_ratio(layer_sizes, entries: int):
    """O9b: (status, q, k [L]) of the one ratio q / 2^32 sized to a budget of ``entries`` kept entries."""
    ls = np.ascontiguousarray(layer_sizes, dtype=np.uint64)
    k = np.zeros(ls.size, np.uint64)
    q = C.c_uint64(0)
    rc = lib().ko_fit_ratio(_p(ls, C.c_uint64), C.c_uint32(ls.size), C.c_uint64(int(entries)), C.byref(q), _p(k, C.c_uint64))
    if rc < 0:
        _chk(rc, "fit_ratio")
    return rc, int(q.value), k


def candidate(n: int, k: int, value_dtype: int, cost_model: int):
    """O13: (bytes, entries kept, dense flag) of candidate k of a layer of n elements."""
    b, ke, dn = C.c_uint64(0), C.c_uint64(0), C.c_int(0)
    lib().ko_candidate(C.c_uint64(int(n)), C.c_uint64(int(k)), C.c_uint32(value_dtype), C.c_uint32(cost_model),
                       C.byref(b), C.byref(ke), C.byref(dn))
    return int(b.value), int(ke.value), int(dn.value)


def units_from_bytes(bytes_tab: np.ndarray, c: int, D: int):
    bt = np.ascontiguousarray(bytes_tab, dtype=np.uint64)
    L, K = bt.shape
    out = np.zeros((L, K), np.uint64)
    st = _chk(lib().ko_units_from_bytes(_p(bt, C.c_uint64), C.c_uint32(L), C.c_uint32(K), C.c_uint64(int(c)), C.c_uint32(D),
                                        _p(out, C.c_uint64)), "units_from_bytes")
    return st, out


def dp_error_axis(err: np.ndarray, ktab: np.ndarray, D: int, value_dtype: int, c: int):
    """O12: (status, j [L], lowest feasible error cell) of the error-axis reading of Algorithm 3."""
    e = np.ascontiguousarray(err, dtype=np.float32)
    kt = np.ascontiguousarray(ktab, dtype=np.uint64)
    L, K = e.shape
    j = np.zeros(L, np.uint32)
    cell = C.c_uint32(0)
    rc = lib().ko_dp_error_axis(_p(e, C.c_float), _p(kt, C.c_uint64), C.c_uint32(L), C.c_uint32(K), C.c_uint32(D),
                                C.c_uint32(value_dtype), C.c_uint64(int(c)), _p(j, C.c_uint32), C.byref(cell))
    if rc < 0:
        _chk(rc, "dp_error_axis")
    return rc, j, int(cell.value)


def apply_packed(layer_sizes, idx, val, offs, value_dtype, est) -> np.ndarray:
    """O10: returns a copy of ``est`` ([N] float32) with one worker's packed message added."""
    ls = np.ascontiguousarray(layer_sizes, dtype=np.uint64)
    ix = np.ascontiguousarray(idx, dtype=np.uint32)
    vv = np.ascontiguousarray(val, dtype=_val_dtype(value_dtype))
    of = np.ascontiguousarray(offs, dtype=np.uint64)
    out = np.array(est, dtype=np.float32, copy=True)
    _chk(lib().ko_apply_packed(_p(ls, C.c_uint64), C.c_uint32(ls.size), _p(ix, C.c_uint32), vv.ctypes.data_as(C.c_void_p),
                               _p(of, C.c_uint64), C.c_uint32(value_dtype), _p(out, C.c_float)), "apply_packed")
    return out


def aggregate(x, est, weights, gamma) -> np.ndarray:
    """O11: returns x - gamma * sum_m w_m est[m] in float32, est [W][N]."""
    e = np.ascontiguousarray(est, dtype=np.float32)
    W, N = e.shape
    out = np.array(x, dtype=np.float32, copy=True).reshape(N)
    w = np.ascontiguousarray(weights, dtype=np.float32).reshape(W)
    _chk(lib().ko_aggregate(_p(out, C.c_float), _p(e, C.c_float), C.c_uint64(N), C.c_uint32(W), C.c_uint64(N),
                            _p(w, C.c_float), C.c_float(gamma)), "aggregate")
    return out


def step(layer_sizes, W, ratios, D, value_dtype, grads, state, bandwidth, t_target, cap=None,
         inject_err=None, policy=0, cost_model=0) -> StepResult:
    """One full pass O1..O8 for W workers; ``state`` is copied, the copy is updated and returned.
    policy 0: layer-adaptive DP (Kimad+); 1: one grid ratio for all layers (Kimad, O9); 2: the DP on the
    error axis (O12); 3: one ratio sized to the budget (O9b; ``ratios`` must have one entry, which plays no
    role).  cost_model 1: sizes with the dense fallback (O13)."""
    ls = np.ascontiguousarray(layer_sizes, dtype=np.uint64)
    r = np.ascontiguousarray(ratios, dtype=np.float64)
    L, K = ls.size, r.size
    N = int(ls.sum())
    grads = np.ascontiguousarray(grads, dtype=np.float32).reshape(W, -1)
    stride = grads.shape[1]
    st_new = np.array(state, dtype=np.float32, copy=True).reshape(W, stride)
    bw = np.ascontiguousarray(bandwidth, dtype=np.float64).reshape(W)
    if cap is None:
        cap = N
    err = np.zeros((W, L, K), np.float32)
    tau = np.zeros((W, L, K), np.uint32)
    keq = np.zeros((W, L, K), np.uint32)
    j = np.zeros((W, L), np.uint32)
    k = np.zeros((W, L), np.uint32)
    idx = np.zeros((W, cap), np.uint32)
    val = np.zeros((W, cap), _val_dtype(value_dtype))
    offs = np.zeros((W, L + 1), np.uint64)
    stats = (_Stats * W)()
    inj = None
    if inject_err is not None:
        inj = np.ascontiguousarray(inject_err, dtype=np.float32).reshape(W, L, K)
    dense = np.zeros((W, L), np.uint32)
    _chk(lib().ko_step_ex(C.c_uint32(policy), C.c_uint32(cost_model), _p(ls, C.c_uint64), C.c_uint32(L), C.c_uint32(W), _p(r, C.c_double), C.c_uint32(K),
                       C.c_uint32(D), C.c_uint32(value_dtype), C.c_uint64(stride), _p(grads, C.c_float),
                       _p(st_new, C.c_float), _p(bw, C.c_double), C.c_double(t_target), _p(inj, C.c_float),
                       _p(err, C.c_float), _p(tau, C.c_uint32), _p(keq, C.c_uint32), _p(j, C.c_uint32),
                       _p(k, C.c_uint32), _p(idx, C.c_uint32), val.ctypes.data_as(C.c_void_p), C.c_uint64(cap),
                       _p(offs, C.c_uint64), stats, _p(dense, C.c_uint32)), "step")
    return StepResult(err, tau, keq, j, k, idx, val, offs,
                      np.array([s.budget_bytes for s in stats], np.uint64),
                      np.array([s.used_bytes for s in stats], np.uint64),
                      np.array([s.n_selected for s in stats], np.uint64),
                      np.array([s.total_err for s in stats], np.float32),
                      np.array([s.status for s in stats], np.int32), st_new, dense)
