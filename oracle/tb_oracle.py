"""ctypes front end of the CPU oracle (``tb_oracle.c``) -- test infrastructure, not product code.

Only tests, the smoke check and the benchmark's cpu_baseline / reference legs may import this
module.  It never imports the CUDA package; the CUDA package never imports it.

Arrays are numpy: fp32 storage as ``float32``, bf16 storage as ``uint16`` (the raw 16 bits).
Every function cites the passage of the paper that defines the step it wraps (see the header of
``tb_oracle.c`` for the full list).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

F32, BF16 = 0, 1
GROUP_SUM, GROUP_MAX = 0, 1
NEIGHBOR_DILATE, NEIGHBOR_CLUSTER = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tb_oracle.c")
_LIB = os.path.join(_HERE, "liborc.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (``-O2 -fopenmp``); returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Unit(C.Structure):
    _fields_ = [("K", C.c_void_p), ("V", C.c_void_p), ("Kimp", C.c_void_p), ("q_imp", C.c_void_p),
                ("q", C.c_void_p), ("idx", C.c_void_p), ("cnt", C.c_void_p), ("out", C.c_void_p),
                ("lse", C.c_void_p), ("L", C.c_int32), ("refresh", C.c_int32)]


class _Params(C.Structure):
    _fields_ = [("g", C.c_int32), ("D", C.c_int32), ("dp", C.c_int32), ("dtype", C.c_int32),
                ("budget", C.c_int32), ("sinks", C.c_int32), ("recent", C.c_int32), ("radius", C.c_int32),
                ("nmode", C.c_int32), ("reduce", C.c_int32), ("score_scale", C.c_double), ("sm_scale", C.c_double)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_select.restype = C.c_int
        _lib.orc_neighbors.restype = C.c_int
        _lib.orc_attended_set.restype = C.c_int
        _lib.orc_max_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p)


def storage_dtype(dtype: int):
    return np.uint16 if dtype == BF16 else np.float32


def _chk(a, dtype=None):
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    if dtype is not None:
        assert a.dtype == storage_dtype(dtype), (a.dtype, dtype)
    return a


def round_to_storage(x: np.ndarray, dtype: int) -> np.ndarray:
    """fp64 -> storage type, one round-to-nearest-even step."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, storage_dtype(dtype))
    lib().orc_round_to_storage(_p(x), C.c_size_t(x.size), C.c_int(dtype), _p(out))
    return out


def widen(x: np.ndarray, dtype: int) -> np.ndarray:
    """storage type -> fp64, exact."""
    x = _chk(np.ascontiguousarray(x), dtype)
    out = np.empty(x.shape, np.float64)
    lib().orc_widen(_p(x), C.c_size_t(x.size), C.c_int(dtype), _p(out))
    return out


def project_keys(K: np.ndarray, W: np.ndarray, dtype: int, want_f64: bool = False):
    """Sec. 3.1 key-cache projection: K [T,D] . W [D,d'] -> K_imp [T,d'] in the storage type."""
    _chk(K, dtype), _chk(W, dtype)
    T, D = K.shape
    dp = W.shape[1]
    assert W.shape[0] == D
    out = np.empty((T, dp), storage_dtype(dtype))
    f64 = np.empty((T, dp), np.float64) if want_f64 else None
    lib().orc_project_keys(_p(K), _p(W), C.c_int(T), C.c_int(D), C.c_int(dp), C.c_int(dtype), _p(out),
                           _p(f64) if want_f64 else None)
    return (out, f64) if want_f64 else out


def score(q_imp: np.ndarray, kimp: np.ndarray, dtype: int, reduce: int = GROUP_SUM, scale: float = 1.0) -> np.ndarray:
    """Sec. 3.4 importance scores of all L cached tokens for one KV head.  q_imp [g,d'] fp32."""
    q_imp = np.ascontiguousarray(q_imp, dtype=np.float32)
    _chk(kimp, dtype)
    g, dp = q_imp.shape
    L = kimp.shape[0]
    assert kimp.shape[1] == dp
    s = np.empty(L, np.float64)
    lib().orc_score(_p(q_imp), C.c_int(g), C.c_int(reduce), _p(kimp), C.c_int(L), C.c_int(dp), C.c_int(dtype),
                    C.c_double(scale), _p(s))
    return s


def candidate_range(L: int, S: int, W: int):
    lo, hi = C.c_int(), C.c_int()
    lib().orc_candidate_range(C.c_int(L), C.c_int(S), C.c_int(W), C.byref(lo), C.byref(hi))
    return lo.value, hi.value


def select(s: np.ndarray, S: int, W: int, budget: int) -> np.ndarray:
    """Sec. 4 token selection policy: ascending positions of the top-`budget` candidates."""
    s = np.ascontiguousarray(s, dtype=np.float64)
    idx = np.empty(max(budget, 1), np.int32)
    n = lib().orc_select(_p(s), C.c_int(s.shape[0]), C.c_int(S), C.c_int(W), C.c_int(budget), _p(idx))
    return idx[:n].copy()


def neighbors(idx: np.ndarray, r: int, mode: int, lo: int, hi: int) -> np.ndarray:
    """Sec. 3.4 neighbour fetching on an ascending selection inside [lo, hi)."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    out = np.empty(max(1, (2 * r + 1) * idx.shape[0]), np.int32)
    n = lib().orc_neighbors(_p(idx), C.c_int(idx.shape[0]), C.c_int(r), C.c_int(mode), C.c_int(lo), C.c_int(hi), _p(out))
    return out[:n].copy()


def attended_set(L: int, S: int, W: int, I: np.ndarray) -> np.ndarray:
    """Sec. 3.3: sinks + important list + local window at the current length."""
    I = np.ascontiguousarray(I, dtype=np.int32)
    A = np.empty(max(1, min(S, L) + I.shape[0] + W), np.int32)
    n = lib().orc_attended_set(C.c_int(L), C.c_int(S), C.c_int(W), _p(I), C.c_int(I.shape[0]), _p(A))
    return A[:n].copy()


def attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, A: np.ndarray, dtype: int, sm_scale: float | None = None):
    """Sec. 3.3 softmax attention of g query heads over rows A of one KV head.  Returns (out, lse)."""
    _chk(q, dtype), _chk(K, dtype), _chk(V, dtype)
    A = np.ascontiguousarray(A, dtype=np.int32)
    g, D = q.shape
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(D)
    out = np.empty((g, D), np.float64)
    lse = np.empty(g, np.float64)
    lib().orc_attention(_p(q), _p(K), _p(V), _p(A), C.c_int(A.shape[0]), C.c_int(g), C.c_int(D), C.c_int(dtype),
                        C.c_double(sm_scale), _p(out), _p(lse))
    return out, lse


def dense_attention(q, K, V, dtype, sm_scale=None):
    """Dense rule (prefill / first decode token): every cached row is attended."""
    return attention(q, K, V, np.arange(K.shape[0], dtype=np.int32), dtype, sm_scale)


def is_prediction_step(step: int, interval: int) -> bool:
    """Sec. 3.4 prediction interval: does decode step `step` (0 = first sparse step) re-select?"""
    v = lib().orc_is_prediction_step(C.c_int(step), C.c_int(interval))
    assert v >= 0, "step >= 0 and interval >= 1"
    return bool(v)


class Unit:
    """One (sequence, layer, KV head): its caches and the stale selection (Sec. 3.4 interval)."""

    def __init__(self, K, V, Kimp, cap):
        self.K, self.V, self.Kimp = K, V, Kimp  # full-capacity arrays; rows [0, L) valid
        self.idx = np.zeros(max(1, cap), np.int32)
        self.cnt = np.zeros(1, np.int32)


def step_units(units, Ls, q_imps, qs, refresh, *, g, D, dp, dtype, budget, sinks, recent, radius=0,
               nmode=NEIGHBOR_DILATE, reduce=GROUP_SUM, score_scale=1.0, sm_scale=None, n_threads=1, want_lse=False):
    """Run one decode step for independent units (OpenMP over units only).

    refresh[i] != 0: score + select + neighbours, result stored in the unit (Sec. 3.4, prediction step);
    otherwise the unit's stale list is reused.  Then attention over sinks + list + window (Sec. 3.3).
    Returns out [n_units, g, D] fp64 (and lse [n_units, g])."""
    n = len(units)
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(D)
    out = np.empty((n, g, D), np.float64)
    lse = np.empty((n, g), np.float64)
    arr = (_Unit * n)()
    keep = []
    for i, u in enumerate(units):
        qi = np.ascontiguousarray(q_imps[i], dtype=np.float32)
        q = _chk(np.ascontiguousarray(qs[i]), dtype)
        keep += [qi, q]
        arr[i].K, arr[i].V, arr[i].Kimp = u.K.ctypes.data, u.V.ctypes.data, u.Kimp.ctypes.data
        arr[i].q_imp, arr[i].q = qi.ctypes.data, q.ctypes.data
        arr[i].idx, arr[i].cnt = u.idx.ctypes.data, u.cnt.ctypes.data
        arr[i].out, arr[i].lse = out[i].ctypes.data, lse[i].ctypes.data
        arr[i].L, arr[i].refresh = int(Ls[i]), int(refresh[i])
    p = _Params(g, D, dp, dtype, budget, sinks, recent, radius, nmode, reduce, score_scale, sm_scale)
    lib().orc_step_units(arr, C.c_int(n), C.byref(p), C.c_int(n_threads))
    return (out, lse) if want_lse else out


ACT_GELU, ACT_SILU, ACT_RELU = 0, 1, 2


def predict_queries(H: np.ndarray, ln_w: np.ndarray, ln_b: np.ndarray, W1: np.ndarray, W2: np.ndarray, dtype: int,
                    eps: float = 1e-5, act: int = ACT_GELU) -> np.ndarray:
    """Importance queries of the predictor (Sec. 3.1 "Query prediction", App. A): q = W2 act(W1 LN(h)) per
    token.  All inputs are stored values (``dtype``): H [tokens, E], ln_w / ln_b [E], W1 [hidden, E],
    W2 [out, hidden]; returns float64 [tokens, out]."""
    H, ln_w, ln_b, W1, W2 = (widen(_chk(a, dtype), dtype) for a in (H, ln_w, ln_b, W1, W2))
    n_tok, E = H.shape
    hid, out = W1.shape[0], W2.shape[0]
    assert W1.shape == (hid, E) and W2.shape == (out, hid) and ln_w.shape == (E,) and ln_b.shape == (E,)
    q = np.empty((n_tok, out), np.float64)
    lib().orc_predict_queries(_p(H), n_tok, E, _p(ln_w), _p(ln_b), C.c_double(eps), _p(W1), hid, _p(W2), out, act, _p(q))
    return q


def max_threads() -> int:
    return lib().orc_max_threads()
