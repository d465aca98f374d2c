"""ctypes front end of the CPU oracle (``psattn_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
CPU-baseline timing of the benchmark.  The CUDA library and its Python binding
never import this module.  All arithmetic is in the C file; this module only
builds it with gcc on first use and marshals numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "psattn_oracle.c")
_SO = os.path.join(_HERE, "libpsattn_oracle.so")
_lock = threading.Lock()
_lib = None

_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source (gcc -O2 -fopenmp)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    with _lock:
        if _lib is None:
            _lib = ctypes.CDLL(build())
            _lib.psattn_oracle_count.restype = ctypes.c_int
            _lib.psattn_oracle_count.argtypes = [ctypes.c_double, ctypes.c_int]
            _lib.psattn_oracle_max_threads.restype = ctypes.c_int
    return _lib


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _i32(a):
    if a is None:
        return None, None
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(_i32p)


def count(c: float, length: int) -> int:
    """n(c, len) = clamp(ceil(c ln len), 1, len): the sample size and the number selected."""
    return int(_load().psattn_oracle_count(float(c), int(length)))


def max_threads() -> int:
    return int(_load().psattn_oracle_max_threads())


def _idx_info(sample_idx, B, H, T):
    sample_idx = np.ascontiguousarray(sample_idx, dtype=np.int32)
    if sample_idx.ndim == 3:
        assert sample_idx.shape[:2] == (B, T)
        return sample_idx, 0
    assert sample_idx.ndim == 4 and sample_idx.shape[:3] == (B, H, T)
    return sample_idx, 1


def measure(Q, K, sample_idx, lengths=None, c=5.0, U_override=0):
    """Eq. 11 for every query.  Returns float64 [B, H, T] (zero at padded positions)."""
    lib = _load()
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    B, H, T, d = Q.shape
    idx, per_head = _idx_info(sample_idx, B, H, T)
    lengths, lp = _i32(lengths)
    M = np.zeros((B, H, T), dtype=np.float64)
    lib.psattn_oracle_measure(qp, kp, B, H, T, d, lp, idx.ctypes.data_as(_i32p),
                              int(idx.shape[-1]), per_head, ctypes.c_double(c),
                              int(U_override), M.ctypes.data_as(_f64p))
    return M


def exact_measure(Q, K, lengths=None):
    """Eq. 10 (log-sum-exp minus mean over all valid keys).  float64 [B, H, T]."""
    lib = _load()
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    B, H, T, d = Q.shape
    lengths, lp = _i32(lengths)
    M = np.zeros((B, H, T), dtype=np.float64)
    lib.psattn_oracle_exact_measure(qp, kp, B, H, T, d, lp, M.ctypes.data_as(_f64p))
    return M


def selected_count(length: int, c: float = 5.0, u_override: int = 0, r_sparse: float = 0.0) -> int:
    """Number of selected queries of a sequence: n(c, len), or ceil(r_sparse * len) in [1, len]
    (Sec. 3.2's L_sparse = r_sparse L) when r_sparse > 0, or min(u_override, len)."""
    lib = _load()
    lib.psattn_oracle_selected_count.restype = ctypes.c_int
    return int(lib.psattn_oracle_selected_count(ctypes.c_double(c), int(u_override),
                                                ctypes.c_double(r_sparse), int(length)))


def select(M, lengths=None, c=5.0, u_override=0, u_max=None, r_sparse=0.0):
    """Top-u query indices per (batch, head): int32 [B, H, u_max], ascending, -1 padded."""
    lib = _load()
    M = np.ascontiguousarray(M, dtype=np.float64)
    B, H, T = M.shape
    lengths, lp = _i32(lengths)
    if u_max is None:
        u_max = u_bound(T, c, u_override, r_sparse)
    sel = np.full((B, H, u_max), -1, dtype=np.int32)
    lib.psattn_oracle_select(M.ctypes.data_as(_f64p), B, H, T, lp, ctypes.c_double(c),
                             int(u_override), ctypes.c_double(r_sparse),
                             sel.ctypes.data_as(_i32p), int(u_max))
    return sel


def u_bound(T, c, u_override=0, r_sparse=0.0):
    """Largest number of selected queries any sequence of length <= T can have."""
    if r_sparse > 0:
        return selected_count(int(T), c, 0, r_sparse) if T > 0 else 0
    if u_override > 0:
        return min(int(u_override), int(T))
    return max(count(c, L) for L in range(1, int(T) + 1)) if T > 0 else 0


def mean_v(V, lengths=None):
    """Column mean of V over valid keys: float64 [B, H, d]."""
    lib = _load()
    V, vp = _f32(V)
    B, H, T, d = V.shape
    lengths, lp = _i32(lengths)
    out = np.zeros((B, H, d), dtype=np.float64)
    lib.psattn_oracle_mean_v(vp, B, H, T, d, lp, out.ctypes.data_as(_f64p))
    return out


def attend_row(Q, K, V, b, h, i, length=None):
    """Eq. 7-8 for one query over the first ``length`` keys: float64 [d]."""
    lib = _load()
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    B, H, T, d = Q.shape
    out = np.zeros(d, dtype=np.float64)
    lib.psattn_oracle_attend_row(qp, kp, vp, H, T, d, int(T if length is None else length),
                                 int(b), int(h), int(i), out.ctypes.data_as(_f64p))
    return out


def forward(Q, K, V, sample_idx, lengths=None, c=5.0, u_override=0, U_override=0,
            fill="mean_v", sel_in=None, nthreads=1, r_sparse=0.0):
    """Steps (a)-(e).  Returns (O float64 [B,H,T,d], sel_idx int32 [B,H,u_max], M float64 [B,H,T])."""
    lib = _load()
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    B, H, T, d = Q.shape
    idx, per_head = _idx_info(sample_idx, B, H, T)
    lengths, lp = _i32(lengths)
    if sel_in is not None:
        sel_in = np.ascontiguousarray(sel_in, dtype=np.int32)
        u_max = int(sel_in.shape[-1])
        sp = sel_in.ctypes.data_as(_i32p)
    else:
        u_max = u_bound(T, c, u_override, r_sparse)
        sp = None
    O = np.zeros((B, H, T, d), dtype=np.float64)
    M = np.zeros((B, H, T), dtype=np.float64)
    sel = np.full((B, H, u_max), -1, dtype=np.int32)
    lib.psattn_oracle_forward(qp, kp, vp, B, H, T, d, lp, idx.ctypes.data_as(_i32p),
                              int(idx.shape[-1]), per_head, ctypes.c_double(c),
                              int(u_override), ctypes.c_double(r_sparse), int(U_override),
                              {"mean_v": 0, "own_v": 1}[fill], sp,
                              O.ctypes.data_as(_f64p), M.ctypes.data_as(_f64p),
                              sel.ctypes.data_as(_i32p), u_max, int(nthreads))
    return O, sel, M


def dense(Q, K, V, lengths=None, nthreads=1):
    """Eq. 6 for every valid query (zero rows at padded positions): float64 [B,H,T,d]."""
    lib = _load()
    Q, qp = _f32(Q)
    K, kp = _f32(K)
    V, vp = _f32(V)
    B, H, T, d = Q.shape
    lengths, lp = _i32(lengths)
    O = np.zeros((B, H, T, d), dtype=np.float64)
    lib.psattn_oracle_dense(qp, kp, vp, B, H, T, d, lp, O.ctypes.data_as(_f64p), int(nthreads))
    return O


def project_qkv(X, Wt, H, lengths=None, nthreads=1):
    """Sec. 3.1: Q = X W_q, K = X W_k, V = X W_v per head.  X [B, T, d_x]; Wt [3, H*d, d_x] holds the
    matrices transposed (row h*d + e = column e of head h).  Returns float64 (Q, K, V), each
    [B, H, T, d], zero at padded positions."""
    lib = _load()
    X, xp = _f32(X)
    Wt, wp = _f32(Wt)
    B, T, dx = X.shape
    assert Wt.ndim == 3 and Wt.shape[0] == 3 and Wt.shape[2] == dx and Wt.shape[1] % H == 0
    d = Wt.shape[1] // H
    lengths, lp = _i32(lengths)
    out = np.zeros((3, B, H, T, d), dtype=np.float64)
    lib.psattn_oracle_project_qkv(xp, wp, B, T, dx, int(H), d, lp, out.ctypes.data_as(_f64p),
                                  int(nthreads))
    return out[0], out[1], out[2]


def project_out(O, Wot, lengths=None, nthreads=1):
    """The output matrix of the attention module: Y[b, t, :] = sum_h O[b, h, t, :] W_o^h.  O [B, H, T, d];
    Wot [d_y, H*d] holds W_o transposed (Wot[n, h*d + e] = W_o[h*d + e, n]).  Returns float64 [B, T, d_y],
    zero at padded positions."""
    lib = _load()
    O, op = _f32(O)
    Wot, wp = _f32(Wot)
    B, H, T, d = O.shape
    assert Wot.ndim == 2 and Wot.shape[1] == H * d
    dy = int(Wot.shape[0])
    lengths, lp = _i32(lengths)
    Y = np.zeros((B, T, dy), dtype=np.float64)
    lib.psattn_oracle_project_out(op, wp, B, H, T, d, dy, lp, Y.ctypes.data_as(_f64p), int(nthreads))
    return Y
