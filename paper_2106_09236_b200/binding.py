"""Thin ctypes binding of libpsattn.so: same names as include/psattn.h, argument marshalling
only.  torch supplies device memory and streams; every step of the computation runs in the
library's CUDA kernels.  There is no fallback: if the library cannot be loaded or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

PSATTN_BF16, PSATTN_FP32 = 0, 1
PSATTN_FILL_MEAN_V, PSATTN_FILL_OWN_V = 0, 1
PSATTN_PATH_AUTO, PSATTN_PATH_STAGED, PSATTN_PATH_FUSED = 0, 1, 2

EXPORTS = [
    "psattn_version", "psattn_launch_count", "psattn_status_string", "psattn_last_cuda_error", "psattn_count",
    "psattn_plan_create", "psattn_plan_destroy", "psattn_plan_limits", "psattn_workspace_bytes",
    "psattn_forward", "psattn_forward_with_selection", "psattn_measure", "psattn_exact_measure", "psattn_select",
    "psattn_mean_v", "psattn_attend_rows", "psattn_dense_forward", "psattn_read_status",
    "psattn_plan_enable_host_io", "psattn_forward_host", "psattn_mean_v_noalloc", "psattn_project_qkv",
    "psattn_probe_gather", "psattn_project_out", "psattn_plan_debug_waits",
]


class psattn_desc_t(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("T_max", ctypes.c_int32),
        ("d_head", ctypes.c_int32), ("dtype", ctypes.c_int32), ("fill_mode", ctypes.c_int32),
        ("u_override", ctypes.c_int32), ("U_override", ctypes.c_int32),
        ("idx_cols", ctypes.c_int32), ("idx_per_head", ctypes.c_int32),
        ("path", ctypes.c_int32), ("idx_shared", ctypes.c_int32), ("c", ctypes.c_double),
        ("r_sparse", ctypes.c_double),
        ("q_stride", ctypes.c_int64 * 3), ("k_stride", ctypes.c_int64 * 3),
        ("v_stride", ctypes.c_int64 * 3), ("o_stride", ctypes.c_int64 * 3),
    ]


class PsattnError(RuntimeError):
    pass


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True):
    """Loads libpsattn.so (building it with nvcc first if it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    override = os.environ.get("PSATTN_LIBRARY")          # another build of the same library (the benchmark's --phases mode)
    if override:
        path = override
    elif build_if_missing:
        path = _build.build()
    if not os.path.exists(path):
        raise PsattnError("libpsattn.so is missing: run paper_2106_09236_b200/build.py")
    lib = ctypes.CDLL(path)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    lib.psattn_version.restype = ctypes.c_int
    lib.psattn_launch_count.restype = ctypes.c_ulonglong
    lib.psattn_status_string.restype = ctypes.c_char_p
    lib.psattn_status_string.argtypes = [ctypes.c_int]
    lib.psattn_last_cuda_error.argtypes = [vp]
    lib.psattn_count.argtypes = [ctypes.c_double, ctypes.c_int]
    lib.psattn_plan_create.argtypes = [ctypes.POINTER(psattn_desc_t), ctypes.POINTER(vp)]
    lib.psattn_plan_destroy.argtypes = [vp]
    lib.psattn_plan_limits.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.psattn_workspace_bytes.argtypes = [vp, ctypes.POINTER(sz)]
    lib.psattn_forward.argtypes = [vp] * 10 + [sz, vp]
    lib.psattn_forward_with_selection.argtypes = [vp] * 8 + [sz, vp]
    lib.psattn_measure.argtypes = [vp] * 7 + [sz, vp]
    lib.psattn_exact_measure.argtypes = [vp] * 6 + [sz, vp]
    lib.psattn_select.argtypes = [vp] * 5 + [sz, vp]
    lib.psattn_project_qkv.argtypes = [vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.psattn_mean_v.argtypes = [vp] * 5 + [sz, vp]
    lib.psattn_project_out.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, sz, vp]
    lib.psattn_attend_rows.argtypes = [vp] * 6 + [i32, vp, vp, sz, vp]
    lib.psattn_dense_forward.argtypes = [vp] * 7 + [sz, vp]
    lib.psattn_read_status.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.psattn_plan_enable_host_io.argtypes = [vp]
    lib.psattn_forward_host.argtypes = [vp] * 9
    lib.psattn_mean_v_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
    lib.psattn_plan_debug_waits.argtypes = [vp, ctypes.c_uint64, ctypes.c_uint32]
    lib.psattn_probe_gather.argtypes = [i32, vp, ctypes.c_int64, i32, i32, i32, vp, vp]
    _lib = lib
    return lib


def _check(rc: int, plan=None):
    if rc != 0:
        lib = load()
        msg = lib.psattn_status_string(rc).decode()
        if plan is not None and rc == 6:
            msg += " (cudaError %d)" % lib.psattn_last_cuda_error(plan)
        raise PsattnError("psattn status %d: %s" % (rc, msg))


def _ptr(t):
    if t is None:
        return None
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def psattn_version() -> int:
    return load().psattn_version()


def psattn_launch_count() -> int:
    return int(load().psattn_launch_count())


def psattn_count(c: float, length: int) -> int:
    return load().psattn_count(float(c), int(length))


def psattn_mean_v_noalloc(V, lengths, vbar, B, H, T_max):
    """mean(V) over valid rows without any allocation: no plan, no workspace.  `vbar` (fp32
    [B, H, 64], device) must be provided by the caller and is filled in place.  For callers
    that may not allocate device memory; see include/psattn.h for capacity and sharing rules."""
    dtype = PSATTN_BF16 if V.dtype == torch.bfloat16 else PSATTN_FP32
    _check(load().psattn_mean_v_noalloc(_ptr(V), _ptr(lengths), _ptr(vbar), int(B), int(H),
                                        int(T_max), dtype, _stream()))
    return vbar


def psattn_probe_gather(mode, rows, n_ctas, warps_per_cta, rounds_per_warp, sink):
    """Launches the gather microbenchmark (see include/psattn.h); returns the number of 128-byte rows it reads."""
    n_rows = 0 if rows is None else rows.numel() * rows.element_size() // 128
    _check(load().psattn_probe_gather(int(mode), _ptr(rows), n_rows, int(n_ctas), int(warps_per_cta),
                                      int(rounds_per_warp), _ptr(sink), _stream()))
    per = {0: 1, 1: 2, 2: 4, 3: 1, 4: 2, 5: 4, 6: 1, 7: 2, 8: 4, 11: 4, 12: 4}[int(mode)]   # the round count is a multiple of this
    rounds = int(rounds_per_warp) // per * per
    if int(mode) == 12:                                     # every sixth warp takes half as many rounds
        n_bulk = len([w for w in range(int(warps_per_cta)) if w % 6 == 5])
        return int(n_ctas) * ((int(warps_per_cta) - n_bulk) * rounds + n_bulk * (rounds // 2)) * 16
    return int(n_ctas) * int(warps_per_cta) * rounds * 16


class Plan:
    """Owns a psattn_plan_t and a zero-initialised workspace tensor on the current device."""

    def __init__(self, B, H, T_max, dtype=torch.bfloat16, c=5.0, idx_cols=None, d_head=64,
                 fill_mode=PSATTN_FILL_MEAN_V, u_override=0, U_override=0, idx_per_head=False,
                 path=PSATTN_PATH_AUTO, strides=None, idx_shared=False, r_sparse=0.0):
        lib = load()
        self.lib = lib
        d = psattn_desc_t()
        d.B, d.H, d.T_max, d.d_head = B, H, T_max, d_head
        d.dtype = PSATTN_BF16 if dtype == torch.bfloat16 else PSATTN_FP32
        d.fill_mode, d.u_override, d.U_override = fill_mode, u_override, U_override
        if idx_cols is None:
            idx_cols = U_override if U_override > 0 else max(
                [psattn_count(c, L) for L in range(1, T_max + 1)] + [1])
        d.idx_cols, d.idx_per_head, d.path, d.c = idx_cols, int(idx_per_head), path, c
        d.idx_shared = int(idx_shared)
        d.r_sparse = float(r_sparse)
        if strides is not None:
            for name in ("q", "k", "v", "o"):
                if name in strides:
                    getattr(d, name + "_stride")[:] = list(strides[name])
        self.desc = d
        self.dtype = dtype
        h = ctypes.c_void_p()
        _check(lib.psattn_plan_create(ctypes.byref(d), ctypes.byref(h)))
        self.handle = h
        um, Um = ctypes.c_int32(), ctypes.c_int32()
        _check(lib.psattn_plan_limits(h, ctypes.byref(um), ctypes.byref(Um)))
        self.u_max, self.U_max = um.value, Um.value
        nbytes = ctypes.c_size_t()
        _check(lib.psattn_workspace_bytes(h, ctypes.byref(nbytes)))
        self.workspace_bytes = nbytes.value
        self.workspace = torch.zeros(nbytes.value, dtype=torch.uint8, device="cuda")
        self.B, self.H, self.T_max, self.d_head, self.idx_cols = B, H, T_max, d_head, idx_cols

    def close(self):
        if getattr(self, "handle", None):
            self.lib.psattn_plan_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ws(self):
        return _ptr(self.workspace), ctypes.c_size_t(self.workspace_bytes)

    # -- same names as the C entry points --------------------------------------------------
    def psattn_forward(self, Q, K, V, lengths, sample_idx, O=None, sel_idx=None, M_out=None):
        if O is None:
            O = torch.empty((self.B, self.H, self.T_max, self.d_head), dtype=self.dtype, device=Q.device)
        if sel_idx is None:
            sel_idx = torch.empty((self.B, self.H, self.u_max), dtype=torch.int32, device=Q.device)
        ws, n = self._ws()
        _check(self.lib.psattn_forward(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths),
                                       _ptr(sample_idx), _ptr(O), _ptr(sel_idx), _ptr(M_out),
                                       ws, n, _stream()), self.handle)
        return O, sel_idx

    def psattn_forward_with_selection(self, Q, K, V, lengths, sel_idx_in, O=None):
        if O is None:
            O = torch.empty((self.B, self.H, self.T_max, self.d_head), dtype=self.dtype, device=Q.device)
        ws, n = self._ws()
        _check(self.lib.psattn_forward_with_selection(self.handle, _ptr(Q), _ptr(K), _ptr(V),
                                                      _ptr(lengths), _ptr(sel_idx_in), _ptr(O),
                                                      ws, n, _stream()), self.handle)
        return O

    def psattn_measure(self, Q, K, lengths, sample_idx, M_out=None):
        if M_out is None:
            M_out = torch.empty((self.B, self.H, self.T_max), dtype=torch.float32, device=Q.device)
        ws, n = self._ws()
        _check(self.lib.psattn_measure(self.handle, _ptr(Q), _ptr(K), _ptr(lengths),
                                       _ptr(sample_idx), _ptr(M_out), ws, n, _stream()), self.handle)
        return M_out

    def psattn_exact_measure(self, Q, K, lengths, M_out=None):
        if M_out is None:
            M_out = torch.empty((self.B, self.H, self.T_max), dtype=torch.float32, device=Q.device)
        ws, n = self._ws()
        _check(self.lib.psattn_exact_measure(self.handle, _ptr(Q), _ptr(K), _ptr(lengths), _ptr(M_out),
                                             ws, n, _stream()), self.handle)
        return M_out

    def psattn_project_qkv(self, X, Wt, lengths=None, Q=None, K=None, V=None, vbar=None):
        """Q, K, V = X W_q, X W_k, X W_v in the attention layout; X [B, T_max, d_x], Wt [3, H*64, d_x].
        Rows at padded positions of freshly allocated outputs are zero (the kernel does not write them)."""
        outs = []
        for t in (Q, K, V):
            if t is None:
                t = torch.zeros((self.B, self.H, self.T_max, self.d_head), dtype=self.dtype, device=X.device)
            outs.append(t)
        ws, n = self._ws()
        _check(self.lib.psattn_project_qkv(self.handle, _ptr(X), _ptr(Wt), int(X.shape[-1]), _ptr(lengths),
                                           _ptr(outs[0]), _ptr(outs[1]), _ptr(outs[2]), _ptr(vbar), ws, n,
                                           _stream()), self.handle)
        return tuple(outs)

    def psattn_project_out(self, O, sel_idx, lengths, Wot, Y=None):
        """Y[b, t, :] = sum_h O[b, h, t, :] W_o^h; Wot [d_y, H*64] holds W_o transposed.  With sel_idx (the index
        sets psattn_forward wrote for this O) the broadcast-plus-corrections form runs, with None the dense product.
        Rows at padded positions of a freshly allocated Y are zero (the kernels do not write them)."""
        d_y = int(Wot.shape[0])
        if Y is None:
            Y = torch.zeros((self.B, self.T_max, d_y), dtype=self.dtype, device=O.device)
        ws, n = self._ws()
        _check(self.lib.psattn_project_out(self.handle, _ptr(O), _ptr(sel_idx), _ptr(lengths), _ptr(Wot), d_y,
                                           _ptr(Y), ws, n, _stream()), self.handle)
        return Y

    def psattn_select(self, M, lengths, sel_idx=None):
        if sel_idx is None:
            sel_idx = torch.empty((self.B, self.H, self.u_max), dtype=torch.int32, device=M.device)
        ws, n = self._ws()
        _check(self.lib.psattn_select(self.handle, _ptr(M), _ptr(lengths), _ptr(sel_idx), ws, n,
                                      _stream()), self.handle)
        return sel_idx

    def psattn_mean_v(self, V, lengths, vbar=None):
        if vbar is None:
            vbar = torch.empty((self.B, self.H, self.d_head), dtype=torch.float32, device=V.device)
        ws, n = self._ws()
        _check(self.lib.psattn_mean_v(self.handle, _ptr(V), _ptr(lengths), _ptr(vbar), ws, n,
                                      _stream()), self.handle)
        return vbar

    def psattn_attend_rows(self, Q, K, V, lengths, row_idx, out=None):
        n_rows = int(row_idx.shape[-1])
        if out is None:
            out = torch.empty((self.B, self.H, n_rows, self.d_head), dtype=torch.float32, device=Q.device)
        ws, n = self._ws()
        _check(self.lib.psattn_attend_rows(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths),
                                           _ptr(row_idx), n_rows, _ptr(out), ws, n, _stream()),
               self.handle)
        return out

    def psattn_dense_forward(self, Q, K, V, lengths, O=None):
        if O is None:
            O = torch.empty((self.B, self.H, self.T_max, self.d_head), dtype=self.dtype, device=Q.device)
        ws, n = self._ws()
        _check(self.lib.psattn_dense_forward(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths),
                                             _ptr(O), ws, n, _stream()), self.handle)
        return O

    def psattn_read_status(self) -> int:
        bits = ctypes.c_uint32()
        _check(self.lib.psattn_read_status(self.handle, _ptr(self.workspace), _stream(),
                                           ctypes.byref(bits)), self.handle)
        return bits.value

    def psattn_plan_debug_waits(self, wait_limit_ns=0, extra_expected_bytes=0):
        """Test hook: shorten the bounded device-side waits and/or make the first TMA barrier never complete."""
        _check(self.lib.psattn_plan_debug_waits(self.handle, int(wait_limit_ns), int(extra_expected_bytes)), self.handle)

    def psattn_plan_enable_host_io(self):
        _check(self.lib.psattn_plan_enable_host_io(self.handle), self.handle)

    def psattn_forward_host(self, Q, K, V, lengths, sample_idx, O, sel_idx):
        """All arguments are HOST tensors (pinned for speed); O and sel_idx are filled in place."""
        _check(self.lib.psattn_forward_host(self.handle, _ptr(Q), _ptr(K), _ptr(V), _ptr(lengths),
                                            _ptr(sample_idx), _ptr(O), _ptr(sel_idx), _stream()),
               self.handle)
        return O, sel_idx
