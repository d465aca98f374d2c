"""CPU-side checks of the C ABI: the library loads, exports what the header declares, and its
host-only entry points behave.  No kernel is launched here."""
import ctypes
import math
import os
import re

import pytest

from paper_2106_09236_b200 import binding as ps

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "psattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(psattn_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ps.load()
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(ps.EXPORTS) == names


def test_version_and_status_strings():
    lib = ps.load()
    assert lib.psattn_version() >= 1000
    seen = set()
    for code in range(0, 8):
        s = lib.psattn_status_string(code).decode()
        assert s and s not in seen
        seen.add(s)
    assert "unknown" in lib.psattn_status_string(99).decode()


def test_count_rule_closed_form():
    """n(c, len) = clamp(ceil(c ln len), 1, len) (Sec. 3.2), natural log, host double."""
    for L in list(range(1, 600)) + [1024, 8192, 65536]:
        for c in (0.5, 1.0, 5.0, 25.0):
            assert ps.psattn_count(c, L) == min(L, max(1, math.ceil(c * math.log(L))))
    assert ps.psattn_count(5.0, 0) == 0 and ps.psattn_count(5.0, -4) == 0
    assert [ps.psattn_count(5.0, T) for T in (128, 512, 1024, 8192)] == [25, 32, 35, 46]


def test_plan_create_rejects_bad_descriptors_before_touching_a_device():
    lib = ps.load()
    h = ctypes.c_void_p()

    def make(**kw):
        d = ps.psattn_desc_t()
        d.B, d.H, d.T_max, d.d_head, d.idx_cols, d.c = 1, 1, 64, 64, 32, 5.0
        for k, v in kw.items():
            setattr(d, k, v)
        return d

    assert lib.psattn_plan_create(None, ctypes.byref(h)) == 1
    for bad in (dict(H=0), dict(T_max=0), dict(dtype=5), dict(fill_mode=9), dict(c=0.0),
                dict(c=float("nan")), dict(idx_cols=0), dict(path=7), dict(u_override=-1),
                dict(r_sparse=-0.1), dict(r_sparse=1.5), dict(r_sparse=float("nan"))):
        assert lib.psattn_plan_create(ctypes.byref(make(**bad)), ctypes.byref(h)) == 2, bad
        assert h.value is None
    assert lib.psattn_plan_create(ctypes.byref(make(d_head=128)), ctypes.byref(h)) == 3
    d = make()
    d.q_stride[:] = [64 * 64, 64 * 64, 60]         # row stride below d_head
    assert lib.psattn_plan_create(ctypes.byref(d), ctypes.byref(h)) == 2
    d = make()
    d.q_stride[:] = [4100, 4100, 68]               # not multiples of 8 elements
    assert lib.psattn_plan_create(ctypes.byref(d), ctypes.byref(h)) == 2
    assert lib.psattn_plan_create(ctypes.byref(make(idx_cols=8)), ctypes.byref(h)) == 2


def test_without_a_gpu_the_library_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(ps.PsattnError, match="device"):
        ps.Plan(1, 1, 64)


def test_null_plan_arguments():
    lib = ps.load()
    assert lib.psattn_plan_destroy(None) == 1
    assert lib.psattn_workspace_bytes(None, None) == 1
    assert lib.psattn_forward(None, None, None, None, None, None, None, None, None, None, 0, None) == 1
    assert lib.psattn_read_status(None, None, None, None) == 1
    assert lib.psattn_last_cuda_error(None) == 0
