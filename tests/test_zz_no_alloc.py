"""The allocation-free mean(V) entry point against the planned one.

psattn_mean_v_noalloc serves callers that cannot allocate device memory at the point of use
(a framework that owns all device memory, a no-allocation-after-start-up pipeline).  Its
scratch is one fixed array inside the library that every call reuses, so the test makes two
calls in a row with different shapes and contents - the second must not see anything the first
left behind - and compares each with psattn_mean_v on the same input.  This file sorts last so
that a failure here cannot hide the results of the other tests.
"""
import numpy as np
import pytest
import torch

from paper_2106_09236_b200 import binding as ps
from paper_2106_09236_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _case(B, H, T, seed, dtype, lengths):
    w = wl.Workload("noalloc", 0, B, H, T, 64, dtype, 5.0, 0.1, 3.0)
    inp = wl.make_inputs(w, 4, seed=seed, lengths=lengths)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    V = torch.from_numpy(inp["V"]).to("cuda", tdt)
    L = torch.from_numpy(inp["lengths"]).cuda()
    return V, L, tdt


def test_two_calls_in_a_row_match_the_planned_entry_point():
    cases = [
        (4, 8, 1500, 1, "bf16", [1500, 1, 777, 256]),     # first call: larger, leaves partials behind
        (2, 3, 300, 2, "fp32", [299, 40]),                # second call: smaller, other element type
    ]
    for B, H, T, seed, dtype, lengths in cases:
        V, L, tdt = _case(B, H, T, seed, dtype, lengths)
        plan = ps.Plan(B, H, T, dtype=tdt, c=5.0)
        want = plan.psattn_mean_v(V, L)
        got = torch.full((B, H, 64), float("nan"), dtype=torch.float32, device="cuda")
        ps.psattn_mean_v_noalloc(V, L, got, B, H, T)
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        assert (got - want).abs().max().item() <= 1e-5     # tolerance of the mean(V) parity test
        ref = np.stack([[inp.mean(0) for inp in seq] for seq in
                        [[V[b, h, :lengths[b]].float().cpu().numpy() for h in range(H)] for b in range(B)]])
        assert np.abs(got.cpu().numpy() - ref).max() <= 1e-4
        plan.close()


def test_capacity_and_argument_errors():
    V = torch.zeros((1, 1, 256, 64), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 1, 64), dtype=torch.float32, device="cuda")
    lib = ps.load()
    # 16385 partial blocks needed > 16384 available: rejected, nothing launched
    before = ps.psattn_launch_count()
    rc = lib.psattn_mean_v_noalloc(V.data_ptr(), None, out.data_ptr(), 16385, 1, 256, 0, None)
    assert rc == 8 and "capacity" in lib.psattn_status_string(rc).decode()
    assert ps.psattn_launch_count() == before
    assert lib.psattn_mean_v_noalloc(None, None, out.data_ptr(), 1, 1, 256, 0, None) == 1
    assert lib.psattn_mean_v_noalloc(V.data_ptr(), None, out.data_ptr(), 1, 1, 256, 7, None) == 2
