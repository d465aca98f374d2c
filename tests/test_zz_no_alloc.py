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


def test_second_call_allocates_nothing_and_lengths_are_clamped():
    """What the entry point is for: once the first call on the device has looked up its scratch array, a call
    leaves the amount of free device memory exactly as it found it.  Lengths outside [0, T_max] are clamped."""
    B, H, T = 3, 2, 700
    V, _, tdt = _case(B, H, T, 3, "bf16", [700, 700, 700])
    L_bad = torch.tensor([700 + 50, -4, 123], dtype=torch.int32, device="cuda")     # too long, negative, fine
    got = torch.empty((B, H, 64), dtype=torch.float32, device="cuda")
    ps.psattn_mean_v_noalloc(V, L_bad, got, B, H, T)            # a first call may do the one-time set-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    ps.psattn_mean_v_noalloc(V, L_bad, got, B, H, T)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the call changed the free device memory"
    v = V.float().cpu().numpy()
    want = np.stack([v[0].mean(axis=1), np.zeros((H, 64), dtype=np.float32), v[2, :, :123].mean(axis=1)])
    assert np.abs(got.cpu().numpy() - want).max() <= 1e-4


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
    # sizes beyond the plan limits are refused before any arithmetic on them
    assert lib.psattn_mean_v_noalloc(V.data_ptr(), None, out.data_ptr(), 1, 1, 2 ** 31 - 1, 0, None) == 2
    assert lib.psattn_mean_v_noalloc(V.data_ptr(), None, out.data_ptr(), 2 ** 21, 1, 256, 0, None) == 2
