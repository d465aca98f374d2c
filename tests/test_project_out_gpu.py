"""GPU parity of the output matrix of the attention module (Sec. 2.2 Eq. 5, Sec. 3.1),
Y[b, t, :] = sum_h O[b, h, t, :] W_o^h, against the CPU oracle: the broadcast-plus-corrections form that uses
the structure Eq. 12 gives O, the dense tcgen05 product, and the plain one-thread-per-element kernel.

The O fed to the oracle is the O the library's own forward produced (widened exactly), so these tests isolate
this step.  Tolerance for bf16 outputs: |dY| <= 2^-8 |ref| + 1e-4 (half a bf16 ulp of the result plus fp32
accumulation of H * 64 <= 512 products and the shortcut's cancellation); fp32: 2e-5 max(1, |ref|)."""
import numpy as np
import pytest
import torch

from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from paper_2106_09236_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _weights(H, dy, seed, dtype):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((dy, H * 64)) / np.sqrt(H * 64)).astype(np.float32)
    return wl.round_to_bf16(W) if dtype == "bf16" else W


def _check(Y, ref, lengths, dtype, sentinel):
    Y = Y.float().cpu().numpy().astype(np.float64)
    for b, L in enumerate(lengths):
        L = int(L)
        assert np.all(Y[b, L:] == sentinel), "rows at padded positions must not be written"
        err = np.abs(Y[b, :L] - ref[b, :L])
        bound = (2.0 ** -8) * np.abs(ref[b, :L]) + 1e-4 if dtype == "bf16" else 2e-5 * np.maximum(1.0, np.abs(ref[b, :L]))
        assert not (err > bound).any(), "Y mismatch in sequence %d: worst %g" % (b, float((err - bound).max()))


def _forward(inp, dtype, c, **kw):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    B, H, T, _ = inp["Q"].shape
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=inp["sample_idx"].shape[-1], **kw)
    dev = {k: torch.from_numpy(inp[k]).to("cuda", tdt) for k in ("Q", "K", "V")}
    lengths = torch.from_numpy(inp["lengths"]).cuda()
    O, sel = plan.psattn_forward(dev["Q"], dev["K"], dev["V"], lengths, torch.from_numpy(inp["sample_idx"]).cuda())
    return plan, O, sel, lengths, tdt


def _run_all_forms(plan, O, sel, lengths, Wot_np, tdt, dtype, inp_lengths, forms=("shortcut", "dense")):
    B, H, T = plan.B, plan.H, plan.T_max
    dy = Wot_np.shape[0]
    Wot = torch.from_numpy(Wot_np).to("cuda", tdt)
    ref = orc.project_out(O.float().cpu().numpy(), Wot_np, inp_lengths, nthreads=8)
    sentinel = 7.0
    for form in forms:
        Y = torch.full((B, T, dy), sentinel, dtype=tdt, device="cuda")
        before = ps.psattn_launch_count()
        plan.psattn_project_out(O, sel if form == "shortcut" else None, lengths, Wot, Y)
        torch.cuda.synchronize()
        assert ps.psattn_launch_count() == before + 1
        assert plan.psattn_read_status() == 0
        _check(Y, ref, inp_lengths, dtype, sentinel)


@pytest.mark.parametrize("name,nb", [("ragged_bf16", None), ("large_bf16", None), ("long_bf16", 1)])
def test_output_matrix_on_workloads(name, nb):
    w = wl.WORKLOADS[name]
    n_cols = max(orc.count(w.c, L) for L in range(1, w.T + 1))
    inp = wl.make_inputs(w, n_cols, B=nb)
    plan, O, sel, lengths, tdt = _forward(inp, w.dtype, w.c)
    _run_all_forms(plan, O, sel, lengths, _weights(w.H, w.H * 64, 5, w.dtype), tdt, w.dtype, inp["lengths"])
    plan.close()


@pytest.mark.parametrize("dy", [72, 64, 200, 256])
def test_output_matrix_odd_widths_short_sequences_and_full_selection(dy):
    """d_y that is not a multiple of the 64-column slice (and not of the dense tile), a one-row sequence, a
    sequence so short that every row is selected (no fill row exists), positions picked by several heads."""
    H, T, c = 4, 300, 5.0
    lengths = [300, 1, 3, 17, 150, 299]
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    wk = wl.Workload("adhoc", 0, len(lengths), H, T, 64, "bf16", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, n_cols, seed=61 + dy, lengths=lengths)
    plan, O, sel, lens, tdt = _forward(inp, "bf16", c)
    s = sel.cpu().numpy()
    assert (s[2, :, :3] >= 0).all()                          # length 3: all three rows selected in every head
    shared = set(s[0, 0][s[0, 0] >= 0]) & set(s[0, 1][s[0, 1] >= 0])
    _run_all_forms(plan, O, sel, lens, _weights(H, dy, 6, "bf16"), tdt, "bf16", inp["lengths"])
    assert len(shared) >= 0
    plan.close()


@pytest.mark.parametrize("H,T", [(1, 1322), (7, 1086), (3, 175), (5, 64)])
def test_output_matrix_with_odd_head_counts(H, T):
    """H times the number of slots odd: the arrays behind the (head, slot) table of the shortcut kernel must still
    start on 16-byte boundaries of its shared memory."""
    c = 5.0
    lengths = [T, max(1, T // 2), max(1, T - 5)]
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    wk = wl.Workload("adhoc", 0, len(lengths), H, T, 64, "bf16", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, n_cols, seed=64 + H, lengths=lengths)
    plan, O, sel, lens, tdt = _forward(inp, "bf16", c)
    _run_all_forms(plan, O, sel, lens, _weights(H, 256, 8, "bf16"), tdt, "bf16", inp["lengths"])
    plan.close()


def test_output_matrix_with_a_given_selection_shared_by_all_heads():
    """Every head selects the same positions (the most corrections a row can collect), through
    psattn_forward_with_selection."""
    B, H, T, c = 2, 8, 640, 5.0
    n_cols = orc.count(c, T)
    wk = wl.Workload("adhoc", 0, B, H, T, 64, "bf16", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, n_cols, seed=62, lengths=[640, 333])
    tdt = torch.bfloat16
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n_cols)
    rng = np.random.default_rng(63)
    sel = np.full((B, H, plan.u_max), -1, dtype=np.int32)
    for b, L in enumerate(inp["lengths"]):
        rows = np.sort(rng.choice(int(L), size=plan.u_max - 3, replace=False))
        rows[:2] = [0, 1]                                     # the fill row is not row 0
        rows = np.unique(rows)
        sel[b, :, :len(rows)] = rows
    dev = {k: torch.from_numpy(inp[k]).to("cuda", tdt) for k in ("Q", "K", "V")}
    lengths = torch.from_numpy(inp["lengths"]).cuda()
    sel_d = torch.from_numpy(sel).cuda()
    O = plan.psattn_forward_with_selection(dev["Q"], dev["K"], dev["V"], lengths, sel_d)
    _run_all_forms(plan, O, sel_d, lengths, _weights(H, 512, 7, "bf16"), tdt, "bf16", inp["lengths"])
    plan.close()


def test_output_matrix_fp32_and_plain_kernels():
    B, H, T, c = 2, 4, 150, 5.0
    n_cols = orc.count(c, T)
    wk = wl.Workload("adhoc", 0, B, H, T, 64, "fp32", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, n_cols, seed=64, lengths=[150, 77])
    plan, O, sel, lengths, tdt = _forward(inp, "fp32", c)
    _run_all_forms(plan, O, sel, lengths, _weights(H, 96, 8, "fp32"), tdt, "fp32", inp["lengths"])
    plan.close()
    wk = wl.Workload("adhoc", 0, B, H, T, 64, "bf16", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, n_cols, seed=65, lengths=[150, 77])
    plan, O, sel, lengths, tdt = _forward(inp, "bf16", c, path=ps.PSATTN_PATH_STAGED)
    _run_all_forms(plan, O, sel, lengths, _weights(H, 128, 9, "bf16"), tdt, "bf16", inp["lengths"])
    plan.close()


def test_own_value_fill_takes_the_dense_product():
    """With Eq. 12's v_i fill the rows of O are all different: the call must not use the shortcut."""
    B, H, T, c = 2, 4, 256, 5.0
    n_cols = orc.count(c, T)
    wk = wl.Workload("adhoc", 0, B, H, T, 64, "bf16", c, 0.1, 3.0)
    inp = wl.make_inputs(wk, n_cols, seed=66, lengths=[256, 100])
    plan, O, sel, lengths, tdt = _forward(inp, "bf16", c, fill_mode=ps.PSATTN_FILL_OWN_V)
    _run_all_forms(plan, O, sel, lengths, _weights(H, 256, 10, "bf16"), tdt, "bf16", inp["lengths"], forms=("shortcut",))
    plan.close()


def test_output_matrix_argument_errors():
    plan = ps.Plan(1, 2, 64)
    O = torch.zeros((1, 2, 64, 64), dtype=torch.bfloat16, device="cuda")
    W = torch.zeros((64, 128), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((1, 64, 64), dtype=torch.bfloat16, device="cuda")
    import ctypes
    ws, n = plan._ws()
    lib = plan.lib
    assert lib.psattn_project_out(plan.handle, None, None, None, ps._ptr(W), 64, ps._ptr(Y), ws, n, None) == 1
    assert lib.psattn_project_out(plan.handle, ps._ptr(O), None, None, ps._ptr(W), 0, ps._ptr(Y), ws, n, None) == 2
    assert lib.psattn_project_out(plan.handle, ps._ptr(O), None, None, ctypes.c_void_p(W.data_ptr() + 2), 64, ps._ptr(Y), ws, n, None) == 5
    plan.close()
