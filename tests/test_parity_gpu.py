"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element.

Every test here needs a B200; inputs are seeded and synthetic (paper_2106_09236_b200.workloads).
"""
import numpy as np
import pytest
import torch

import parity
from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from paper_2106_09236_b200 import workloads as wl

pytestmark = pytest.mark.gpu

PATHS = [ps.PSATTN_PATH_STAGED, ps.PSATTN_PATH_AUTO]
PATH_IDS = ["staged", "auto"]


def _dev(inp, dtype):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    out = {k: torch.from_numpy(inp[k]).to("cuda", tdt) for k in ("Q", "K", "V")}
    out["lengths"] = torch.from_numpy(inp["lengths"]).cuda()
    out["sample_idx"] = torch.from_numpy(inp["sample_idx"]).cuda()
    return out, tdt


def _synth(B, H, T, seed, n_cols, dtype="bf16", lengths=None, scale_peaky=3.0):
    w = wl.Workload("adhoc", 0, B, H, T, 64, dtype, 5.0, 0.1, scale_peaky)
    return wl.make_inputs(w, n_cols, seed=seed, lengths=lengths)


def _run_forward(inp, dtype, c, path, want_M=True, **plan_kw):
    dev, tdt = _dev(inp, dtype)
    B, H, T, d = inp["Q"].shape
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=inp["sample_idx"].shape[-1], path=path, **plan_kw)
    M = torch.full((B, H, T), float("nan"), dtype=torch.float32, device="cuda") if want_M else None
    O = torch.full((B, H, T, d), float("nan"), dtype=tdt, device="cuda")
    sel = torch.full((B, H, plan.u_max), -7, dtype=torch.int32, device="cuda")
    plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"], O, sel, M)
    torch.cuda.synchronize()
    status = plan.psattn_read_status()
    res = (O.float().cpu().numpy(), sel.cpu().numpy(), None if M is None else M.cpu().numpy(), status)
    plan.close()
    return res


# ---- the five workloads, full size ---------------------------------------------------------

@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("name", ["tiny_fp32", "base_bf16", "ragged_bf16", "large_bf16", "long_bf16"])
def test_forward_matches_oracle_on_workload(name, path):
    w = wl.WORKLOADS[name]
    n_cols = max(orc.count(w.c, L) for L in range(1, w.T + 1))
    inp = wl.make_inputs(w, n_cols)
    O, sel, M, status = _run_forward(inp, w.dtype, w.c, path)
    assert status == 0
    info = parity.check_forward(O, sel, M, inp, inp["lengths"], w.dtype, w.c)
    assert info["swapped_units"] <= max(1, (w.B * w.H) // 8)


# ---- ragged sizes, several tiles and tails ------------------------------------------------

@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("T", [1, 2, 3, 17, 127, 129, 300, 1100, 2500])
def test_forward_small_and_ragged(T, dtype, path):
    B, H, c = 3, 2, 5.0
    lengths = [T, max(1, T // 2), max(1, T - 1)]
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    inp = _synth(B, H, T, 500 + T, n_cols, dtype, lengths)
    O, sel, M, status = _run_forward(inp, dtype, c, path)
    assert status == 0
    parity.check_forward(O, sel, M, inp, inp["lengths"], dtype, c)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_padding_contents_are_never_read(path):
    B, H, T, c = 2, 2, 200, 5.0
    lengths = [77, 200]
    n_cols = orc.count(c, T)
    inp = _synth(B, H, T, 42, n_cols, "bf16", lengths)
    ref = _run_forward(inp, "bf16", c, path)
    poisoned = {k: v.copy() for k, v in inp.items()}
    for k in ("Q", "K", "V"):
        poisoned[k][0, :, 77:] = np.nan
    poisoned["sample_idx"][0, 77:] = 10 ** 6        # rows of padded queries are never read either
    got = _run_forward(poisoned, "bf16", c, path)
    assert got[3] == 0
    np.testing.assert_array_equal(got[0], ref[0])
    np.testing.assert_array_equal(got[1], ref[1])
    np.testing.assert_array_equal(got[2], ref[2])


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_all_selected_equals_dense_attention(path):
    """u = len: every row goes through step (d); the result is Eq. 6."""
    B, H, T, c = 2, 2, 96, 5.0
    lengths = [96, 51]
    inp = _synth(B, H, T, 43, orc.count(c, T), "fp32", lengths)
    O, sel, M, status = _run_forward(inp, "fp32", c, path, u_override=T)
    dense = orc.dense(inp["Q"], inp["K"], inp["V"], inp["lengths"])
    assert np.abs(O - dense).max() <= parity.O_ATOL["fp32"]
    for b in range(B):
        assert [int(x) for x in sel[b, 0] if x >= 0] == list(range(lengths[b]))


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_zero_queries_tie_rule_and_exact_zero_measure(path):
    B, H, T, c = 1, 2, 150, 5.0
    inp = _synth(B, H, T, 44, orc.count(c, T), "bf16")
    inp["Q"][:] = 0.0
    O, sel, M, status = _run_forward(inp, "bf16", c, path)
    assert np.all(M == 0.0)
    u = orc.count(c, T)
    for h in range(H):
        assert [int(x) for x in sel[0, h] if x >= 0] == list(range(u))
    vbar = orc.mean_v(inp["V"])
    assert np.abs(O - vbar[:, :, None, :]).max() <= parity.O_ATOL["bf16"]


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_duplicate_samples_and_constant_rows(path):
    B, H, T, c = 1, 2, 64, 5.0
    n = orc.count(c, T)
    inp = _synth(B, H, T, 45, n, "fp32")
    inp["sample_idx"][0, :, 1] = inp["sample_idx"][0, :, 0]
    inp["sample_idx"][0, 5, :] = 9
    O, sel, M, status = _run_forward(inp, "fp32", c, path)
    assert np.all(M >= 0.0)
    assert M[0, 0, 5] == 0.0 and M[0, 1, 5] == 0.0
    parity.check_forward(O, sel, M, inp, inp["lengths"], "fp32", c)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_own_value_fill_and_sample_override(path):
    """Eq. 12 as printed (v_i for the rest) with the paper's r_sparse = 0.5 and a small sample."""
    B, H, T, c = 2, 2, 120, 5.0
    lengths = [120, 64]
    inp = _synth(B, H, T, 46, 8, "bf16", lengths)
    O, sel, M, status = _run_forward(inp, "bf16", c, path, u_override=60, U_override=8,
                                     fill_mode=ps.PSATTN_FILL_OWN_V)
    parity.check_forward(O, sel, M, inp, inp["lengths"], "bf16", c, u_override=60, U_override=8,
                         fill="own_v")


@pytest.mark.parametrize("r_sparse", [0.35, 0.5])
@pytest.mark.parametrize("dtype,T", [("bf16", 1024), ("fp32", 300)])
def test_paper_literal_variant_at_scale(dtype, T, r_sparse):
    """Sec. 3.2's own rule u = ceil(r_sparse * T) (hundreds of selected rows per unit: several
    128-row tiles of the tensor-core attention and a ragged last one) with Eq. 12's v_i fill."""
    B, H, c = 2, 4, 5.0
    lengths = [T, T - 37]
    u = int(np.ceil(r_sparse * T))
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    inp = _synth(B, H, T, 146 + T, n_cols, dtype, lengths)
    O, sel, M, status = _run_forward(inp, dtype, c, ps.PSATTN_PATH_AUTO, u_override=u,
                                     fill_mode=ps.PSATTN_FILL_OWN_V)
    assert status == 0
    assert sel.shape[-1] == u
    parity.check_forward(O, sel, M, inp, inp["lengths"], dtype, c, u_override=u, fill="own_v")


@pytest.mark.parametrize("r_sparse", [0.35, 0.5])
@pytest.mark.parametrize("dtype,T", [("bf16", 500), ("bf16", 1400), ("fp32", 160)])
def test_paper_count_rule_per_sequence(dtype, T, r_sparse):
    """Sec. 3.2 as stated: L_sparse = r_sparse L from every sequence's OWN length (descriptor field
    r_sparse), ragged batch, Eq. 12's v_i fill; r_sample = 1 (c = 1) as in the paper's timed model."""
    H, c = 4, 1.0
    rng = np.random.default_rng(900 + T)
    lengths = [T, 1, 40] + [int(x) for x in rng.integers(40, T + 1, size=5)]
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    inp = _synth(len(lengths), H, T, 147 + T, n_cols, dtype, lengths)
    O, sel, M, status = _run_forward(inp, dtype, c, ps.PSATTN_PATH_AUTO, r_sparse=r_sparse,
                                     fill_mode=ps.PSATTN_FILL_OWN_V)
    assert status == 0
    assert sel.shape[-1] == int(np.ceil(r_sparse * T))
    for b, L in enumerate(lengths):
        assert int((sel[b, 0] >= 0).sum()) == max(1, int(np.ceil(r_sparse * L)))
    parity.check_forward(O, sel, M, inp, inp["lengths"], dtype, c, fill="own_v", r_sparse=r_sparse)


@pytest.mark.parametrize("T", [80, 1300])           # keys resident in shared memory / streamed from L2
@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_out_of_range_inputs_set_status_bits_without_faulting(path, T):
    B, H, c = 2, 1, 5.0
    n = orc.count(c, T)
    inp = _synth(B, H, T, 47, n, "bf16")
    bad = {k: v.copy() for k, v in inp.items()}
    bad["sample_idx"][0, 3, 2] = T + 1000
    bad["sample_idx"][1, 7, 0] = -5
    O, sel, M, status = _run_forward(bad, "bf16", c, path)
    assert status & 1
    fixed = {k: v.copy() for k, v in inp.items()}
    fixed["sample_idx"][0, 3, 2] = T - 1             # clamped to the last valid key
    fixed["sample_idx"][1, 7, 0] = 0                 # clamped to the first key
    O2, sel2, M2, status2 = _run_forward(fixed, "bf16", c, path)
    assert status2 == 0
    np.testing.assert_array_equal(M, M2)
    np.testing.assert_array_equal(O, O2)
    too_long = {k: v.copy() for k, v in inp.items()}
    too_long["lengths"] = np.array([T + 5, -3], dtype=np.int32)
    O3, sel3, M3, status3 = _run_forward(too_long, "bf16", c, path)
    assert status3 & 2
    assert np.all(O3[1] == 0.0) and np.all(sel3[1] == -1)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_run_to_run_determinism(path):
    w = wl.WORKLOADS["base_bf16"]
    n = orc.count(w.c, w.T)
    inp = wl.make_inputs(w, n, B=4)
    a = _run_forward(inp, "bf16", w.c, path)
    b = _run_forward(inp, "bf16", w.c, path)
    for x, y in zip(a[:3], b[:3]):
        np.testing.assert_array_equal(x, y)


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("dtype,T", [("bf16", 300), ("bf16", 1500), ("fp32", 200)])
def test_workspace_contents_do_not_matter_and_its_bounds_are_kept(dtype, T, path):
    """The scratch beyond the status word needs no initialisation: a run on a workspace full of 0xFF bytes
    (NaN as floats, -1 as indices) gives bit-identical results, and the bytes on either side of the
    workspace are not touched."""
    B, H, c = 3, 2, 5.0
    n = max(orc.count(c, L) for L in range(1, T + 1))
    inp = _synth(B, H, T, 900 + T, n, dtype, [T, T // 3, T - 1])
    ref = _run_forward(inp, dtype, c, path)
    dev, tdt = _dev(inp, dtype)
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n, path=path)
    guard = 4096
    big = torch.full((plan.workspace_bytes + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    ws = big[guard:guard + plan.workspace_bytes]
    assert ws.data_ptr() % 256 == 0
    ws.fill_(0xFF)
    ws[:256] = 0                                          # the status block is the one part that must be zero
    plan.workspace = ws
    M = torch.full((B, H, T), float("nan"), dtype=torch.float32, device="cuda")
    O = torch.full((B, H, T, 64), float("nan"), dtype=tdt, device="cuda")
    sel = torch.full((B, H, plan.u_max), -7, dtype=torch.int32, device="cuda")
    for _ in range(2):                                    # the second call sees the first call's leftovers
        plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"], O, sel, M)
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    np.testing.assert_array_equal(O.float().cpu().numpy(), ref[0])
    np.testing.assert_array_equal(sel.cpu().numpy(), ref[1])
    np.testing.assert_array_equal(M.cpu().numpy(), ref[2])
    assert bool((big[:guard] == 0xA5).all()) and bool((big[guard + plan.workspace_bytes:] == 0xA5).all())
    plan.close()


@pytest.mark.parametrize("dtype,T", [("bf16", 300), ("bf16", 1500), ("fp32", 200)])
def test_forward_inside_a_cuda_graph_matches_the_direct_call(dtype, T):
    """The call may fork work onto the plan's side stream and uses programmatic dependent launches: a stream
    capture has to follow all of it, and a replay on new input values has to give what a direct call gives."""
    B, H, c = 3, 2, 5.0
    n = max(orc.count(c, L) for L in range(1, T + 1))
    lengths = [T, T // 2, T - 3]
    first = _synth(B, H, T, 700 + T, n, dtype, lengths)
    second = _synth(B, H, T, 800 + T, n, dtype, lengths)
    want = _run_forward(second, dtype, c, ps.PSATTN_PATH_AUTO)
    dev, tdt = _dev(first, dtype)
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n)
    M = torch.empty((B, H, T), dtype=torch.float32, device="cuda")
    O = torch.empty((B, H, T, 64), dtype=tdt, device="cuda")
    sel = torch.empty((B, H, plan.u_max), dtype=torch.int32, device="cuda")

    def call():
        plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"], O, sel, M)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()                                             # warm-up outside the capture (one-time attribute calls)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    dev2, _ = _dev(second, dtype)
    for key in ("Q", "K", "V", "sample_idx"):
        dev[key].copy_(dev2[key])
    O.fill_(float("nan")); sel.fill_(-7); M.fill_(float("nan"))
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    np.testing.assert_array_equal(O.float().cpu().numpy(), want[0])
    np.testing.assert_array_equal(sel.cpu().numpy(), want[1])
    np.testing.assert_array_equal(M.cpu().numpy(), want[2])
    plan.close()


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_strided_bthd_layout(path):
    """Q, K, V, O stored [B][T][H][d] (projection output order) through the stride fields."""
    B, H, T, c, d = 2, 4, 160, 5.0, 64
    n = orc.count(c, T)
    inp = _synth(B, H, T, 48, n, "bf16", [160, 90])
    dev, tdt = _dev(inp, "bf16")
    st = (T * H * d, d, H * d)
    perm = {k: dev[k].permute(0, 2, 1, 3).contiguous() for k in ("Q", "K", "V")}   # [B,T,H,d]
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n, path=path,
                   strides={"q": st, "k": st, "v": st, "o": st})
    O = torch.full((B, T, H, d), float("nan"), dtype=tdt, device="cuda")
    sel = torch.empty((B, H, plan.u_max), dtype=torch.int32, device="cuda")
    M = torch.empty((B, H, T), dtype=torch.float32, device="cuda")
    plan.psattn_forward(perm["Q"], perm["K"], perm["V"], dev["lengths"], dev["sample_idx"], O, sel, M)
    torch.cuda.synchronize()
    parity.check_forward(O.permute(0, 2, 1, 3).float().cpu().numpy(), sel.cpu().numpy(),
                         M.cpu().numpy(), inp, inp["lengths"], "bf16", c)
    plan.close()


# ---- per-step entry points -----------------------------------------------------------------------

def test_measure_entry_point():
    w = wl.WORKLOADS["base_bf16"]
    n = orc.count(w.c, w.T)
    inp = wl.make_inputs(w, n, B=3)
    dev, tdt = _dev(inp, "bf16")
    plan = ps.Plan(3, w.H, w.T, dtype=tdt, c=w.c, idx_cols=n)
    M = plan.psattn_measure(dev["Q"], dev["K"], dev["lengths"], dev["sample_idx"])
    torch.cuda.synchronize()
    parity.check_measure(M.cpu().numpy(), orc.measure(inp["Q"], inp["K"], inp["sample_idx"],
                                                      inp["lengths"], c=w.c), inp["lengths"])
    plan.close()


@pytest.mark.parametrize("U_override", [0, 9, 46])
@pytest.mark.parametrize("T", [1024, 3000])        # keys resident in shared memory / gathered from L2
def test_measure_with_structured_samples(T, U_override):
    """Sample rows that are not uniform: every sample in the first 1024 keys, every sample in the last 100
    keys, one key repeated, a row of equal-score keys (exact zero), ascending runs, an odd and an even sample
    count, a sequence shorter than T_max whose length is no multiple of any tile; then out-of-range entries,
    which must be clamped and reported, never followed."""
    B, H, c = 3, 2, 5.0
    lengths = [T, T - 37, 129]
    n_cols = max(orc.count(c, T), U_override)
    inp = _synth(B, H, T, 700 + T, n_cols, "bf16", lengths)
    idx = inp["sample_idx"]
    rng = np.random.default_rng(701)
    for b, L in enumerate(lengths):
        idx[b, 0:L:7] = rng.integers(0, min(L, 1024), size=idx[b, 0:L:7].shape)        # all in the first chunk
        idx[b, 1:L:7] = rng.integers(max(0, L - 100), L, size=idx[b, 1:L:7].shape)      # all at the end
        idx[b, 2:L:7] = rng.integers(0, L, size=(len(range(2, L, 7)), 1))               # one key, repeated
        idx[b, 3:L:7] = np.sort(idx[b, 3:L:7], axis=-1)                                 # ascending
    inp["K"][0, :, 5:9] = inp["K"][0, :, 5:6]                                           # four identical key rows
    idx[0, 11] = np.resize(np.array([5, 6, 7, 8], dtype=np.int32), n_cols)              # -> constant scores
    dev, tdt = _dev(inp, "bf16")
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n_cols, U_override=U_override)
    M = plan.psattn_measure(dev["Q"], dev["K"], dev["lengths"], dev["sample_idx"])
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    Mh = M.cpu().numpy()
    parity.check_measure(Mh, orc.measure(inp["Q"], inp["K"], idx, inp["lengths"], c=c, U_override=U_override),
                         inp["lengths"])
    assert np.all(Mh[0, :, 11] == 0.0) and np.all(Mh[:, :, 2][:, :] == 0.0)           # constant scores: exactly zero
    assert Mh.min() >= 0.0
    # out-of-range entries: clamped into [0, len), status bit 0, no fault
    bad = idx.copy()
    bad[1, 40, 0] = T + 12345
    bad[2, 3, 1] = -7
    M2 = plan.psattn_measure(dev["Q"], dev["K"], dev["lengths"], torch.from_numpy(bad).cuda())
    torch.cuda.synchronize()
    assert plan.psattn_read_status() & 1
    clamped = bad.copy()
    clamped[1, 40, 0] = lengths[1] - 1
    clamped[2, 3, 1] = 0
    parity.check_measure(M2.cpu().numpy(), orc.measure(inp["Q"], inp["K"], clamped, inp["lengths"], c=c,
                                                       U_override=U_override), inp["lengths"])
    plan.close()


def test_measure_per_head_samples():
    B, H, T, c = 2, 3, 70, 5.0
    n = orc.count(c, T)
    inp = _synth(B, H, T, 49, n, "fp32")
    rng = np.random.default_rng(2)
    idx = rng.integers(0, T, size=(B, H, T, n)).astype(np.int32)
    plan = ps.Plan(B, H, T, dtype=torch.float32, c=c, idx_cols=n, idx_per_head=True)
    M = plan.psattn_measure(torch.from_numpy(inp["Q"]).cuda(), torch.from_numpy(inp["K"]).cuda(),
                            None, torch.from_numpy(idx).cuda())
    torch.cuda.synchronize()
    parity.check_measure(M.cpu().numpy(), orc.measure(inp["Q"], inp["K"], idx, None, c=c))
    plan.close()


# ---- one sample per sequence (the other reading of Sec. 3.2's sampled key matrix) -----------

def _shared_sample(inp):
    """The compact [B][U] sample (query 0's draw of each sequence) and the per-query array the
    oracle reads, every query row holding that same sample."""
    B, H, T, _ = inp["Q"].shape
    compact = np.ascontiguousarray(inp["sample_idx"][:, 0, :])
    expanded = np.ascontiguousarray(np.broadcast_to(compact[:, None, :], (B, T, compact.shape[-1])))
    return compact, expanded


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("dtype,T", [("bf16", 300), ("fp32", 300), ("bf16", 1500)])
def test_shared_sample_forward(dtype, T, path):
    B, H, c = 3, 2, 5.0
    lengths = [T, max(1, T // 3), T - 1]
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    inp = _synth(B, H, T, 700 + T, n_cols, dtype, lengths)
    compact, expanded = _shared_sample(inp)
    O, sel, M, status = _run_forward(dict(inp, sample_idx=compact), dtype, c, path, idx_shared=True)
    assert status == 0
    parity.check_forward(O, sel, M, dict(inp, sample_idx=expanded), inp["lengths"], dtype, c)


def test_shared_sample_measure_large_and_per_head():
    w = wl.WORKLOADS["large_bf16"]
    n = orc.count(w.c, w.T)
    inp = wl.make_inputs(w, n, B=2)
    B, H, T = 2, w.H, w.T
    rng = np.random.default_rng(77)
    compact = rng.integers(0, T, size=(B, H, n)).astype(np.int32)
    compact[0, 1, 3] = compact[0, 1, 2]                  # a key drawn twice counts twice
    expanded = np.ascontiguousarray(np.broadcast_to(compact[:, :, None, :], (B, H, T, n)))
    plan = ps.Plan(B, H, T, dtype=torch.bfloat16, c=w.c, idx_cols=n, idx_per_head=True, idx_shared=True)
    dev, _ = _dev(inp, "bf16")
    M = plan.psattn_measure(dev["Q"], dev["K"], None, torch.from_numpy(compact).cuda())
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    parity.check_measure(M.cpu().numpy(), orc.measure(inp["Q"], inp["K"], expanded, None, c=w.c))
    plan.close()


# ---- the exact measure of Eq. 10 (dense pass) ------------------------------------------------

@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
@pytest.mark.parametrize("dtype,T", [("bf16", 300), ("bf16", 1100), ("fp32", 150)])
def test_exact_measure_entry_point(dtype, T, path):
    """ln sum exp(s) - mean(s) over all valid keys against the oracle's fp64 evaluation of Eq. 10
    (tensor-core form for bf16 on the automatic path, one warp per query otherwise)."""
    B, H, c = 2, 3, 5.0
    lengths = [T, max(1, T - 129)]
    inp = _synth(B, H, T, 900 + T, orc.count(c, T), dtype, lengths)
    dev, tdt = _dev(inp, dtype)
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, path=path)
    M = plan.psattn_exact_measure(dev["Q"], dev["K"], dev["lengths"])
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    plan.close()
    ref = orc.exact_measure(inp["Q"], inp["K"], inp["lengths"])
    parity.check_measure(M.cpu().numpy(), ref, inp["lengths"])


def test_select_entry_point_is_exact_including_ties():
    B, H, T, c = 3, 2, 700, 5.0
    rng = np.random.default_rng(50)
    M = rng.standard_normal((B, H, T)).astype(np.float32)
    M[0, 0] = np.round(M[0, 0] * 2) / 2            # heavy ties
    M[1, 1] = 0.0                                   # all equal
    M[2, 0, ::3] = -M[2, 0, ::3] * 1e-30            # tiny values of both signs
    M[2, 1] = -np.abs(M[2, 1])                      # all negative
    lengths = np.array([700, 333, 41], dtype=np.int32)
    plan = ps.Plan(B, H, T, c=c)
    sel = plan.psattn_select(torch.from_numpy(M).cuda(), torch.from_numpy(lengths).cuda())
    torch.cuda.synchronize()
    ref = orc.select(M.astype(np.float64), lengths, c=c, u_max=plan.u_max)
    np.testing.assert_array_equal(sel.cpu().numpy(), ref)
    plan.close()


@pytest.mark.parametrize("T", [40, 700, 2500])
def test_select_treats_signed_zeros_as_one_value(T):
    """-0.0 and +0.0 are equal values: they tie, the lower position first, as in the oracle."""
    B, H, c = 2, 2, 5.0
    rng = np.random.default_rng(70 + T)
    M = np.where(rng.random((B, H, T)) < 0.5, 0.0, -0.0).astype(np.float32)
    M[0, 0, ::11] = rng.standard_normal(M[0, 0, ::11].shape).astype(np.float32)     # a few real values of both signs
    M[1, 1] = np.round(rng.standard_normal(T) * 2) / 2                              # steps of 0.5: zeros of both signs among them
    lengths = np.array([T, max(1, T - 13)], dtype=np.int32)
    plan = ps.Plan(B, H, T, c=c)
    sel = plan.psattn_select(torch.from_numpy(M).cuda(), torch.from_numpy(lengths).cuda())
    torch.cuda.synchronize()
    np.testing.assert_array_equal(sel.cpu().numpy(), orc.select(M.astype(np.float64), lengths, c=c, u_max=plan.u_max))
    plan.close()


@pytest.mark.parametrize("B,H,T", [(3, 2, 9000), (4, 8, 8192), (1, 1, 8200)])
def test_select_of_few_long_units_is_exact_including_ties(B, H, T):
    """Few units of long sequences are selected range by range and then among the ranges' candidates:
    the result must still be the oracle's, ties (equal values: lower position first) included."""
    c = 5.0
    rng = np.random.default_rng(60 + T)
    M = rng.standard_normal((B, H, T)).astype(np.float32)
    M[0, 0] = np.round(M[0, 0] * 2) / 2            # heavy ties, spread over every range
    M[-1, -1] = 0.0                                 # all equal: the first u positions win, all in the first range
    if B > 1:
        M[1, 0, :] = -np.abs(M[1, 0])               # all negative
        M[1, 0, T - 7:] = 3.0                       # the winners sit at the very end of the last range, tied
    lengths = rng.integers(1, T + 1, size=B).astype(np.int32)
    lengths[0] = T
    if B > 1:
        lengths[1] = T
    if B > 2:
        lengths[2] = 1500                           # shorter than two ranges: the other ranges are empty
    plan = ps.Plan(B, H, T, c=c)
    sel = plan.psattn_select(torch.from_numpy(M).cuda(), torch.from_numpy(lengths).cuda())
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    ref = orc.select(M.astype(np.float64), lengths, c=c, u_max=plan.u_max)
    np.testing.assert_array_equal(sel.cpu().numpy(), ref)
    plan.close()


def test_mean_v_entry_point():
    B, H, T = 3, 2, 900
    inp = _synth(B, H, T, 51, 4, "bf16", [900, 257, 1])
    dev, tdt = _dev(inp, "bf16")
    plan = ps.Plan(B, H, T, dtype=tdt, c=5.0)
    vbar = plan.psattn_mean_v(dev["V"], dev["lengths"])
    torch.cuda.synchronize()
    ref = orc.mean_v(inp["V"], inp["lengths"])
    assert np.abs(vbar.cpu().numpy() - ref).max() <= 1e-5
    plan.close()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_attend_rows_entry_point(dtype):
    B, H, T, c = 2, 2, 1500, 5.0
    lengths = [1500, 1029]
    inp = _synth(B, H, T, 52, 4, dtype, lengths)
    dev, tdt = _dev(inp, dtype)
    plan = ps.Plan(B, H, T, dtype=tdt, c=c)
    rng = np.random.default_rng(3)
    n_rows = min(9, plan.u_max)
    rows = np.stack([[rng.choice(lengths[b], size=n_rows, replace=False) for _ in range(H)]
                     for b in range(B)]).astype(np.int32)
    rows[1, 0, 2] = -1                               # skipped slot -> zero row
    rows[1, 1, 4] = 1400                             # beyond the valid length -> zero row
    out = plan.psattn_attend_rows(dev["Q"], dev["K"], dev["V"], dev["lengths"],
                                  torch.from_numpy(rows).cuda())
    torch.cuda.synchronize()
    out = out.cpu().numpy()
    tol = 1e-4 if dtype == "fp32" else 2e-3          # fp32 output rows: no bf16 output rounding
    for b in range(B):
        for h in range(H):
            for r in range(n_rows):
                i = int(rows[b, h, r])
                if i < 0 or i >= lengths[b]:
                    assert np.all(out[b, h, r] == 0.0)
                else:
                    ref = orc.attend_row(inp["Q"], inp["K"], inp["V"], b, h, i, lengths[b])
                    assert np.abs(out[b, h, r] - ref).max() <= tol
    plan.close()


@pytest.mark.parametrize("path", PATHS, ids=PATH_IDS)
def test_forward_with_given_selection(path):
    """Sec. 4.4: a selection computed once is reused; also covers arbitrary (random) index sets."""
    B, H, T, c = 2, 2, 260, 5.0
    lengths = [260, 130]
    n = orc.count(c, T)
    inp = _synth(B, H, T, 53, n, "bf16", lengths)
    dev, tdt = _dev(inp, "bf16")
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n, path=path)
    rng = np.random.default_rng(4)
    sel_in = np.full((B, H, plan.u_max), -1, dtype=np.int32)
    for b in range(B):
        for h in range(H):
            k = orc.count(c, lengths[b])
            sel_in[b, h, :k] = np.sort(rng.choice(lengths[b], size=k, replace=False))
    O = plan.psattn_forward_with_selection(dev["Q"], dev["K"], dev["V"], dev["lengths"],
                                           torch.from_numpy(sel_in).cuda())
    torch.cuda.synchronize()
    O_ref, _, _ = orc.forward(inp["Q"], inp["K"], inp["V"], inp["sample_idx"], inp["lengths"],
                              c=c, sel_in=sel_in)
    parity.check_outputs(O.float().cpu().numpy(), O_ref, {}, inp, inp["lengths"], "bf16")
    plan.close()


@pytest.mark.parametrize("fill", ["mean_v", "own_v"])
@pytest.mark.parametrize("T", [200, 1024])
def test_forward_with_given_selection_one_kernel_form(T, fill):
    """Enough units that steps (d)+(e) run as one kernel per unit; the list is unsorted, shorter than its
    width for short sequences, and holds entries outside the sequence (ignored) in some units."""
    B, H, c = 21, 4, 5.0
    rng = np.random.default_rng(77 + T)
    lengths = rng.integers(1, T + 1, size=B).astype(np.int32)
    lengths[0], lengths[1] = T, 1
    n = orc.count(c, T)
    inp = _synth(B, H, T, 61, n, "bf16", lengths)
    dev, tdt = _dev(inp, "bf16")
    plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n,
                   fill_mode=ps.PSATTN_FILL_OWN_V if fill == "own_v" else ps.PSATTN_FILL_MEAN_V)
    sel_in = np.full((B, H, plan.u_max), -1, dtype=np.int32)
    for b in range(B):
        for h in range(H):
            k = min(plan.u_max, int(lengths[b]), orc.count(c, int(lengths[b])) + 3)
            sel_in[b, h, :k] = rng.permutation(int(lengths[b]))[:k]           # unsorted
    given = sel_in.copy()
    given[2, 1, -1] = int(lengths[2]) + 5 if lengths[2] + 5 < 2 ** 30 else -1  # beyond the sequence: ignored
    given[3, 0, -1] = -9
    clean = given.copy()
    clean[2, 1, -1] = -1
    clean[3, 0, -1] = -1
    O = torch.full((B, H, T, 64), float("nan"), dtype=tdt, device="cuda")
    before = ps.psattn_launch_count()
    plan.psattn_forward_with_selection(dev["Q"], dev["K"], dev["V"], dev["lengths"], torch.from_numpy(given).cuda(), O)
    torch.cuda.synchronize()
    assert ps.psattn_launch_count() - before == 1
    assert plan.psattn_read_status() == 0
    O_ref, _, _ = orc.forward(inp["Q"], inp["K"], inp["V"], inp["sample_idx"], inp["lengths"], c=c, sel_in=clean,
                              fill=fill, nthreads=orc.max_threads())
    parity.check_outputs(O.float().cpu().numpy(), O_ref, {}, inp, inp["lengths"], "bf16")
    plan.close()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_dense_comparator(dtype):
    B, H, T = 2, 2, 300
    lengths = [300, 171]
    inp = _synth(B, H, T, 54, 4, dtype, lengths)
    dev, tdt = _dev(inp, dtype)
    plan = ps.Plan(B, H, T, dtype=tdt, c=5.0)
    O = plan.psattn_dense_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"])
    torch.cuda.synchronize()
    ref = orc.dense(inp["Q"], inp["K"], inp["V"], inp["lengths"])
    assert np.abs(O.float().cpu().numpy() - ref).max() <= parity.O_ATOL[dtype]
    plan.close()


def test_host_buffer_front_end():
    w = wl.WORKLOADS["ragged_bf16"]
    n = max(orc.count(w.c, L) for L in range(1, w.T + 1))
    inp = wl.make_inputs(w, n, B=4)
    tdt = torch.bfloat16
    plan = ps.Plan(4, w.H, w.T, dtype=tdt, c=w.c, idx_cols=n)
    plan.psattn_plan_enable_host_io()
    hQ, hK, hV = (torch.from_numpy(inp[k]).to(tdt).pin_memory() for k in ("Q", "K", "V"))
    hl = torch.from_numpy(inp["lengths"]).pin_memory()
    hi = torch.from_numpy(inp["sample_idx"]).pin_memory()
    hO = torch.empty((4, w.H, w.T, 64), dtype=tdt).pin_memory()
    hs = torch.empty((4, w.H, plan.u_max), dtype=torch.int32).pin_memory()
    plan.psattn_forward_host(hQ, hK, hV, hl, hi, hO, hs)
    parity.check_forward(hO.float().numpy(), hs.numpy(), None, inp, inp["lengths"], "bf16", w.c)
    plan.close()


def test_argument_errors_are_status_codes():
    plan = ps.Plan(1, 1, 64, c=5.0)
    x = torch.zeros((1, 1, 64, 64), dtype=torch.bfloat16, device="cuda")
    idx = torch.zeros((1, 64, plan.idx_cols), dtype=torch.int32, device="cuda")
    with pytest.raises(ps.PsattnError, match="NULL"):
        plan.psattn_forward(x, x, None, None, idx)
    with pytest.raises(ps.PsattnError, match="aligned"):
        plan.psattn_measure(x.view(-1)[1:], x, None, idx)
    small = plan.workspace
    plan.workspace_bytes_saved = plan.workspace_bytes
    plan.workspace_bytes = 16
    with pytest.raises(ps.PsattnError, match="workspace"):
        plan.psattn_forward(x, x, x, None, idx)
    plan.workspace_bytes = plan.workspace_bytes_saved
    with pytest.raises(ps.PsattnError):
        ps.Plan(1, 1, 64, d_head=32)
    with pytest.raises(ps.PsattnError):
        ps.Plan(1, 1, 64, idx_cols=3)                # narrower than the rule's U
    del small
    plan.close()


def test_forced_fused_path_and_its_limits():
    """PSATTN_PATH_FUSED runs the one-kernel schedule where it applies and refuses, with a status
    code, where it does not (fp32 inputs; keys that do not fit in shared memory)."""
    B, H, T, c = 2, 2, 384, 5.0
    n = orc.count(c, T)
    inp = _synth(B, H, T, 60, n, "bf16", [384, 201])
    before = ps.psattn_launch_count()
    O, sel, M, status = _run_forward(inp, "bf16", c, ps.PSATTN_PATH_FUSED)
    assert ps.psattn_launch_count() - before == 1          # the whole path was one kernel
    assert status == 0
    parity.check_forward(O, sel, M, inp, inp["lengths"], "bf16", c)
    inp32 = _synth(1, 1, 64, 61, orc.count(c, 64), "fp32")
    with pytest.raises(ps.PsattnError, match="unsupported"):
        _run_forward(inp32, "fp32", c, ps.PSATTN_PATH_FUSED)
    big = _synth(1, 1, 4096, 62, orc.count(c, 4096), "bf16")
    with pytest.raises(ps.PsattnError, match="unsupported"):
        _run_forward(big, "bf16", c, ps.PSATTN_PATH_FUSED)
