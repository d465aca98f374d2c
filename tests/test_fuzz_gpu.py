"""Randomised parity sweep: psattn_forward against the oracle on seeded random shapes around the boundaries of the
kernels' regimes (tile sizes, the longest sequence the fused kernel takes), ragged and near-empty lengths, both
schedules, both fills, the count rules of Sec. 3.2."""
import numpy as np
import pytest
import torch

import parity
from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from test_parity_gpu import _dev, _run_forward, _shared_sample, _synth

pytestmark = pytest.mark.gpu

EDGES_A = [1023, 1024, 1025, 1087, 1088, 1089, 1099, 1100, 1101, 1151, 1152, 1153, 1279, 1280, 1281]
EDGES_B = [255, 256, 257, 383, 384, 385, 511, 512, 513, 767, 768, 769]


def _case(rng, it):
    kind = rng.integers(0, 4)
    if kind == 0:
        T = int(rng.integers(1, 400))
    elif kind == 1:
        T = int(rng.choice(EDGES_A))
    elif kind == 2:
        T = int(rng.integers(1100, 3200))
    else:
        T = int(rng.choice(EDGES_B))
    B, H = int(rng.integers(1, 5)), int(rng.integers(1, 5))
    if T > 1500:
        B, H = min(B, 2), min(H, 3)
    c = float(rng.choice([5.0, 5.0, 3.0, 8.0]))
    dtype = "bf16" if rng.random() < 0.8 else "fp32"
    lengths = [int(rng.integers(max(1, T // 3), T + 1)) if rng.random() < 0.7 else T for _ in range(B)]
    if rng.random() < 0.15:
        lengths[0] = int(rng.integers(0, 3))
    path = [ps.PSATTN_PATH_AUTO, ps.PSATTN_PATH_STAGED][int(rng.integers(0, 2))]
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    if n_cols > 64 and dtype == "bf16":
        c = 5.0
        n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    plan_kw, check_kw = {}, {}
    opt = rng.integers(0, 5)
    if opt == 1:
        plan_kw["fill_mode"], check_kw["fill"] = ps.PSATTN_FILL_OWN_V, "own_v"
    elif opt == 2:
        r = float(rng.choice([0.1, 0.35, 0.5]))
        plan_kw.update(r_sparse=r, fill_mode=ps.PSATTN_FILL_OWN_V)
        check_kw.update(r_sparse=r, fill="own_v")
    elif opt == 3 and T >= 8:
        u = int(rng.integers(1, min(T, 200)))
        plan_kw["u_override"], check_kw["u_override"] = u, u
    return dict(B=B, H=H, T=T, c=c, dtype=dtype, lengths=lengths, path=path, n_cols=n_cols, seed=9000 + it,
                plan_kw=plan_kw, check_kw=check_kw)


@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_match_the_oracle(seed):
    rng = np.random.default_rng(seed)
    for it in range(40):
        k = _case(rng, it)
        inp = _synth(k["B"], k["H"], k["T"], k["seed"], k["n_cols"], k["dtype"], k["lengths"])
        O, sel, M, status = _run_forward(inp, k["dtype"], k["c"], k["path"], **k["plan_kw"])
        assert status == 0, k
        try:
            parity.check_forward(O, sel, M, inp, inp["lengths"], k["dtype"], k["c"], **k["check_kw"])
        except AssertionError as e:
            raise AssertionError("case %r: %s" % ({x: k[x] for x in k if x != "check_kw"}, e))


@pytest.mark.parametrize("seed", [1, 2])
def test_random_dense_row_list_and_selection_calls_match_the_oracle(seed):
    """The per-step entry points on random shapes: the dense comparator, step (d) for random row lists (few rows:
    the 64-row kernel; with a larger u: the 256-row kernel; holes and repeated rows included) and step (c) on
    random values with heavy ties and zeros of both signs."""
    rng = np.random.default_rng(seed)
    for it in range(30):
        T = int(rng.choice([rng.integers(1, 300), rng.choice([127, 128, 129, 255, 256, 257, 511, 512, 513, 1023, 1024, 1025]),
                            rng.integers(300, 2600)]))
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 4))
        dtype = "bf16" if rng.random() < 0.8 else "fp32"
        lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
        inp = _synth(B, H, T, 7000 + it, 4, dtype, lengths)
        dev, tdt = _dev(inp, dtype)
        u_over = int(rng.integers(65, 300)) if (dtype == "bf16" and T > 300 and rng.random() < 0.4) else 0
        plan = ps.Plan(B, H, T, dtype=tdt, c=5.0, u_override=u_over)
        what = dict(B=B, H=H, T=T, dtype=dtype, lengths=lengths, u_override=u_over)
        if T <= 1300:
            O = plan.psattn_dense_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"])
            torch.cuda.synchronize()
            ref = orc.dense(inp["Q"], inp["K"], inp["V"], inp["lengths"], nthreads=8)
            assert np.abs(O.float().cpu().numpy() - ref).max() <= parity.O_ATOL[dtype], what
        n_rows = int(rng.integers(1, plan.u_max + 1))
        rows = np.stack([[rng.integers(0, lengths[b], size=n_rows) for _ in range(H)] for b in range(B)]).astype(np.int32)
        rows[rng.random(rows.shape) < 0.05] = -1
        if T > 3:
            rows[0, 0, 0] = T - 1
        out = plan.psattn_attend_rows(dev["Q"], dev["K"], dev["V"], dev["lengths"], torch.from_numpy(rows).cuda())
        torch.cuda.synchronize()
        out = out.cpu().numpy()
        # fp32 rows out; with bf16 inputs the weights are rounded to bf16 (2^-9 relative) before they meet |V| <= 4
        tol = 1e-4 if dtype == "fp32" else 8e-3
        for b in range(B):
            for h in range(H):
                for r in rng.choice(n_rows, size=min(n_rows, 6), replace=False):
                    i = int(rows[b, h, r])
                    if i < 0 or i >= lengths[b]:
                        assert np.all(out[b, h, r] == 0.0), what
                    else:
                        ref = orc.attend_row(inp["Q"], inp["K"], inp["V"], b, h, i, lengths[b])
                        assert np.abs(out[b, h, r] - ref).max() <= tol, what
        M = rng.standard_normal((B, H, T)).astype(np.float32)
        if rng.random() < 0.5:
            M = np.round(M * 2) / 2                           # steps of 0.5: many ties, -0.0 and +0.0 among them
        sel = plan.psattn_select(torch.from_numpy(M).cuda(), dev["lengths"])
        torch.cuda.synchronize()
        np.testing.assert_array_equal(sel.cpu().numpy(), orc.select(M.astype(np.float64), np.asarray(lengths, dtype=np.int32),
                                                                    c=5.0, u_override=u_over, u_max=plan.u_max), err_msg=repr(what))
        assert plan.psattn_read_status() == 0, what
        plan.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_index_layouts_strides_and_reused_selections_match_the_oracle(seed):
    """Per-head sample arrays, one sample per sequence, U overrides, the [B][T][H][d] layout through the stride fields,
    and a selection computed on one set of tensors reused on another (Sec. 4.4), on random shapes."""
    rng = np.random.default_rng(seed)
    c, d = 5.0, 64
    for it in range(24):
        T = int(rng.choice([rng.integers(2, 300), rng.choice([255, 256, 257, 1023, 1024, 1025, 1099, 1100, 1101]),
                            rng.integers(300, 2600)]))
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 5))
        dtype = "bf16" if rng.random() < 0.75 else "fp32"
        lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
        path = [ps.PSATTN_PATH_AUTO, ps.PSATTN_PATH_STAGED][int(rng.integers(0, 2))]
        U_over = int(rng.choice([0, 0, rng.integers(1, 64)]))
        n_cols = max(max(orc.count(c, L) for L in range(1, T + 1)), U_over)
        inp = _synth(B, H, T, 5000 + it, n_cols, dtype, lengths)
        mode = int(rng.integers(0, 4))
        what = dict(B=B, H=H, T=T, dtype=dtype, lengths=lengths, path=path, U_override=U_over, mode=mode)
        if mode == 0:
            idx = rng.integers(0, np.asarray(lengths)[:, None, None, None], size=(B, H, T, n_cols)).astype(np.int32)
            O, sel, M, status = _run_forward(dict(inp, sample_idx=idx), dtype, c, path, idx_per_head=True, U_override=U_over)
            assert status == 0, what
            parity.check_forward(O, sel, M, dict(inp, sample_idx=idx), inp["lengths"], dtype, c, U_override=U_over)
        elif mode == 1:
            compact, expanded = _shared_sample(inp)
            O, sel, M, status = _run_forward(dict(inp, sample_idx=compact), dtype, c, path, idx_shared=True, U_override=U_over)
            assert status == 0, what
            parity.check_forward(O, sel, M, dict(inp, sample_idx=expanded), inp["lengths"], dtype, c, U_override=U_over)
        elif mode == 2:
            dev, tdt = _dev(inp, dtype)
            st = (T * H * d, d, H * d)
            perm = {k: dev[k].permute(0, 2, 1, 3).contiguous() for k in ("Q", "K", "V")}
            plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n_cols, path=path, U_override=U_over,
                           strides={"q": st, "k": st, "v": st, "o": st})
            O = torch.full((B, T, H, d), float("nan"), dtype=tdt, device="cuda")
            sel = torch.empty((B, H, plan.u_max), dtype=torch.int32, device="cuda")
            M = torch.empty((B, H, T), dtype=torch.float32, device="cuda")
            plan.psattn_forward(perm["Q"], perm["K"], perm["V"], dev["lengths"], dev["sample_idx"], O, sel, M)
            torch.cuda.synchronize()
            assert plan.psattn_read_status() == 0, what
            parity.check_forward(O.permute(0, 2, 1, 3).float().cpu().numpy(), sel.cpu().numpy(), M.cpu().numpy(), inp,
                                 inp["lengths"], dtype, c, U_override=U_over)
            plan.close()
        else:
            dev, tdt = _dev(inp, dtype)
            inp2 = _synth(B, H, T, 6000 + it, n_cols, dtype, lengths)
            dev2, _ = _dev(inp2, dtype)
            plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n_cols, path=path, U_override=U_over)
            _, sel = plan.psattn_forward(dev["Q"], dev["K"], dev["V"], dev["lengths"], dev["sample_idx"])
            O2 = plan.psattn_forward_with_selection(dev2["Q"], dev2["K"], dev2["V"], dev["lengths"], sel)
            torch.cuda.synchronize()
            assert plan.psattn_read_status() == 0, what
            O2, s_host = O2.float().cpu().numpy(), sel.cpu().numpy()
            vbar = orc.mean_v(inp2["V"], inp["lengths"])
            for b in range(B):
                L = lengths[b]
                for h in range(H):
                    chosen = set(int(x) for x in s_host[b, h] if x >= 0)
                    for i in list(chosen)[:4] + [int(x) for x in rng.integers(0, L, size=4)]:
                        ref = orc.attend_row(inp2["Q"], inp2["K"], inp2["V"], b, h, i, L) if i in chosen else vbar[b, h]
                        assert np.abs(O2[b, h, i] - ref).max() <= parity.O_ATOL[dtype], what
                    assert np.all(O2[b, h, L:] == 0.0), what
            plan.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_projection_shapes_match_the_oracle(seed):
    """The projections in front of the path on random widths (multiples of 64, of 8, and widths the tensor map cannot
    take), head counts, lengths with empty sequences, NaN in the padding."""
    import test_projection_gpu as tpj
    from paper_2106_09236_b200 import workloads as wl
    rng = np.random.default_rng(seed)
    for it in range(20):
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 7))
        T = int(rng.choice([rng.integers(1, 200), rng.choice([127, 128, 129, 255, 256, 257, 383, 384, 385]), rng.integers(200, 900)]))
        dx = int(rng.choice([8 * rng.integers(1, 80), 64 * rng.integers(1, 9), 512, 4 * rng.integers(1, 30) + 2]))
        lengths = [int(rng.integers(0, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
        X = wl.round_to_bf16(rng.standard_normal((B, T, dx), dtype=np.float32))
        Wt = wl.round_to_bf16(rng.standard_normal((3, H * 64, dx), dtype=np.float32) / np.float32(np.sqrt(dx)))
        inp = {"X": X, "Wt": Wt, "lengths": np.array(lengths, dtype=np.int32)}
        for b, L in enumerate(lengths):
            inp["X"][b, L:] = np.nan                              # never read
        res, vbar = tpj._run(inp, H, "bf16")
        inp["X"] = np.nan_to_num(inp["X"], nan=0.0)
        tpj._compare(inp, H, "bf16", res, vbar)


@pytest.mark.parametrize("seed", [1, 2])
def test_random_counts_around_64_long_ragged_and_many_short_units(seed):
    """c chosen so that u and U fall around 63 / 64 / 65 (the limits of the 64-row attention kernel, of the fused
    kernel and of the tensor-datapath measure kernels), sequences of 3000-10000 positions with ragged lengths, and
    batches of many short units."""
    rng = np.random.default_rng(seed)
    for it in range(18):
        kind = int(rng.integers(0, 3))
        if kind == 0:
            T = int(rng.choice([rng.integers(900, 1101), rng.integers(1101, 3000)]))
            c, B, H = float(rng.uniform(8.4, 9.8)), int(rng.integers(1, 3)), int(rng.integers(1, 4))
        elif kind == 1:
            T, c, B, H = int(rng.integers(3000, 10000)), 5.0, int(rng.integers(1, 4)), int(rng.integers(1, 9))
        else:
            T, c = int(rng.integers(1, 200)), float(rng.choice([1.0, 5.0, 12.0]))
            B, H = int(rng.integers(4, 40)), int(rng.integers(1, 9))
        dtype = "bf16" if rng.random() < 0.85 else "fp32"
        lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.7 else T for _ in range(B)]
        path = [ps.PSATTN_PATH_AUTO, ps.PSATTN_PATH_STAGED][int(rng.integers(0, 2))]
        n_cols = max(orc.count(c, L) for L in range(1, T + 1))
        inp = _synth(B, H, T, 3000 + it, n_cols, dtype, lengths)
        what = dict(B=B, H=H, T=T, c=c, dtype=dtype, lengths=lengths[:6], path=path, U=n_cols)
        O, sel, M, status = _run_forward(inp, dtype, c, path)
        assert status == 0, what
        try:
            parity.check_forward(O, sel, M, inp, inp["lengths"], dtype, c)
        except AssertionError as e:
            raise AssertionError("case %r: %s" % (what, e))


@pytest.mark.parametrize("seed", [1, 2])
def test_random_output_matrix_shapes_match_the_oracle(seed):
    """The output matrix behind the path, both forms, on random head counts (odd ones included), widths, lengths."""
    import test_project_out_gpu as tpo
    from paper_2106_09236_b200 import workloads as wl
    rng = np.random.default_rng(seed)
    for it in range(20):
        H, B = int(rng.integers(1, 9)), int(rng.integers(1, 5))
        T = int(rng.choice([rng.integers(1, 300), rng.choice([127, 128, 129, 255, 256, 257]), rng.integers(300, 2200)]))
        c = float(rng.choice([5.0, 5.0, 2.0, 9.0]))
        dy = int(rng.choice([64 * rng.integers(1, 9), 8 * rng.integers(1, 70), 512]))
        lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
        n_cols = max(orc.count(c, L) for L in range(1, T + 1))
        if n_cols > 64:
            c = 5.0
            n_cols = max(orc.count(c, L) for L in range(1, T + 1))
        wk = wl.Workload("adhoc", 0, B, H, T, 64, "bf16", c, 0.1, 3.0)
        inp = wl.make_inputs(wk, n_cols, seed=8000 + it, lengths=lengths)
        plan, O, sel, lens, tdt = tpo._forward(inp, "bf16", c)
        tpo._run_all_forms(plan, O, sel, lens, tpo._weights(H, dy, 9 + it, "bf16"), tdt, "bf16", inp["lengths"])
        plan.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_calls_of_the_other_entry_points_match_the_oracle(seed):
    """The exact measure of Eq. 10, mean(V), the sampled measure alone on long ragged sequences, row lists over long sequences (key splits and their merge), and the
    host-buffer front end."""
    rng = np.random.default_rng(seed)
    for it in range(20):
        mode = int(rng.integers(0, 5))
        B, H = int(rng.integers(1, 4)), int(rng.integers(1, 6))
        dtype = "bf16" if rng.random() < 0.75 else "fp32"
        path = [ps.PSATTN_PATH_AUTO, ps.PSATTN_PATH_STAGED][int(rng.integers(0, 2))]
        c = 5.0
        what = dict(mode=mode, B=B, H=H, dtype=dtype, path=path)
        if mode == 0:      # exact measure
            T = int(rng.choice([rng.integers(1, 200), rng.choice([127, 128, 129, 255, 256, 257, 511, 512, 513]), rng.integers(200, 900)]))
            lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
            what.update(T=T, lengths=lengths)
            inp = _synth(B, H, T, 100 + it, orc.count(c, T), dtype, lengths)
            dev, tdt = _dev(inp, dtype)
            plan = ps.Plan(B, H, T, dtype=tdt, c=c, path=path)
            M = plan.psattn_exact_measure(dev["Q"], dev["K"], dev["lengths"]); torch.cuda.synchronize()
            assert plan.psattn_read_status() == 0
            parity.check_measure(M.cpu().numpy(), orc.exact_measure(inp["Q"], inp["K"], inp["lengths"]), inp["lengths"])
            plan.close()
        elif mode == 1:    # mean(V)
            T = int(rng.integers(1, 5000))
            lengths = [int(rng.integers(0, T + 1)) if rng.random() < 0.7 else T for _ in range(B)]
            what.update(T=T, lengths=lengths)
            inp = _synth(B, H, T, 200 + it, 4, dtype, [max(1, L) for L in lengths])
            inp["lengths"] = np.asarray(lengths, dtype=np.int32)
            dev, tdt = _dev(inp, dtype)
            plan = ps.Plan(B, H, T, dtype=tdt, c=c)
            vb = plan.psattn_mean_v(dev["V"], dev["lengths"])
            torch.cuda.synchronize()
            ref = orc.mean_v(inp["V"], inp["lengths"])
            assert np.abs(vb.cpu().numpy() - ref).max() <= 1e-4, what
            plan.close()
        elif mode == 2:    # measure alone, long and ragged
            T = int(rng.integers(1101, 9000)); B = min(B, 2); H = min(H, 3)
            lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
            what.update(T=T, lengths=lengths, B=B, H=H)
            n = max(orc.count(c, L) for L in range(1, T + 1))
            inp = _synth(B, H, T, 300 + it, n, dtype, lengths)
            dev, tdt = _dev(inp, dtype)
            plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n, path=path)
            M = plan.psattn_measure(dev["Q"], dev["K"], dev["lengths"], dev["sample_idx"]); torch.cuda.synchronize()
            assert plan.psattn_read_status() == 0
            parity.check_measure(M.cpu().numpy(), orc.measure(inp["Q"], inp["K"], inp["sample_idx"], inp["lengths"], c=c), inp["lengths"])
            plan.close()
        elif mode == 3:    # row lists over long sequences (key splits and their merge)
            T = int(rng.integers(1500, 9000)); B = min(B, 2); H = min(H, 3)
            lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.5 else T for _ in range(B)]
            what.update(T=T, lengths=lengths, B=B, H=H)
            inp = _synth(B, H, T, 400 + it, 4, dtype, lengths)
            dev, tdt = _dev(inp, dtype)
            u_over = int(rng.integers(65, 200)) if (dtype == "bf16" and rng.random() < 0.4) else 0
            plan = ps.Plan(B, H, T, dtype=tdt, c=c, u_override=u_over, path=path)
            n_rows = int(rng.integers(1, plan.u_max + 1))
            rows = np.stack([[rng.integers(0, lengths[b], size=n_rows) for _ in range(H)] for b in range(B)]).astype(np.int32)
            out = plan.psattn_attend_rows(dev["Q"], dev["K"], dev["V"], dev["lengths"], torch.from_numpy(rows).cuda())
            torch.cuda.synchronize(); out = out.cpu().numpy()
            assert plan.psattn_read_status() == 0
            tol = 1e-4 if dtype == "fp32" else 8e-3
            for b in range(B):
                for h in range(H):
                    for r in rng.choice(n_rows, size=min(n_rows, 3), replace=False):
                        ref = orc.attend_row(inp["Q"], inp["K"], inp["V"], b, h, int(rows[b, h, r]), lengths[b])
                        assert np.abs(out[b, h, r] - ref).max() <= tol, ("row", b, h, r)
            plan.close()
        else:              # host buffers
            T = int(rng.choice([rng.integers(1, 300), rng.integers(1101, 2500)])); B = int(rng.integers(1, 6))
            lengths = [int(rng.integers(1, T + 1)) if rng.random() < 0.6 else T for _ in range(B)]
            what.update(T=T, lengths=lengths, B=B)
            n = max(orc.count(c, L) for L in range(1, T + 1))
            inp = _synth(B, H, T, 500 + it, n, "bf16", lengths)
            tdt = torch.bfloat16
            plan = ps.Plan(B, H, T, dtype=tdt, c=c, idx_cols=n, path=path)
            plan.psattn_plan_enable_host_io()
            hQ, hK, hV = (torch.from_numpy(inp[k]).to(tdt).pin_memory() for k in ("Q", "K", "V"))
            hl = torch.from_numpy(inp["lengths"]).pin_memory(); hi = torch.from_numpy(inp["sample_idx"]).pin_memory()
            hO = torch.empty((B, H, T, 64), dtype=tdt).pin_memory(); hs = torch.empty((B, H, plan.u_max), dtype=torch.int32).pin_memory()
            plan.psattn_forward_host(hQ, hK, hV, hl, hi, hO, hs)
            parity.check_forward(hO.float().numpy(), hs.numpy(), None, inp, inp["lengths"], "bf16", c)
            plan.close()



def test_more_units_than_a_grid_dimension_holds():
    """70 000 units of 16 positions: more than the 65 535 blocks a grid's y or z dimension can number."""
    B, H, T, c = 8750, 8, 16, 5.0
    n_cols = max(orc.count(c, L) for L in range(1, T + 1))
    lengths = [T if b % 3 else T // 2 for b in range(B)]
    inp = _synth(B, H, T, 5, n_cols, "bf16", lengths)
    O, sel, M, status = _run_forward(inp, "bf16", c, ps.PSATTN_PATH_AUTO)
    assert status == 0
    parity.check_forward(O, sel, M, inp, inp["lengths"], "bf16", c, nthreads=16)


@pytest.mark.parametrize("B,H,T,lengths", [(1, 2, 65536, [65536]), (1, 1, 200000, [199999])])
def test_very_long_sequences(B, H, T, lengths):
    """Far beyond the longest named workload: the streaming measure kernel, the selection over ranges (65 536) or over
    a list too long for shared memory (200 000), many key splits in step (d)."""
    c = 5.0
    n_cols = orc.count(c, T)
    inp = _synth(B, H, T, 6, n_cols, "bf16", lengths)
    O, sel, M, status = _run_forward(inp, "bf16", c, ps.PSATTN_PATH_AUTO)
    assert status == 0
    parity.check_forward(O, sel, M, inp, inp["lengths"], "bf16", c, nthreads=16)
