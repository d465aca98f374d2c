"""Randomised parity sweep: psattn_forward against the oracle on seeded random shapes around the boundaries of the
kernels' regimes (tile sizes, the longest sequence the fused kernel takes), ragged and near-empty lengths, both
schedules, both fills, the count rules of Sec. 3.2."""
import numpy as np
import pytest
import torch

import parity
from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from test_parity_gpu import _dev, _run_forward, _synth

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
