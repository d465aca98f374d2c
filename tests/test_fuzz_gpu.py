"""Randomised parity sweep: psattn_forward against the oracle on seeded random shapes around the boundaries of the
kernels' regimes (tile sizes, the longest sequence the fused kernel takes), ragged and near-empty lengths, both
schedules, both fills, the count rules of Sec. 3.2."""
import numpy as np
import pytest

import parity
from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from test_parity_gpu import _run_forward, _synth

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
