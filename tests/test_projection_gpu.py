"""GPU parity of the projections Q = X W_q, K = X W_k, V = X W_v (Sec. 3.1) against the CPU oracle.

Tolerances.  The library accumulates in fp32 and rounds once to the output type; the oracle works in
fp64 on the same input values.
  * bf16 outputs: |d| <= 2^-8 |ref| + 1e-4.  Round-to-nearest leaves at most half a bf16 ulp
    (<= 2^-8 |ref|); the fp32 accumulation of d_x <= 512 products of size ~1/sqrt(d_x) adds ~1e-6.
    In addition the stored value must EQUAL the oracle's value rounded to bf16 except where the fp32 and
    fp64 sums straddle a rounding boundary: at most 0.5 % of the entries of size > 2^-6 (below that the
    fp32 accumulation error, ~1e-7 absolute, exceeds a bf16 ulp), and never by more than one ulp + 1e-5.
  * fp32 outputs: |d| <= 2e-5 max(1, |ref|).
  * mean(V): |d| <= 1e-4 + 2^-5 / len against the column mean of the oracle's V rounded to the output
    type: the stored V may differ from it by one bf16 ulp (<= 2^-6 for |v| < 4) in a few entries, and two
    such entries in one column of a sequence of `len` rows move its mean by 2^-5 / len.
Rows at positions >= lengths[b] must be left untouched (the outputs are pre-filled with NaN).
"""
import numpy as np
import pytest
import torch

from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import binding as ps
from paper_2106_09236_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _bf16_ulp(x):
    x = np.abs(x).astype(np.float32)
    e = np.floor(np.log2(np.maximum(x, 1e-30)))
    return np.exp2(e - 7)


def _check(got, ref, lengths, dtype):
    """got: float32 [B,H,T,d] read back from the device (NaN where never written); ref: float64."""
    B, H, T, d = ref.shape
    for b in range(B):
        L = int(lengths[b])
        assert np.isnan(got[b, :, L:]).all(), "a padded row was written (b=%d)" % b
        g, r = got[b, :, :L].astype(np.float64), ref[b, :, :L]
        assert not np.isnan(g).any(), "a valid row was not written (b=%d)" % b
        err = np.abs(g - r)
        if dtype == "bf16":
            assert (err <= 2.0 ** -8 * np.abs(r) + 1e-4).all(), "worst %g" % err.max()
            want = wl.round_to_bf16(r.astype(np.float32)).astype(np.float64)
            off = (g != want) & (np.abs(r) > 2.0 ** -6)
            assert off.size == 0 or off.mean() <= 5e-3, "%.3g of the entries differ from the rounded oracle value" % off.mean()
            assert (np.abs(g - want) <= 1.001 * _bf16_ulp(want) + 1e-5).all()
        else:
            assert (err <= 2e-5 * np.maximum(1.0, np.abs(r))).all(), "worst %g" % err.max()


def _run(inp, H, dtype, path=ps.PSATTN_PATH_AUTO, strides=None, with_vbar=True, alloc=None):
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    X = torch.from_numpy(inp["X"]).to("cuda", tdt)
    Wt = torch.from_numpy(inp["Wt"]).to("cuda", tdt)
    lengths = torch.from_numpy(inp["lengths"]).cuda()
    B, T, dx = inp["X"].shape
    plan = ps.Plan(B, H, T, dtype=tdt, path=path, strides=strides)
    if alloc is None:
        outs = [torch.full((B, H, T, 64), float("nan"), dtype=tdt, device="cuda") for _ in range(3)]
        views = outs
    else:
        outs, views = alloc(B, H, T, tdt)
    vbar = torch.full((B, H, 64), float("nan"), dtype=torch.float32, device="cuda") if with_vbar else None
    before = ps.psattn_launch_count()
    plan.psattn_project_qkv(X, Wt, lengths, outs[0], outs[1], outs[2], vbar)
    torch.cuda.synchronize()
    assert ps.psattn_launch_count() > before
    assert plan.psattn_read_status() == 0
    plan.close()
    res = [v.float().cpu().numpy() for v in views]
    return res, None if vbar is None else vbar.cpu().numpy()


def _compare(inp, H, dtype, res, vbar):
    ref = orc.project_qkv(inp["X"], inp["Wt"], H, inp["lengths"], nthreads=orc.max_threads())
    for got, r in zip(res, ref):
        _check(got, r, inp["lengths"], dtype)
    if vbar is not None:
        Vr = ref[2].astype(np.float32)
        if dtype == "bf16":
            Vr = wl.round_to_bf16(Vr)
        want = orc.mean_v(Vr, inp["lengths"])
        for b, L in enumerate(inp["lengths"]):
            assert np.abs(vbar[b] - want[b]).max() <= 1e-4 + 2.0 ** -5 / max(int(L), 1)


@pytest.mark.parametrize("name,nb", [("tiny_fp32", None), ("base_bf16", 4), ("ragged_bf16", 6), ("large_bf16", 2)])
def test_projection_matches_oracle_on_workload_shapes(name, nb):
    w = wl.WORKLOADS[name]
    inp = wl.make_projection_inputs(w, B=nb)
    res, vbar = _run(inp, w.H, w.dtype)
    _compare(inp, w.H, w.dtype, res, vbar)


@pytest.mark.parametrize("name", ["large_bf16", "long_bf16"])
def test_projection_full_size_on_sampled_tokens(name):
    # the full batch runs on the device; the oracle recomputes 96 sampled tokens per sequence
    w = wl.WORKLOADS[name]
    inp = wl.make_projection_inputs(w)
    res, vbar = _run(inp, w.H, w.dtype, with_vbar=False)
    rng = np.random.default_rng(99)
    for b in range(w.B):
        ts = np.sort(rng.choice(w.T, size=96, replace=False))
        ts[0], ts[-1] = 0, w.T - 1
        sub = {"X": inp["X"][b:b + 1, ts], "Wt": inp["Wt"], "lengths": np.array([len(ts)], dtype=np.int32)}
        ref = orc.project_qkv(sub["X"], sub["Wt"], w.H, sub["lengths"], nthreads=orc.max_threads())
        for got, r in zip(res, ref):
            _check(got[b:b + 1][:, :, ts], r, sub["lengths"], w.dtype)


@pytest.mark.parametrize("B,H,T,dx,lengths", [
    (3, 3, 130, 200, [130, 1, 129]),          # K tail (200 = 3 * 64 + 8), partial column tile (9 head blocks), 2 row tiles
    (2, 1, 300, 64, [0, 300]),                # one head: 3 blocks in one column tile; an empty sequence
    (2, 5, 128, 328, [128, 127]),             # 15 head blocks over 4 column tiles
    (1, 2, 40, 36, [40]),                     # d_x not a multiple of 8: no tensor map, plain kernel
])
def test_projection_ragged_shapes(B, H, T, dx, lengths):
    rng = np.random.default_rng(1000 + dx)
    X = wl.round_to_bf16(rng.standard_normal((B, T, dx), dtype=np.float32))
    Wt = wl.round_to_bf16(rng.standard_normal((3, H * 64, dx), dtype=np.float32) / np.float32(np.sqrt(dx)))
    inp = {"X": X, "Wt": Wt, "lengths": np.array(lengths, dtype=np.int32)}
    for b, L in enumerate(lengths):
        inp["X"][b, L:] = np.nan                                 # never read
    res, vbar = _run(inp, H, "bf16")
    inp["X"] = np.nan_to_num(inp["X"], nan=0.0)
    _compare(inp, H, "bf16", res, vbar)
    for b, L in enumerate(lengths):
        if L == 0:
            assert (vbar[b] == 0).all()


def test_projection_without_tensor_cores_and_fp32():
    w = wl.WORKLOADS["base_bf16"]
    inp = wl.make_projection_inputs(w, B=1, lengths=[300])
    res, vbar = _run(inp, w.H, "bf16", path=ps.PSATTN_PATH_STAGED)
    _compare(inp, w.H, "bf16", res, vbar)
    w32 = wl.Workload("adhoc", 0, 2, 2, 70, 64, "fp32", 5.0, 0.1, 3.0)
    inp = wl.make_projection_inputs(w32, lengths=[70, 33])
    res, vbar = _run(inp, 2, "fp32")
    _compare(inp, 2, "fp32", res, vbar)


def test_projection_writes_the_strided_layout_the_attention_reads():
    # outputs as [B][T][H][64] storage viewed as [B][H][T][64]: what a fused QKV buffer would look like
    w = wl.WORKLOADS["base_bf16"]
    inp = wl.make_projection_inputs(w, B=2, lengths=[512, 301])
    H, T = w.H, w.T
    st = [T * H * 64, 64, H * 64]

    def alloc(B, H_, T_, tdt):
        bufs = [torch.full((B, T_, H_, 64), float("nan"), dtype=tdt, device="cuda") for _ in range(3)]
        return bufs, [x.permute(0, 2, 1, 3) for x in bufs]
    res, vbar = _run(inp, H, "bf16", strides={"q": st, "k": st, "v": st}, alloc=alloc)
    _compare(inp, H, "bf16", res, vbar)


def test_projection_is_deterministic_and_feeds_the_forward_call():
    w = wl.WORKLOADS["base_bf16"]
    inp = wl.make_projection_inputs(w, B=3, lengths=[512, 200, 77])
    a, va = _run(inp, w.H, "bf16")
    b, vb = _run(inp, w.H, "bf16")
    for x, y in zip(a, b):
        np.testing.assert_array_equal(np.nan_to_num(x, nan=-1.0), np.nan_to_num(y, nan=-1.0))
    np.testing.assert_array_equal(va, vb)
    # the projected tensors go straight into the attention call (plumbing check: status, shapes, fill rows)
    tdt = torch.bfloat16
    n_cols = max(ps.psattn_count(w.c, L) for L in range(1, w.T + 1))
    plan = ps.Plan(3, w.H, w.T, dtype=tdt, c=w.c, idx_cols=n_cols)
    X = torch.from_numpy(inp["X"]).to("cuda", tdt)
    Wt = torch.from_numpy(inp["Wt"]).to("cuda", tdt)
    lengths = torch.from_numpy(inp["lengths"]).cuda()
    vbar = torch.empty((3, w.H, 64), dtype=torch.float32, device="cuda")
    Q, K, V = plan.psattn_project_qkv(X, Wt, lengths, vbar=vbar)
    rng = np.random.default_rng(3)
    idx = np.zeros((3, w.T, n_cols), dtype=np.int32)
    for bb, L in enumerate(inp["lengths"]):
        idx[bb, :L] = rng.integers(0, L, size=(L, n_cols))
    O, sel = plan.psattn_forward(Q, K, V, lengths, torch.from_numpy(idx).cuda())
    torch.cuda.synchronize()
    assert plan.psattn_read_status() == 0
    O, sel, vbar = O.float().cpu().numpy(), sel.cpu().numpy(), vbar.cpu().numpy()
    for bb, L in enumerate(inp["lengths"]):
        for h in range(w.H):
            chosen = set(int(i) for i in sel[bb, h] if i >= 0)
            rest = [i for i in range(int(L)) if i not in chosen]
            # every non-selected row holds mean(V), which the projection already reported
            assert np.abs(O[bb, h, rest] - vbar[bb, h]).max() <= 2e-2
    plan.close()


def test_projection_argument_errors():
    plan = ps.Plan(1, 2, 64, dtype=torch.bfloat16)
    X = torch.zeros((1, 64, 128), dtype=torch.bfloat16, device="cuda")
    Wt = torch.zeros((3, 128, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ps.PsattnError):
        plan.lib.psattn_project_qkv.restype = int
        ps._check(plan.lib.psattn_project_qkv(plan.handle, None, ps._ptr(Wt), 128, None, ps._ptr(X), ps._ptr(X),
                                              ps._ptr(X), None, *plan._ws(), None))
    with pytest.raises(ps.PsattnError):
        ps._check(plan.lib.psattn_project_qkv(plan.handle, ps._ptr(X), ps._ptr(Wt), 0, None, ps._ptr(X), ps._ptr(X),
                                              ps._ptr(X), None, *plan._ws(), None))
    plan.close()
