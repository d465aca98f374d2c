"""Pins for the CPU oracle: brute force, closed forms, invariants, special cases.

None of these tests touches the CUDA library.  Each pin names the passage of
the paper (arXiv 2106.09236) that fixes the expected value.
"""
import math
import os

import numpy as np
import pytest

import brute
from oracle import psattn_oracle as orc
from paper_2106_09236_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(B, H, T, d, seed, n_cols, lengths=None):
    rng = np.random.default_rng(seed)
    Q = rng.standard_normal((B, H, T, d)).astype(np.float32)
    K = rng.standard_normal((B, H, T, d)).astype(np.float32)
    V = rng.standard_normal((B, H, T, d)).astype(np.float32)
    if lengths is None:
        lengths = np.full(B, T, dtype=np.int32)
    idx = np.zeros((B, T, n_cols), dtype=np.int32)
    for b in range(B):
        L = int(lengths[b])
        idx[b, :L] = rng.integers(0, L, size=(L, n_cols))
    return Q, K, V, idx, np.asarray(lengths, dtype=np.int32)


# ---- sample-size rule (Sec. 3.2: L~ = r_sample ln L) -----------------------------------

def test_count_golden_table():
    """The workload definitions state the counts 25/32/35/46 for c = 5."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "sample_counts.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) >= 4
    for T, c, n in rows:
        assert orc.count(float(c), int(T)) == int(n)


def test_count_closed_form_and_clamps():
    for L in range(1, 700):
        for c in (0.3, 1.0, 5.0, 40.0):
            want = min(L, max(1, math.ceil(c * math.log(L))))
            assert orc.count(c, L) == want
    assert orc.count(5.0, 1) == 1          # ln 1 = 0 -> clamp up to one sample
    assert orc.count(5.0, 3) == 3          # ceil(5.49) = 6 -> clamp down to len
    assert orc.count(5.0, 0) == 0


# ---- P1: whole oracle vs brute force ----------------------------------------------------

@pytest.mark.parametrize("T", [1, 2, 3, 5, 8, 17, 32])
@pytest.mark.parametrize("fill", ["mean_v", "own_v"])
def test_brute_force_tiny(T, fill):
    B, H, d, c = 2, 2, 8, 1.5
    lengths = np.array([T, max(1, T - 2)], dtype=np.int32)
    ncol = max(brute.n_count(c, T), 1)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 100 + T, ncol, lengths)
    O, sel, M = orc.forward(Q, K, V, idx, lengths, c=c, fill=fill)
    Ob, selb, Mb = brute.forward(Q, K, V, idx, lengths, c, fill=fill)
    np.testing.assert_allclose(M, Mb, rtol=0, atol=1e-12)
    np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
    k = 0
    for b in range(B):
        for h in range(H):
            got = [int(x) for x in sel[b, h] if x >= 0]
            assert got == selb[k], (b, h)
            assert got == sorted(got)
            k += 1


def test_brute_force_d64_with_duplicates():
    """d = 64 as in the model; sample rows with forced duplicates (multiplicity in the mean)."""
    B, H, T, d, c = 1, 2, 24, 64, 2.0
    ncol = brute.n_count(c, T)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 7, ncol)
    idx[:, :, 1] = idx[:, :, 0]            # every row has a duplicate
    idx[:, 3, :] = 5                       # one row is a single key repeated
    O, sel, M = orc.forward(Q, K, V, idx, lengths, c=c)
    Ob, selb, Mb = brute.forward(Q, K, V, idx, lengths, c)
    np.testing.assert_allclose(M, Mb, atol=1e-12)
    np.testing.assert_allclose(O, Ob, atol=1e-12)
    assert M[0, 0, 3] == 0.0 and M[0, 1, 3] == 0.0


def test_brute_force_per_head_samples():
    """Sec. 3.2 leaves open whether the heads of a sequence share one sample; with a 4-D sample_idx
    [B][H][T][cols] every head has its own rows.  Different rows per head, ragged lengths: a wrong
    row stride in the per-head addressing of measure or forward fails here."""
    B, H, T, d, c = 2, 3, 19, 16, 2.0
    lengths = np.array([19, 11], dtype=np.int32)
    ncol = brute.n_count(c, T)
    rng = np.random.default_rng(4242)
    Q = rng.standard_normal((B, H, T, d)).astype(np.float32)
    K = rng.standard_normal((B, H, T, d)).astype(np.float32)
    V = rng.standard_normal((B, H, T, d)).astype(np.float32)
    idx = np.zeros((B, H, T, ncol), dtype=np.int32)
    for b in range(B):
        L = int(lengths[b])
        idx[b, :, :L] = rng.integers(0, L, size=(H, L, ncol))
    assert not np.array_equal(idx[:, 0], idx[:, 1])
    Mb = brute.forward(Q, K, V, idx, lengths, c)[2]
    M = orc.measure(Q, K, idx, lengths, c=c)
    np.testing.assert_allclose(M, Mb, rtol=0, atol=1e-12)
    for fill in ("mean_v", "own_v"):
        O, sel, M2 = orc.forward(Q, K, V, idx, lengths, c=c, fill=fill)
        Ob, selb, _ = brute.forward(Q, K, V, idx, lengths, c, fill=fill)
        np.testing.assert_allclose(M2, Mb, rtol=0, atol=1e-12)
        np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
        got = [[int(x) for x in sel[b, h] if x >= 0] for b in range(B) for h in range(H)]
        assert got == selb
    # the shared layout is the per-head layout with equal rows in every head
    shared = idx[:, 0]
    M_sh = orc.measure(Q, K, shared, lengths, c=c)
    M_rep = orc.measure(Q, K, np.repeat(shared[:, None], H, axis=1), lengths, c=c)
    np.testing.assert_array_equal(M_sh, M_rep)
    assert not np.allclose(M_sh, M)


def test_paper_count_rule_per_sequence():
    """Sec. 3.2: L_sparse = r_sparse L from every sequence's own length (rounded up, at least one).
    Ragged lengths: each sequence gets its own count; brute force on the whole path."""
    for L, r, want in ((1, 0.5, 1), (2, 0.5, 1), (3, 0.5, 2), (40, 0.35, 14), (500, 0.35, 175),
                       (501, 0.5, 251), (7, 0.01, 1), (7, 1.0, 7), (0, 0.5, 0)):
        assert orc.selected_count(L, r_sparse=r) == want
    assert orc.selected_count(100, c=5.0) == brute.n_count(5.0, 100)
    assert orc.selected_count(10, u_override=4) == 4 and orc.selected_count(3, u_override=4) == 3
    B, H, T, d, c = 3, 2, 21, 8, 1.5
    lengths = np.array([21, 9, 4], dtype=np.int32)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 77, brute.n_count(c, T), lengths)
    for r in (0.35, 0.5):
        O, sel, M = orc.forward(Q, K, V, idx, lengths, c=c, fill="own_v", r_sparse=r)
        Ob, selb, Mb = brute.forward(Q, K, V, idx, lengths, c, fill="own_v", r_sparse=r)
        assert sel.shape[-1] == math.ceil(r * T)
        np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
        got = [[int(x) for x in sel[b, h] if x >= 0] for b in range(B) for h in range(H)]
        assert got == selb
        for b in range(B):
            assert len(got[b * H]) == math.ceil(r * int(lengths[b]))
        sel2 = orc.select(M, lengths, c=c, r_sparse=r)
        np.testing.assert_array_equal(sel2, sel)


# ---- P2: u = len  ==> dense softmax attention (Eq. 6) ------------------------------------

def test_all_selected_equals_dense_attention():
    import torch
    B, H, T, d = 2, 3, 40, 16
    lengths = np.array([40, 29], dtype=np.int32)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 11, 6, lengths)
    O, sel, _ = orc.forward(Q, K, V, idx, lengths, c=1.0, u_override=T)
    Od = orc.dense(Q, K, V, lengths)
    np.testing.assert_allclose(O, Od, atol=1e-13)
    for b in range(B):
        L = int(lengths[b])
        assert [int(x) for x in sel[b, 0] if x >= 0] == list(range(L))
        q = torch.from_numpy(Q[b, :, :L]).double()
        k = torch.from_numpy(K[b, :, :L]).double()
        v = torch.from_numpy(V[b, :, :L]).double()
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v).numpy()
        np.testing.assert_allclose(O[b, :, :L], ref, atol=1e-10)
        assert np.all(O[b, :, L:] == 0.0)


# ---- P3: non-selected rows are the column mean of V -------------------------------------

def test_non_selected_rows_equal_mean_v():
    B, H, T, d, c = 2, 2, 50, 8, 1.0
    lengths = np.array([50, 33], dtype=np.int32)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 12, brute.n_count(c, T), lengths)
    O, sel, _ = orc.forward(Q, K, V, idx, lengths, c=c)
    vb = orc.mean_v(V, lengths)
    for b in range(B):
        L = int(lengths[b])
        for h in range(H):
            np.testing.assert_allclose(vb[b, h], V[b, h, :L].astype(np.float64).mean(axis=0),
                                       atol=1e-14)
            chosen = set(int(x) for x in sel[b, h] if x >= 0)
            assert len(chosen) == brute.n_count(c, L)
            for i in range(L):
                if i not in chosen:
                    np.testing.assert_array_equal(O[b, h, i], vb[b, h])


def test_own_value_fill_is_eq12_as_printed():
    B, H, T, d, c = 1, 2, 30, 8, 1.0
    Q, K, V, idx, lengths = _rand(B, H, T, d, 13, brute.n_count(c, T))
    O, sel, _ = orc.forward(Q, K, V, idx, lengths, c=c, fill="own_v")
    for h in range(H):
        chosen = set(int(x) for x in sel[0, h] if x >= 0)
        for i in range(T):
            if i not in chosen:
                np.testing.assert_array_equal(O[0, h, i], V[0, h, i].astype(np.float64))


# ---- P4: M >= 0, and M == 0 for a constant-score query ---------------------------------

def test_measure_nonnegative_and_zero_for_constant_scores():
    B, H, T, d = 1, 2, 64, 64
    Q, K, V, idx, lengths = _rand(B, H, T, d, 14, 21)
    Q[0, 0, 7] = 0.0                        # q = 0 -> every score 0
    idx[0, 9, :] = 4                        # one key repeated -> constant scores
    M = orc.measure(Q, K, idx, lengths, U_override=21)
    assert np.all(M >= 0.0)
    assert M[0, 0, 7] == 0.0
    assert M[0, 0, 9] == 0.0 and M[0, 1, 9] == 0.0
    K2 = np.broadcast_to(K[:, :, :1], K.shape).copy()   # all key rows equal
    M2 = orc.measure(Q, K2, idx, lengths, U_override=21)
    assert np.all(M2 == 0.0)


# ---- P5: closed form with orthogonal keys -------------------------------------------------

def test_measure_closed_form_orthogonal_keys():
    """K rows orthogonal with norm rho, q = alpha k_p, p drawn m times out of U:
    scores are alpha rho^2/sqrt(d) on p and 0 elsewhere, so
    M = (alpha rho^2 / sqrt(d)) (1 - m/U)."""
    T = d = 16
    rho, alpha, U = 1.5, 2.0, 8
    K = np.zeros((1, 1, T, d), dtype=np.float32)
    K[0, 0] = rho * np.eye(T, dtype=np.float32)
    Q = np.zeros_like(K)
    idx = np.zeros((1, T, U), dtype=np.int32)
    want = np.zeros(T)
    rng = np.random.default_rng(3)
    for i in range(T):
        p = (i * 5 + 1) % T
        m = i % (U + 1)                     # 0..U occurrences of p
        Q[0, 0, i] = alpha * K[0, 0, p]
        others = [j for j in range(T) if j != p]
        row = [p] * m + list(rng.choice(others, size=U - m))
        rng.shuffle(row)
        idx[0, i] = row
        want[i] = 0.0 if m == 0 else (alpha * rho * rho / math.sqrt(d)) * (1.0 - m / U)
    M = orc.measure(Q, K, idx, None, U_override=U)
    np.testing.assert_allclose(M[0, 0], want, atol=1e-14)


# ---- P6 / P7: relation to the exact measure (Eq. 10) --------------------------------------

def test_full_sample_is_max_minus_mean_over_all_keys():
    B, H, T, d = 1, 2, 20, 8
    Q, K, V, _, lengths = _rand(B, H, T, d, 15, 1)
    idx = np.tile(np.arange(T, dtype=np.int32), (B, T, 1))     # every key exactly once
    M = orc.measure(Q, K, idx, lengths, U_override=T)
    S = np.einsum("bhid,bhjd->bhij", Q.astype(np.float64), K.astype(np.float64)) / math.sqrt(d)
    np.testing.assert_allclose(M, S.max(-1) - S.mean(-1), atol=1e-13)
    # max <= LSE <= max + ln U  ==>  M~ <= M_exact <= M~ + ln U  on the same key multiset
    Mx = orc.exact_measure(Q, K, lengths)
    assert np.all(M <= Mx + 1e-12)
    assert np.all(Mx <= M + math.log(T) + 1e-12)
    lse = np.log(np.exp(S).sum(-1))
    np.testing.assert_allclose(Mx, lse - S.mean(-1), atol=1e-12)


def test_exact_measure_closed_forms():
    # Eq. 9-10: M - ln L is the divergence of the attention distribution from the uniform one: zero for
    # constant scores (M = ln L exactly), and in closed form for one score s above L - 1 zeros:
    # M = ln(e^s + L - 1) - s / L.  Padded keys (NaN here) are never read.
    B, H, T, d = 2, 2, 12, 16
    rng = np.random.default_rng(3)
    lengths = np.array([12, 7], dtype=np.int32)
    K = np.zeros((B, H, T, d), dtype=np.float32)
    rho = 1.5
    for t in range(T):
        K[:, :, t, t] = rho                                   # orthogonal keys of norm rho (T <= d)
    Q0 = np.zeros((B, H, T, d), dtype=np.float32)
    Q1 = np.zeros((B, H, T, d), dtype=np.float32)
    alpha = 2.0
    for b in range(B):
        for i in range(int(lengths[b])):
            Q1[b, :, i] = alpha * K[b, :, (i * 5) % int(lengths[b])]
    K[1, :, 7:] = np.nan
    Q0[1, :, 7:] = np.nan
    Q1[1, :, 7:] = np.nan
    M0 = orc.exact_measure(Q0, K, lengths)
    M1 = orc.exact_measure(Q1, K, lengths)
    s = alpha * rho * rho / math.sqrt(d)
    for b in range(B):
        L = int(lengths[b])
        np.testing.assert_allclose(M0[b, :, :L], math.log(L), atol=1e-13)
        np.testing.assert_allclose(M1[b, :, :L], math.log(math.exp(s) + L - 1) - s / L, atol=1e-13)
        assert np.all(M0[b, :, L:] == 0.0) and np.all(M1[b, :, L:] == 0.0)


# ---- P8: invariances -------------------------------------------------------------------

def test_invariances():
    B, H, T, d, c = 1, 2, 37, 16, 2.0
    ncol = brute.n_count(c, T)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 16, ncol)
    O, sel, M = orc.forward(Q, K, V, idx, lengths, c=c)
    rng = np.random.default_rng(5)
    # (i) order inside a sample row does not matter
    idx2 = idx.copy()
    for i in range(T):
        rng.shuffle(idx2[0, i])
    O2, sel2, M2 = orc.forward(Q, K, V, idx2, lengths, c=c)
    np.testing.assert_allclose(M2, M, atol=1e-13)
    np.testing.assert_array_equal(sel2, sel)
    # (ii) permuting keys and values together (sample remapped) leaves everything unchanged
    perm = rng.permutation(T)
    inv = np.argsort(perm)
    K3, V3 = K[:, :, perm], V[:, :, perm]
    idx3 = inv[idx].astype(np.int32)
    O3, sel3, M3 = orc.forward(Q, K3, V3, idx3, lengths, c=c)
    np.testing.assert_allclose(M3, M, atol=1e-13)
    np.testing.assert_array_equal(sel3, sel)
    np.testing.assert_allclose(O3, O, atol=1e-12)
    # (iii) one constant vector added to every key shifts all scores of a query equally
    shift = rng.standard_normal(d).astype(np.float32)
    K4 = (K.astype(np.float64) + shift).astype(np.float32)
    O4, sel4, M4 = orc.forward(Q, K4, V, idx, lengths, c=c)
    np.testing.assert_allclose(M4, M, atol=5e-5)      # float32 rounding of the shifted keys
    np.testing.assert_allclose(O4, O, atol=5e-4)


# ---- P9: linear in V; constant V -------------------------------------------------------

def test_constant_value_rows_and_linearity():
    B, H, T, d, c = 1, 2, 33, 8, 2.0
    Q, K, V, idx, lengths = _rand(B, H, T, d, 17, brute.n_count(c, T))
    w = np.arange(1, d + 1, dtype=np.float32)
    Vc = np.broadcast_to(w, V.shape).copy()
    O, _, _ = orc.forward(Q, K, Vc, idx, lengths, c=c)
    np.testing.assert_allclose(O, np.broadcast_to(w.astype(np.float64), O.shape), atol=1e-12)
    V2 = np.random.default_rng(1).standard_normal(V.shape).astype(np.float32)
    Oa, _, _ = orc.forward(Q, K, V, idx, lengths, c=c)
    Ob, _, _ = orc.forward(Q, K, V2, idx, lengths, c=c)
    Vs = (2.0 * V.astype(np.float64) + 0.5 * V2.astype(np.float64))
    # 2V + V2/2 is exact in float32 only up to rounding; compare with that rounding in mind
    Os, _, _ = orc.forward(Q, K, Vs.astype(np.float32), idx, lengths, c=c)
    np.testing.assert_allclose(Os, 2.0 * Oa + 0.5 * Ob, atol=1e-5)


# ---- P10: Q = 0 -> tie rule and uniform attention ----------------------------------------

def test_zero_queries_pick_lowest_indices_and_output_mean():
    B, H, T, d, c = 2, 2, 45, 8, 2.0
    lengths = np.array([45, 20], dtype=np.int32)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 18, brute.n_count(c, T), lengths)
    Q[:] = 0.0
    O, sel, M = orc.forward(Q, K, V, idx, lengths, c=c)
    assert np.all(M == 0.0)
    vb = orc.mean_v(V, lengths)
    for b in range(B):
        L = int(lengths[b])
        u = brute.n_count(c, L)
        for h in range(H):
            assert [int(x) for x in sel[b, h] if x >= 0] == list(range(u))
            assert np.all(sel[b, h, u:] == -1)
            np.testing.assert_allclose(O[b, h, :L], np.broadcast_to(vb[b, h], (L, d)), atol=1e-13)


# ---- signed zeros are one value -------------------------------------------------------------

def test_signed_zeros_tie_in_the_selection():
    """-0.0 and +0.0 compare equal, so among them the lower position wins (the tie rule), whatever their signs;
    checked against a stable sort of the values."""
    T, c = 40, 5.0
    rng = np.random.default_rng(77)
    M = np.where(rng.random((1, 1, T)) < 0.5, 0.0, -0.0)
    M[0, 0, [5, 17, 30]] = [1.0, -1.0, 2.0]
    u = brute.n_count(c, T)
    order = np.argsort(-M[0, 0], kind="stable")             # equal values keep their position order
    want = np.sort(order[:u])
    sel = orc.select(M, np.array([T], dtype=np.int32), c=c)
    assert [int(x) for x in sel[0, 0] if x >= 0] == [int(x) for x in want]
    assert 17 not in want and 5 in want and 30 in want


# ---- P11: planted spikes ---------------------------------------------------------------

def test_planted_spikes_are_selected():
    B, H, T, d, c = 1, 2, 96, 64, 3.0
    u = brute.n_count(c, T)
    Q, K, V, idx, lengths = _rand(B, H, T, d, 19, u)
    Q *= 0.05                               # flat background
    rng = np.random.default_rng(9)
    planted = []
    for h in range(H):
        qs = np.sort(rng.choice(T, size=u, replace=False))
        planted.append(list(int(x) for x in qs))
    # the sample is shared by the heads, so plant the same key column for every query
    for i in range(T):
        idx[0, i, 0] = (i * 7 + 3) % T
    for h in range(H):
        for i in planted[h]:
            Q[0, h, i] = 4.0 * K[0, h, idx[0, i, 0]]
    _, sel, _ = orc.forward(Q, K, V, idx, lengths, c=c)
    for h in range(H):
        assert [int(x) for x in sel[0, h] if x >= 0] == planted[h]


# ---- P12: padding --------------------------------------------------------------------------

def test_padding_contents_and_padded_length_do_not_matter():
    B, H, d, c = 2, 2, 16, 2.0
    lengths = np.array([19, 26], dtype=np.int32)
    T1, T2 = 26, 40
    Q, K, V, idx, lengths = _rand(B, H, T1, d, 20, brute.n_count(c, T1), lengths)
    O1, sel1, M1 = orc.forward(Q, K, V, idx, lengths, c=c)

    def grow(x, fillv):
        out = np.full((B, H, T2, d), fillv, dtype=np.float32)
        for b in range(B):
            out[b, :, :lengths[b]] = x[b, :, :lengths[b]]
        return out

    idx2 = np.zeros((B, T2, idx.shape[2]), dtype=np.int32)
    idx2[:, :T1] = idx
    O2, sel2, M2 = orc.forward(grow(Q, np.nan), grow(K, np.nan), grow(V, np.nan), idx2,
                               lengths, c=c)
    w1 = sel1.shape[-1]                     # u_max grows with the padded length; extra slots are -1
    np.testing.assert_array_equal(sel2[..., :w1], sel1)
    assert np.all(sel2[..., w1:] == -1)
    for b in range(B):
        L = int(lengths[b])
        np.testing.assert_array_equal(O2[b, :, :L], O1[b, :, :L])
        np.testing.assert_array_equal(M2[b, :, :L], M1[b, :, :L])
        assert np.all(O2[b, :, L:] == 0.0)


# ---- Sec. 4.4: a given index set is reused ------------------------------------------------

def test_given_selection_is_used_as_is():
    B, H, T, d, c = 1, 2, 30, 8, 2.0
    Q, K, V, idx, lengths = _rand(B, H, T, d, 21, brute.n_count(c, T))
    sel_in = np.full((B, H, 4), -1, dtype=np.int32)
    sel_in[0, 0, :3] = [2, 9, 17]
    sel_in[0, 1, :4] = [0, 1, 28, 29]
    O, sel, _ = orc.forward(Q, K, V, idx, lengths, c=c, sel_in=sel_in)
    np.testing.assert_array_equal(sel, sel_in)
    vb = orc.mean_v(V, lengths)
    for h in range(H):
        chosen = set(int(x) for x in sel_in[0, h] if x >= 0)
        for i in range(T):
            want = (brute.softmax_attention(Q[0, h, i], K[0, h], V[0, h]) if i in chosen
                    else vb[0, h])
            np.testing.assert_allclose(O[0, h, i], want, atol=1e-12)


# ---- the seeded workloads themselves -----------------------------------------------------

def test_workload_generator_is_deterministic_and_in_range():
    w = wl.WORKLOADS["ragged_bf16"]
    a = wl.make_inputs(w, 32, B=3)
    b = wl.make_inputs(w, 32, B=3)
    for k in a:
        np.testing.assert_array_equal(a[k], b[k])
    for bb in range(3):
        L = int(a["lengths"][bb])
        assert 40 <= L <= 500
        assert a["sample_idx"][bb, :L].min() >= 0 and a["sample_idx"][bb, :L].max() < L
        assert np.all(a["Q"][bb, :, L:] == 0)
    # bf16 rounding: the low 16 bits of every value are zero, and rounding is to nearest even
    assert np.all((a["Q"].view(np.uint32) & 0xFFFF) == 0)
    x = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20], dtype=np.float32)
    r = wl.round_to_bf16(x)
    np.testing.assert_array_equal(r, np.array([1.0, 1.0 + 2.0 ** -6, 1.0 + 2.0 ** -7], dtype=np.float32))


def test_peaky_queries_dominate_selection_on_tiny_workload():
    """On the tiny workload most selected queries are peaky ones (they are what M~ detects)."""
    w = wl.WORKLOADS["tiny_fp32"]
    n = orc.count(w.c, w.T)
    inp = wl.make_inputs(w, n)
    _, sel, _ = orc.forward(inp["Q"], inp["K"], inp["V"], inp["sample_idx"], inp["lengths"], c=w.c)
    hits = sum(bool(inp["peaky"][0, h, i]) for h in range(w.H) for i in sel[0, h] if i >= 0)
    total = int((sel >= 0).sum())
    assert total == w.H * n
    assert hits >= 0.3 * total      # 13 peaky of 128 per head; chance level would be ~10 %


# ---- projections (Sec. 3.1: Q = X W_q, K = X W_k, V = X W_v) ----------------------------------
def _proj_rand(B, T, dx, H, d, seed):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((B, T, dx)).astype(np.float32)
    Wt = rng.standard_normal((3, H * d, dx)).astype(np.float32)
    return X, Wt


def test_projection_equals_library_matmul():
    # the definition written with a library routine: per head, X @ W with W = Wt-slice transposed
    B, T, dx, H, d = 2, 7, 12, 3, 5
    X, Wt = _proj_rand(B, T, dx, H, d, 11)
    got = orc.project_qkv(X, Wt, H)
    for r in range(3):
        for h in range(H):
            W = Wt[r, h * d:(h + 1) * d, :].astype(np.float64).T          # (d_x, d)
            want = X.astype(np.float64) @ W                               # (B, T, d)
            np.testing.assert_allclose(got[r][:, h], want, rtol=1e-13, atol=1e-13)


def test_projection_identity_and_one_hot_cases():
    # W_q = I, W_k = 2 I, W_v = a cyclic shift of the columns: each head reads its own slice of X
    B, T, H, d = 1, 4, 2, 3
    dx = H * d
    rng = np.random.default_rng(5)
    X = rng.standard_normal((B, T, dx)).astype(np.float32)
    eye = np.eye(dx, dtype=np.float32)
    Wt = np.stack([eye, 2 * eye, np.roll(eye, 1, axis=1)])               # row o of role v picks x[(o + 1) % dx]
    Q, K, V = orc.project_qkv(X, Wt, H)
    for h in range(H):
        np.testing.assert_array_equal(Q[:, h], X[:, :, h * d:(h + 1) * d].astype(np.float64))
        np.testing.assert_array_equal(K[:, h], 2.0 * X[:, :, h * d:(h + 1) * d].astype(np.float64))
        cols = [(h * d + e + 1) % dx for e in range(d)]
        np.testing.assert_array_equal(V[:, h], X[:, :, cols].astype(np.float64))
    # a one-hot input row reads out one column of each transposed matrix: catches a transposed operand
    X1 = np.zeros((1, 1, dx), dtype=np.float32)
    X1[0, 0, 4] = 1.0
    _, Wr = _proj_rand(1, 1, dx, H, d, 6)
    out = orc.project_qkv(X1, Wr, H)
    for r in range(3):
        for h in range(H):
            np.testing.assert_array_equal(out[r][0, h, 0], Wr[r, h * d:(h + 1) * d, 4].astype(np.float64))


def test_projection_linearity_and_padding():
    B, T, dx, H, d = 2, 6, 8, 2, 4
    X, Wt = _proj_rand(B, T, dx, H, d, 21)
    X2, _ = _proj_rand(B, T, dx, H, d, 22)
    a = orc.project_qkv(X, Wt, H)
    b = orc.project_qkv(X2, Wt, H)
    s = orc.project_qkv((X.astype(np.float64) + 0.5 * X2).astype(np.float32), Wt, H)
    for r in range(3):
        np.testing.assert_allclose(s[r], a[r] + 0.5 * b[r], rtol=0, atol=2e-6)   # float32 rounding of the sum of inputs
    lengths = np.array([3, 6], dtype=np.int32)
    Xn = X.copy()
    Xn[0, 3:] = np.nan                                                   # padded rows are never read
    p = orc.project_qkv(Xn, Wt, H, lengths)
    for r in range(3):
        assert np.all(p[r][0, :, 3:] == 0.0)
        np.testing.assert_array_equal(p[r][0, :, :3], a[r][0, :, :3])
        np.testing.assert_array_equal(p[r][1], a[r][1])


def test_projection_workload_generator():
    w = wl.WORKLOADS["tiny_fp32"]
    a, b = wl.make_projection_inputs(w), wl.make_projection_inputs(w)
    assert a["X"].shape == (w.B, w.T, w.H * w.d) and a["Wt"].shape == (3, w.H * w.d, w.H * w.d)
    np.testing.assert_array_equal(a["X"], b["X"])
    np.testing.assert_array_equal(a["Wt"], b["Wt"])
    Q, _, _ = orc.project_qkv(a["X"], a["Wt"], w.H)
    assert 0.8 < Q.std() < 1.2                                           # unit-variance activations by construction


# ---- the output matrix that merges the heads (Sec. 2.2 Eq. 5, Sec. 3.1) ---------------------------

def test_output_projection_equals_library_matmul_of_concatenated_heads():
    rng = np.random.default_rng(31)
    B, H, T, d, dy = 2, 3, 7, 4, 5
    O = rng.standard_normal((B, H, T, d)).astype(np.float32)
    Wot = rng.standard_normal((dy, H * d)).astype(np.float32)
    lengths = np.array([7, 4], dtype=np.int32)
    Y = orc.project_out(O, Wot, lengths)
    concat = O.transpose(0, 2, 1, 3).reshape(B, T, H * d).astype(np.float64)     # heads side by side
    want = concat @ Wot.astype(np.float64).T
    want[1, 4:] = 0.0
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-12)


def test_output_projection_one_hot_identity_and_linearity():
    rng = np.random.default_rng(32)
    B, H, T, d = 1, 3, 5, 4
    O = rng.standard_normal((B, H, T, d)).astype(np.float32)
    # identity: the output is the concatenation of the heads (head h lands in columns h*d .. h*d+d-1)
    Y = orc.project_out(O, np.eye(H * d, dtype=np.float32))
    for h in range(H):
        np.testing.assert_array_equal(Y[0, :, h * d:(h + 1) * d], O[0, h].astype(np.float64))
    # one weight only, Wot[n0, k0] = 1: column n0 of Y reads feature k0 = (h0, e0); a transposed or
    # head-swapped operand reads another one
    dy, n0, h0, e0 = 6, 4, 2, 1
    Wot = np.zeros((dy, H * d), dtype=np.float32)
    Wot[n0, h0 * d + e0] = 1.0
    Y = orc.project_out(O, Wot)
    np.testing.assert_array_equal(Y[0, :, n0], O[0, h0, :, e0].astype(np.float64))
    assert np.count_nonzero(np.delete(Y, n0, axis=2)) == 0
    # linear in O and in the weights
    W1 = rng.standard_normal((dy, H * d)).astype(np.float32)
    O2 = rng.standard_normal((B, H, T, d)).astype(np.float32)
    np.testing.assert_allclose(orc.project_out(O + O2, W1), orc.project_out(O, W1) + orc.project_out(O2, W1),
                               atol=1e-5)


def test_output_projection_of_unselected_rows_is_one_row():
    """Eq. 12 with the mean(V) fill: every non-selected row of a unit is the same vector, so their rows of Y
    are identical (what the library's shortcut relies on); the selected rows differ."""
    B, H, T, d, c = 1, 2, 30, 8, 1.0
    Q, K, V, idx, lengths = _rand(B, H, T, d, 33, brute.n_count(c, T))
    O, sel, _ = orc.forward(Q, K, V, idx, lengths, c=c)
    rng = np.random.default_rng(34)
    Wot = rng.standard_normal((6, H * d)).astype(np.float32)
    Y = orc.project_out(O.astype(np.float32), Wot)
    chosen = set(int(x) for x in sel.reshape(-1) if x >= 0)
    rest = [t for t in range(T) if t not in chosen]
    assert len(rest) > 2 and len(chosen) > 0
    for t in rest[1:]:
        np.testing.assert_array_equal(Y[0, t], Y[0, rest[0]])
    vbar = orc.mean_v(V, lengths).astype(np.float32).astype(np.float64)
    want = sum(vbar[0, h] @ Wot[:, h * d:(h + 1) * d].astype(np.float64).T for h in range(H))
    np.testing.assert_allclose(Y[0, rest[0]], want, atol=1e-5)
    assert any(not np.allclose(Y[0, t], Y[0, rest[0]]) for t in chosen)
