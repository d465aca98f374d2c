"""Tiny-size brute force in numpy float64, written straight from the paper's
equations and independent of ``oracle/`` (pure Python loops; only for T <= ~40).

Used to pin the oracle: a wrong sign, index or transposed operand in the C
oracle shows up as a mismatch against these few lines.
"""
import math

import numpy as np


def n_count(c, L):
    return min(L, max(1, math.ceil(c * math.log(L)))) if L > 0 else 0


def softmax_attention(q, Kmat, Vmat):
    """Eq. 7-8: sum_j softmax_j(q.k_j / sqrt(d)) v_j."""
    d = q.shape[0]
    s = Kmat.astype(np.float64) @ q.astype(np.float64) / math.sqrt(d)
    p = np.exp(s - s.max())
    p /= p.sum()
    return p @ Vmat.astype(np.float64)


def sampled_measure(q, Kmat, idx):
    """Eq. 11 on the sampled keys (duplicates count twice)."""
    d = q.shape[0]
    s = np.array([float(np.dot(q.astype(np.float64), Kmat[j].astype(np.float64))) / math.sqrt(d)
                  for j in idx])
    return s.max() - s.mean()


def forward(Q, K, V, sample_idx, lengths, c, u_override=0, U_override=0, fill="mean_v", r_sparse=0.0):
    """sample_idx [B, T, cols] (one sample per query, shared by the heads) or [B, H, T, cols]
    (every head draws its own).  r_sparse > 0: L_sparse = ceil(r_sparse * L) queries are selected
    (Sec. 3.2) instead of n(c, L)."""
    B, H, T, d = Q.shape
    per_head = np.ndim(sample_idx) == 4
    O = np.zeros((B, H, T, d))
    M = np.zeros((B, H, T))
    sels = []
    for b in range(B):
        L = int(lengths[b]) if lengths is not None else T
        U = U_override if U_override > 0 else n_count(c, L)
        u = min(u_override, L) if u_override > 0 else n_count(c, L)
        if r_sparse > 0 and L > 0:
            u = min(L, max(1, math.ceil(r_sparse * L)))
        for h in range(H):
            for i in range(L):
                row = sample_idx[b, h, i] if per_head else sample_idx[b, i]
                M[b, h, i] = sampled_measure(Q[b, h, i], K[b, h], row[:U])
            order = sorted(range(L), key=lambda i: (-M[b, h, i], i))
            chosen = sorted(order[:u])
            sels.append(chosen)
            vbar = V[b, h, :L].astype(np.float64).mean(axis=0)
            for i in range(L):
                if i in chosen:
                    O[b, h, i] = softmax_attention(Q[b, h, i], K[b, h, :L], V[b, h, :L])
                elif fill == "own_v":
                    O[b, h, i] = V[b, h, i]
                else:
                    O[b, h, i] = vbar
    return O, sels, M
