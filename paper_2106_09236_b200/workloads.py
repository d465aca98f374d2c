"""Seeded synthetic workloads shaped like Conformer self-attention inputs.

This module only *draws inputs*.  It holds none of the method's arithmetic (no
scores, no measure, no selection, no sample-size rule): the number of sample
columns to draw is an argument.  Both the CUDA tests/benchmark and the CPU
oracle tests read their inputs from here so that they see identical data.

Shapes follow the model sizes of Sec. 4.2 of the paper (d_model 256 or 512,
4 or 8 heads => d_head = 64; T = number of 10 ms frames / 4 after the
convolutional down-sampling).  Values are synthetic stand-ins for activations
of AISHELL-1 / LibriSpeech utterances, which are not available offline:
Q, K, V ~ N(0, 1) i.i.d.; a fraction of the queries is made "peaky" by adding
a multiple of one key row, so that a few queries have far-from-uniform
attention, the situation the sparsity measure is meant to detect.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

BASE_SEED = 20210616


@dataclass(frozen=True)
class Workload:
    name: str
    number: int          # 1-based position in the configuration list
    B: int
    H: int
    T: int               # padded length T_max
    d: int
    dtype: str           # "fp32" or "bf16"
    c: float             # sampling factor (sample size and number selected grow as c ln len)
    peaky_frac: float
    peaky_scale: float
    ragged: tuple | None = None   # (lo, hi) inclusive range of valid lengths, or None

    @property
    def seed(self) -> int:
        return BASE_SEED + self.number


WORKLOADS = {
    "tiny_fp32": Workload("tiny_fp32", 1, 1, 4, 128, 64, "fp32", 5.0, 0.10, 3.0),
    "base_bf16": Workload("base_bf16", 2, 32, 4, 512, 64, "bf16", 5.0, 0.10, 3.0),
    "ragged_bf16": Workload("ragged_bf16", 3, 64, 4, 500, 64, "bf16", 5.0, 0.10, 3.0, (40, 500)),
    "large_bf16": Workload("large_bf16", 4, 16, 8, 1024, 64, "bf16", 5.0, 0.05, 4.0),
    "long_bf16": Workload("long_bf16", 5, 4, 8, 8192, 64, "bf16", 5.0, 0.10, 3.0),
}


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = x.view(np.uint32).astype(np.uint64)
    bias = ((bits >> 16) & 1) + 0x7FFF
    out = (((bits + bias) >> 16) << 16).astype(np.uint32)
    return out.view(np.float32).reshape(x.shape)


def make_inputs(w: Workload, n_cols: int, seed: int | None = None, B: int | None = None,
                pad_value: float = 0.0, lengths=None):
    """Draw one batch.

    n_cols  number of sampled-key columns drawn for every query (the caller
            derives it from the sample-size rule of whichever side it tests).
    B       optional override of the batch size (same per-sequence recipe).
    lengths optional explicit valid lengths (then none are drawn).
    Returns a dict of numpy arrays: Q, K, V float32 [B,H,T,d] (already rounded
    to bf16 values when w.dtype == "bf16"), lengths int32 [B], sample_idx int32
    [B,T,n_cols] with every entry of row (b, i) in [0, lengths[b]), and `peaky`
    bool [B,H,T].  Rows at padded positions hold `pad_value`.
    Draw order: lengths, Q, K, V, peaky query sets, peaky key choices, sample_idx.
    """
    rng = np.random.default_rng(w.seed if seed is None else seed)
    nb = w.B if B is None else B
    H, T, d = w.H, w.T, w.d
    if lengths is not None:
        lengths = np.asarray(lengths, dtype=np.int32)
        nb = int(lengths.shape[0])
    elif w.ragged is not None:
        lengths = rng.integers(w.ragged[0], w.ragged[1] + 1, size=nb).astype(np.int32)
    else:
        lengths = np.full(nb, T, dtype=np.int32)
    Q = rng.standard_normal((nb, H, T, d), dtype=np.float32)
    K = rng.standard_normal((nb, H, T, d), dtype=np.float32)
    V = rng.standard_normal((nb, H, T, d), dtype=np.float32)
    peaky = np.zeros((nb, H, T), dtype=bool)
    for b in range(nb):
        L = int(lengths[b])
        n_peaky = int(round(w.peaky_frac * L))
        for h in range(H):
            qs = rng.choice(L, size=n_peaky, replace=False)
            ks = rng.integers(0, L, size=n_peaky)
            Q[b, h, qs] += np.float32(w.peaky_scale) * K[b, h, ks]
            peaky[b, h, qs] = True
    sample_idx = np.zeros((nb, T, n_cols), dtype=np.int32)
    for b in range(nb):
        L = int(lengths[b])
        sample_idx[b, :L] = rng.integers(0, L, size=(L, n_cols), dtype=np.int32)
    for b in range(nb):
        L = int(lengths[b])
        if L < T:
            Q[b, :, L:] = pad_value
            K[b, :, L:] = pad_value
            V[b, :, L:] = pad_value
    if w.dtype == "bf16":
        Q, K, V = round_to_bf16(Q), round_to_bf16(K), round_to_bf16(V)
    return {"Q": Q, "K": K, "V": V, "lengths": lengths, "sample_idx": sample_idx, "peaky": peaky}


def make_projection_inputs(w: Workload, seed: int | None = None, B: int | None = None, lengths=None,
                           pad_value: float = 0.0):
    """Draw the inputs of the projections that precede the attention (Sec. 3.1): the layer input
    X float32 [B, T, d_x] with d_x = H * d (the model width of Sec. 4.2), i.i.d. N(0, 1), and the
    three weight matrices stored transposed, Wt float32 [3, H*d, d_x], i.i.d. N(0, 1/d_x) so that
    projected values have unit variance.  Rounded to bf16 values when w.dtype == "bf16".  Rows of X
    at padded positions hold `pad_value`.  Draw order: lengths, X, Wt."""
    rng = np.random.default_rng((w.seed if seed is None else seed) + 7919)
    nb = w.B if B is None else B
    dx = w.H * w.d
    if lengths is not None:
        lengths = np.asarray(lengths, dtype=np.int32)
        nb = int(lengths.shape[0])
    elif w.ragged is not None:
        lengths = rng.integers(w.ragged[0], w.ragged[1] + 1, size=nb).astype(np.int32)
    else:
        lengths = np.full(nb, w.T, dtype=np.int32)
    X = rng.standard_normal((nb, w.T, dx), dtype=np.float32)
    Wt = rng.standard_normal((3, w.H * w.d, dx), dtype=np.float32) / np.float32(np.sqrt(dx))
    for b in range(nb):
        if int(lengths[b]) < w.T:
            X[b, int(lengths[b]):] = pad_value
    if w.dtype == "bf16":
        X, Wt = round_to_bf16(X), round_to_bf16(Wt)
    return {"X": X, "Wt": Wt, "lengths": lengths}
