"""Float64 oracle of the RoPElite search (Algorithm 1 of the paper, Section 3.1).  TEST
INFRASTRUCTURE ONLY: imported by tests/, by __graft_entry__.smoke() and by bench.py's CPU-baseline
legs; the CUDA library never calls into it and shares no code with it.

For one attention head the search keeps a list e of elite chunks.  In every round it computes the
attention scores with RoPE on all chunks (the model as trained), and, for each chunk j not yet
chosen, the scores with RoPE on e + [j] only (the other chunks enter un-rotated); the chunk whose
scores are closest in L1 distance joins e.  The scores are the pre-softmax products
s_t = q_t K_t^T of Section 2.1, taken at every decoding step t of a calibration sequence: the
pairs (query position m, key position n <= m).

Readings where the paper is silent: positions are 0 .. n-1 (token t at position t); the L1
distance sums over all causal pairs of the sequence; a tie goes to the lowest chunk id.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _theta(d_h: int, base: float) -> np.ndarray:
    return F64(base) ** (-2.0 * np.arange(d_h // 2, dtype=F64) / F64(d_h))     # Section 2.2


def scores_with_rope_on(Q, K, chunks, d_h: int, base: float = 10000.0) -> np.ndarray:
    """S[m][n] = q_m K_n^T with the chunks in `chunks` rotated by their positions (Eq. 1a: chunk
    i of the token at position p turns by p * theta_i) and all other chunks left as they are.
    Q, K: [n][d_h], token t at position t.  Returns the full [n][n] matrix (no mask)."""
    Q = np.asarray(Q, dtype=F64).copy()
    K = np.asarray(K, dtype=F64).copy()
    n = Q.shape[0]
    th = _theta(d_h, base)
    pos = np.arange(n, dtype=F64)
    for i in chunks:
        ang = pos * th[i]
        c, s = np.cos(ang), np.sin(ang)
        for X in (Q, K):
            x0, x1 = X[:, 2 * i].copy(), X[:, 2 * i + 1].copy()
            X[:, 2 * i] = x0 * c - x1 * s
            X[:, 2 * i + 1] = x0 * s + x1 * c
    return Q @ K.T


def distances(Q, K, elite, d_h: int, base: float = 10000.0) -> np.ndarray:
    """One round of Algorithm 1 for one head: distance[j] = || s - s'_j ||_1 over the causal
    pairs, s with RoPE on every chunk, s'_j with RoPE on elite + [j].  Chunks already in `elite`
    get +inf (they are not candidates)."""
    half = d_h // 2
    n = np.asarray(Q).shape[0]
    causal = np.tril(np.ones((n, n), dtype=bool))
    full = scores_with_rope_on(Q, K, range(half), d_h, base)
    out = np.full(half, np.inf, dtype=F64)
    for j in range(half):
        if j in elite:
            continue
        trial = scores_with_rope_on(Q, K, list(elite) + [j], d_h, base)
        out[j] = np.abs(full - trial)[causal].sum()
    return out


def search(Q, K, r: int, d_h: int, base: float = 10000.0):
    """Algorithm 1 for one head: r greedy rounds.  Returns (elite list in the order chosen,
    [r][d_h/2] distances of every round)."""
    elite, trace = [], []
    for _ in range(r):
        d = distances(Q, K, elite, d_h, base)
        trace.append(d)
        elite.append(int(np.argmin(d)))        # first minimum: a tie goes to the lowest chunk id
    return elite, np.stack(trace) if trace else np.zeros((0, d_h // 2))
