"""Pins for the RoPElite search oracle (Algorithm 1): comparisons with things that are not the
oracle -- brute force with complex arithmetic on a tiny input, closed forms, invariants."""
import cmath

import numpy as np

from oracle import ropelite_oracle as R


def _brute_distance(Q, K, elite, j, d_h, base):
    """Pure-Python loops: pair by pair, chunk by chunk, complex rotation."""
    n, half = len(Q), d_h // 2
    keep = set(elite) | {j}
    total = 0.0
    for m in range(n):
        for t in range(m + 1):
            full = trial = 0.0
            for i in range(half):
                th = base ** (-2.0 * i / d_h)
                q = complex(Q[m][2 * i], Q[m][2 * i + 1])
                k = complex(K[t][2 * i], K[t][2 * i + 1])
                rot = (q * cmath.exp(1j * m * th) * (k * cmath.exp(1j * t * th)).conjugate()).real
                plain = (q * k.conjugate()).real
                full += rot
                trial += rot if i in keep else plain
            total += abs(full - trial)
    return total


def test_distances_against_brute_force():
    g = np.random.default_rng(3)
    d_h, n = 8, 6
    Q, K = g.standard_normal((n, d_h)), g.standard_normal((n, d_h))
    for elite in ([], [2], [3, 0]):
        got = R.distances(Q, K, elite, d_h, base=50.0)
        for j in range(d_h // 2):
            if j in elite:
                assert np.isinf(got[j])
            else:
                assert abs(got[j] - _brute_distance(Q.tolist(), K.tolist(), elite, j, d_h, 50.0)) < 1e-10


def test_closed_forms():
    g = np.random.default_rng(4)
    d_h, n = 12, 9
    Q, K = g.standard_normal((n, d_h)), g.standard_normal((n, d_h))
    half = d_h // 2
    # every chunk but one already elite: adding the last one reproduces the full scores exactly
    d = R.distances(Q, K, [0, 1, 2, 4, 5], d_h)
    assert abs(d[3]) < 1e-10 and np.isinf(d[[0, 1, 2, 4, 5]]).all()
    # a single token: every relative angle is zero, rotation changes nothing
    assert np.allclose(R.distances(Q[:1], K[:1], [], d_h), 0.0, atol=1e-12)
    # energy in one chunk only: that chunk alone explains the scores, the others explain nothing
    Q1, K1 = np.zeros_like(Q), np.zeros_like(K)
    Q1[:, 6:8], K1[:, 6:8] = Q[:, 6:8], K[:, 6:8]
    d = R.distances(Q1, K1, [], d_h)
    assert abs(d[3]) < 1e-10
    others = [j for j in range(half) if j != 3]
    assert np.allclose(d[others], d[others][0]) and d[others][0] > 1e-3
    # ... and that common value is the L1 norm of (rotated - plain) scores of chunk 3, by hand
    th = 10000.0 ** (-2.0 * 3 / d_h)
    want = 0.0
    for m in range(n):
        for t in range(m + 1):
            a = Q[m, 6] * K[t, 6] + Q[m, 7] * K[t, 7]
            b = Q[m, 7] * K[t, 6] - Q[m, 6] * K[t, 7]
            ph = (m - t) * th
            want += abs(a * (np.cos(ph) - 1.0) - b * np.sin(ph))
    assert abs(d[others][0] - want) < 1e-10
    # scaling queries scales every distance
    assert np.allclose(R.distances(3.0 * Q, K, [1], d_h)[[0, 2, 3, 4, 5]], 3.0 * R.distances(Q, K, [1], d_h)[[0, 2, 3, 4, 5]])


def test_search_picks_dominant_chunks_in_order_and_breaks_ties_low():
    """Chunk energies graded by factors of 10 and scrambled: the greedy rounds must pick the
    chunks in the order of their energy (removing the dominant remaining term always wins)."""
    g = np.random.default_rng(5)
    d_h, n, half = 16, 24, 8
    order = [5, 2, 7, 0, 3, 6, 1, 4]
    Q, K = g.standard_normal((n, d_h)), g.standard_normal((n, d_h))
    for rank, i in enumerate(order):
        Q[:, 2 * i:2 * i + 2] *= 10.0 ** (-rank)
    elite, trace = R.search(Q, K, 5, d_h, base=100.0)
    assert elite == order[:5]
    assert trace.shape == (5, half)
    assert np.isinf(trace[3][[5, 2, 7]]).all() and np.isfinite(trace[3][[0, 3, 6, 1, 4]]).all()
    # the distance of the chosen chunk shrinks round by round here (each round removes the dominant term)
    chosen = [trace[k][elite[k]] for k in range(5)]
    assert all(chosen[k + 1] < chosen[k] for k in range(4))
    # all-zero activations: every distance is 0, ties go to the lowest free chunk id
    z = np.zeros((4, d_h))
    assert R.search(z, z, 3, d_h)[0] == [0, 1, 2]


def test_scores_with_full_rope_depend_on_relative_position_only():
    """Eq. 1a = Eq. 1b: with RoPE on every chunk, S[m][n] is a function of m - n for fixed vectors."""
    g = np.random.default_rng(6)
    d_h, n = 8, 7
    q, k = g.standard_normal(d_h), g.standard_normal(d_h)
    S = R.scores_with_rope_on(np.tile(q, (n, 1)), np.tile(k, (n, 1)), range(4), d_h, base=30.0)
    for d in range(-3, 4):
        diag = np.diagonal(S, offset=-d)
        assert np.allclose(diag, diag[0], atol=1e-12)
    # no chunk rotated: the plain product
    assert np.allclose(R.scores_with_rope_on(np.tile(q, (n, 1)), np.tile(k, (n, 1)), [], d_h), q @ k)
