"""Pins for the float64 oracle: every check here compares it with something that is NOT the
oracle -- a closed form, an invariant the paper states, an independently written textbook
routine, a library routine on a special case, or brute force on a tiny input."""
import cmath
import math
import os

import numpy as np
import pytest
import scipy.special
import torch

from oracle import elitekv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _random_case(seed, n_h=3, d_h=16, r=3, d_c=10, n=9):
    g = _rng(seed)
    idx = np.stack([g.permutation(d_h // 2)[:r] for _ in range(n_h)]).astype(np.int64)
    q = g.standard_normal((n_h, d_h))
    k_e = g.standard_normal((n, n_h, r, 2))
    c = g.standard_normal((n, d_c))
    W_uk = g.standard_normal((d_c, n_h * (d_h - 2 * r))) / math.sqrt(d_c)
    W_uv = g.standard_normal((d_c, n_h * d_h)) / math.sqrt(d_c)
    pos = np.arange(n)
    return dict(idx=idx, q=q, k_e=k_e, c=c, W_uk=W_uk, W_uv=W_uv, pos=pos, q_pos=n - 1, d_h=d_h)


def _decode_case(z, **kw):
    return O.decode_from_raw(z["q"], z["q_pos"], z["k_e"], z["pos"], z["c"], z["W_uk"], z["W_uv"],
                             z["idx"], z["d_h"], **kw)


# ------------------------------------------------------------------ bf16 rounding
def test_bf16_rounding_matches_library_rounding():
    g = _rng(1)
    x = np.concatenate([g.standard_normal(20000) * 10.0 ** g.integers(-6, 6, 20000),
                        # exact ties and neighbours around them
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8,
                                  -(1.0 + 2.0 ** -8), 255.5, 256.5 * 2, 0.0, -0.0, 3.0 * 2.0 ** -9])])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.f64_to_bf16_bits(x), want)
    # just above a tie: a single rounding goes up (a detour through float32 would land on the
    # tie and round to even, i.e. down) -- 1 + 2^-7 is 0x3F81
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8 + 2.0 ** -30]))[0] == 0x3F81
    assert O.f64_to_bf16_bits(np.array([1.0 + 2.0 ** -8]))[0] == 0x3F80       # tie -> even
    assert O.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 0x3F82   # tie -> even
    x32 = x.astype(np.float32)
    want32 = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.f32_to_bf16_bits(x32), want32)
    back = O.bf16_bits_to_f64(want32)
    assert np.array_equal(back, torch.from_numpy(x32).to(torch.bfloat16).double().numpy())


# ------------------------------------------------------------------ hand-worked example
def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "worked_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, *v = line.split()
            vals[k] = [float(t) for t in v]
    return vals


def test_worked_two_token_example():
    gold = _golden()
    # closed form retyped from the derivation in the fixture's header
    p1 = 1.0 / (1.0 + math.exp(-(1.0 - math.cos(1.0) / 2.0)))
    assert abs(p1 - gold["p1"][0]) < 1e-15
    idx = np.array([[0]])
    q = np.array([[1.0, 0.0, 2.0, -1.0]])
    k_e = np.array([[[[1.0, 0.0]]], [[[0.0, 1.0]]]])
    c = np.array([[1.0, 0.0], [0.0, 2.0]])
    W_uk = np.array([[1.0, 0.0], [0.5, -1.0]])
    W_uv = np.array([[1.0, 2.0, 3.0, 4.0], [0.0, 1.0, 0.0, -1.0]])
    k_rope = O.rotate_elite_keys(k_e, [0, 1], idx, 4)
    assert np.allclose(k_rope[1, 0], [-math.sin(1.0), math.cos(1.0)], atol=1e-15)
    s = O.scores(q, 1, k_rope, c, W_uk, idx, 4)
    assert np.allclose(s[0], [gold["s0"][0], gold["s1"][0]], atol=1e-14)
    o = O.decode(q, 1, k_rope, c, W_uk, W_uv, idx, 4)
    assert np.allclose(o[0], gold["o"], atol=1e-14)
    o2 = O.decode_absorbed(q, 1, k_rope, c, W_uk, W_uv, idx, 4)
    assert np.allclose(o2[0], gold["o"], atol=1e-14)


# ------------------------------------------------------------------ full-RoPE special case
def _textbook_rope_mha(q, q_pos, k, pos, v, base):
    """Independent statement of Eq. 1a with complex numbers: chunk (2i, 2i+1) is the complex
    number x0 + i x1, rotating by an angle is multiplying by exp(i angle); the chunk's score
    contribution is Re(q_hat * conj(k_hat)).  Pure Python loops."""
    n_h, d_h = len(q), len(q[0])
    out = []
    for h in range(n_h):
        s = []
        for t in range(len(k)):
            acc = 0.0
            for i in range(d_h // 2):
                th = base ** (-2.0 * i / d_h)
                qh = complex(q[h][2 * i], q[h][2 * i + 1]) * cmath.exp(1j * q_pos * th)
                kh = complex(k[t][h][2 * i], k[t][h][2 * i + 1]) * cmath.exp(1j * pos[t] * th)
                acc += (qh * kh.conjugate()).real
            s.append(acc / math.sqrt(d_h))
        m = max(s)
        e = [math.exp(x - m) for x in s]
        z = sum(e)
        out.append([sum(e[t] / z * v[t][h][j] for t in range(len(k))) for j in range(d_h)])
    return np.array(out)


def test_all_chunks_elite_is_standard_rope_attention():
    n_h, d_h, n = 2, 8, 6
    g = _rng(7)
    q = g.standard_normal((n_h, d_h))
    k = g.standard_normal((n, n_h, d_h))
    v = g.standard_normal((n, n_h, d_h))
    pos = np.array([3, 4, 5, 9, 10, 17])
    # every chunk elite, in a scrambled per-head order; latent = all heads' values, W_uv = I
    idx = np.stack([g.permutation(d_h // 2) for _ in range(n_h)])
    k_e = np.zeros((n, n_h, d_h // 2, 2))
    for h in range(n_h):
        for j, i in enumerate(idx[h]):
            k_e[:, h, j, 0] = k[:, h, 2 * i]
            k_e[:, h, j, 1] = k[:, h, 2 * i + 1]
    c = v.reshape(n, n_h * d_h)
    W_uk = np.zeros((n_h * d_h, 0))
    W_uv = np.eye(n_h * d_h)
    got = O.decode_from_raw(q, 21, k_e, pos, c, W_uk, W_uv, idx, d_h, base=500.0)
    want = _textbook_rope_mha(q.tolist(), 21, k.tolist(), pos.tolist(), v.tolist(), 500.0)
    assert np.allclose(got, want, atol=1e-12)
    # the comparator's definition agrees too once keys and query are rotated up front
    all_idx = np.tile(np.arange(d_h // 2), (n_h, 1))
    kk = k.reshape(n, n_h, d_h // 2, 2)
    K_hat = O.rotate_elite_keys(kk, pos, all_idx, d_h, 500.0)
    q_hat, _ = O.query_parts(q, 21, all_idx, d_h, 500.0)
    assert np.allclose(O.mha_decode(q_hat, K_hat, v), want, atol=1e-12)


# ------------------------------------------------------------------ RoPElite score equation
def test_score_equation_relative_form_with_partial_rope():
    """Section 3.1's score: elite chunks through R((m-n) theta_i), the others un-rotated.
    Full keys are given; the oracle sees them only through (k_e, c, W_uk) with c holding every
    head's non-elite key dims and W_uk selecting them back.  Pins the gather of elite chunks,
    the ascending order of the remaining dims and the per-head column blocks of W_uk."""
    n_h, d_h, r, n = 3, 12, 2, 5
    g = _rng(11)
    idx = np.stack([g.permutation(d_h // 2)[:r] for _ in range(n_h)])
    q = g.standard_normal((n_h, d_h))
    k = g.standard_normal((n, n_h, d_h))
    pos = np.array([0, 2, 3, 7, 8])
    m, base = 8, 10000.0
    want = np.zeros((n_h, n))
    for h in range(n_h):
        for t in range(n):
            for i in range(d_h // 2):
                q2, k2 = q[h, 2 * i:2 * i + 2], k[t, h, 2 * i:2 * i + 2]
                if i in idx[h]:
                    a = (m - pos[t]) * base ** (-2.0 * i / d_h)
                    R = np.array([[math.cos(a), math.sin(a)], [-math.sin(a), math.cos(a)]])
                    want[h, t] += q2 @ R @ k2
                else:
                    want[h, t] += q2 @ k2
    dn = d_h - 2 * r
    k_e = np.zeros((n, n_h, r, 2))
    c = np.zeros((n, n_h * dn))
    for h in range(n_h):
        rest = [d for d in range(d_h) if d // 2 not in idx[h]]
        c[:, h * dn:(h + 1) * dn] = k[:, h, rest]
        for j, i in enumerate(idx[h]):
            k_e[:, h, j] = k[:, h, 2 * i:2 * i + 2]
    W_uk = np.eye(n_h * dn)
    k_rope = O.rotate_elite_keys(k_e, pos, idx, d_h, base)
    got = O.scores(q, m, k_rope, c, W_uk, idx, d_h, base)
    assert np.allclose(got, want, atol=1e-12)


def test_shift_invariance():
    z = _random_case(3)
    o0 = _decode_case(z)
    z2 = dict(z, pos=z["pos"] + 1234, q_pos=z["q_pos"] + 1234)
    assert np.allclose(_decode_case(z2), o0, atol=1e-9)
    z3 = dict(z, pos=z["pos"] + 5)   # shifting only the keys must change the result
    assert not np.allclose(_decode_case(z3), o0, atol=1e-6)


def test_no_elite_chunks_is_plain_attention_over_up_projected_latent():
    n_h, d_h, d_c, n = 2, 8, 5, 7
    g = _rng(5)
    q = g.standard_normal((n_h, d_h))
    c = g.standard_normal((n, d_c))
    W_uk = g.standard_normal((d_c, n_h * d_h))
    W_uv = g.standard_normal((d_c, n_h * d_h))
    idx = np.zeros((n_h, 0), dtype=np.int64)
    got = O.decode(q, 6, np.zeros((n, n_h, 0)), c, W_uk, W_uv, idx, d_h)
    K = (c @ W_uk).reshape(n, n_h, d_h)
    V = (c @ W_uv).reshape(n, n_h, d_h)
    p = scipy.special.softmax(np.einsum("hd,thd->ht", q, K) / math.sqrt(d_h), axis=1)
    assert np.allclose(got, np.einsum("ht,thd->hd", p, V), atol=1e-12)


def test_absorbed_equals_unabsorbed():
    for seed in (21, 22):
        z = _random_case(seed, n_h=4, d_h=32, r=5, d_c=24, n=33)
        k_rope = O.rotate_elite_keys(z["k_e"], z["pos"], z["idx"], z["d_h"])
        a = O.decode(z["q"], z["q_pos"], k_rope, z["c"], z["W_uk"], z["W_uv"], z["idx"], z["d_h"])
        b = O.decode_absorbed(z["q"], z["q_pos"], k_rope, z["c"], z["W_uk"], z["W_uv"], z["idx"],
                              z["d_h"])
        assert np.allclose(a, b, atol=1e-12)
        sub = O.decode_absorbed(z["q"], z["q_pos"], k_rope, z["c"], z["W_uk"], z["W_uv"], z["idx"],
                                z["d_h"], heads=[2, 0])
        assert np.allclose(sub, a[[2, 0]], atol=1e-12)


def test_softmax_special_cases():
    z = _random_case(9, n=1)
    o = _decode_case(z)
    d_h = z["d_h"]
    for h in range(o.shape[0]):     # one token: o_h = c_0 W_uv,h whatever the score
        assert np.allclose(o[h], z["c"][0] @ z["W_uv"][:, h * d_h:(h + 1) * d_h], atol=1e-13)
    # identical tokens at one position: any softmax is uniform over equal values
    z = _random_case(10, n=6)
    z["k_e"][:] = z["k_e"][0]
    z["c"][:] = z["c"][0]
    z["pos"] = np.full(6, 4)
    o = _decode_case(z)
    for h in range(o.shape[0]):
        assert np.allclose(o[h], z["c"][0] @ z["W_uv"][:, h * d_h:(h + 1) * d_h], atol=1e-12)
    # an extra latent dim equal to 1 for every token shifts all scores of a head by the same
    # amount (whatever its W_uk row) and, with a zero W_uv row, leaves the output unchanged
    z = _random_case(12)
    o0 = _decode_case(z)
    g = _rng(13)
    z2 = dict(z, c=np.concatenate([z["c"], np.ones((z["c"].shape[0], 1))], axis=1),
              W_uk=np.concatenate([z["W_uk"], 50 * g.standard_normal((1, z["W_uk"].shape[1]))]),
              W_uv=np.concatenate([z["W_uv"], np.zeros((1, z["W_uv"].shape[1]))]))
    assert np.allclose(_decode_case(z2), o0, atol=1e-10)
    # empty context
    ze = _random_case(14, n=0)
    assert np.array_equal(_decode_case(ze), np.zeros_like(o0))


def test_scale_and_default_scale():
    z = _random_case(15)
    assert np.allclose(_decode_case(z), _decode_case(z, scale=1.0 / math.sqrt(z["d_h"])), atol=0)
    assert not np.allclose(_decode_case(z), _decode_case(z, scale=1.0), atol=1e-6)


def test_half_split_pairing_is_a_permutation_of_query_dims():
    z = _random_case(16)
    d_h = z["d_h"]
    perm = np.concatenate([np.arange(0, d_h, 2), np.arange(1, d_h, 2)])  # new[i]=old[2i], new[i+d/2]=old[2i+1]
    q_half = z["q"][:, perm]
    a0, _ = O.query_parts(z["q"], 5, z["idx"], d_h, pair_mode=0)
    a1, _ = O.query_parts(q_half, 5, z["idx"], d_h, pair_mode=1)
    assert np.allclose(a0, a1, atol=0)
    # the remaining dims keep ascending order of THEIR OWN layout
    for h in range(z["idx"].shape[0]):
        n1 = O.nope_dims(z["idx"][h], d_h, 1)
        assert np.all(np.diff(n1) > 0) and len(n1) == d_h - 2 * z["idx"].shape[1]


def test_cache_elements_per_token_match_paper_ratios():
    # (2 r n_h + d_c) / (2 n_h d_h): 50 %, 25 %, 12.5 % rows of Table 1 on the 7B shape
    full = 2 * 32 * 128
    assert O.cache_elements_per_token(32, 16, 3072) / full == 0.5
    assert O.cache_elements_per_token(32, 8, 1536) / full == 0.25
    assert O.cache_elements_per_token(32, 4, 768) / full == 0.125
    assert O.cache_elements_per_token(40, 8, 1920) / (2 * 40 * 128) == 0.25
    assert O.cache_elements_per_token(4, 2, 64) == 80


# ------------------------------------------------------------------ append: layout and values
def test_token_slot_against_plain_loops():
    g = _rng(31)
    B, page, max_pages = 5, 8, 6
    perm = g.permutation(B * max_pages)
    table = perm.reshape(B, max_pages)
    for _ in range(200):
        s, p = int(g.integers(B)), int(g.integers(page * max_pages))
        want = int(table[s][p // page]) * page + (p % page)
        assert int(O.token_slot([s], [p], page_table=table, page_size=page)[0]) == want
        assert int(O.token_slot([s], [p], max_ctx=100)[0]) == s * 100 + p


def test_append_expected_places_rows_and_only_those():
    g = _rng(32)
    n_h, r, d_c, d_h = 2, 2, 8, 8
    idx = np.array([[1, 3], [0, 2]])
    page, B = 4, 2
    table = np.array([[5, 0, 3], [1, 4, 2]])
    slots = 6 * page
    rope0 = g.integers(0, 65535, (slots, n_h * 2 * r)).astype(np.uint16)
    lat0 = g.integers(0, 65535, (slots, d_c)).astype(np.uint16)
    k_e = torch.randn(3, n_h, r, 2).to(torch.bfloat16)
    c = torch.randn(3, d_c).to(torch.bfloat16)
    kb = k_e.view(torch.int16).numpy().view(np.uint16)
    cb = c.view(torch.int16).numpy().view(np.uint16)
    seq, pos = [0, 1, 1], [5, 0, 11]
    rope, lat = O.append_expected(rope0, lat0, kb, cb, seq, pos, idx, d_h, page_table=table,
                                  page_size=page)
    where = [0 * page + 1, 1 * page + 0, 2 * page + 3]
    untouched = np.setdiff1d(np.arange(slots), where)
    assert np.array_equal(rope[untouched], rope0[untouched])
    assert np.array_equal(lat[untouched], lat0[untouched])
    assert np.array_equal(lat[where], cb)
    want = O.rotate_elite_keys(k_e.double().numpy(), pos, idx, d_h).reshape(3, -1)
    got = O.bf16_bits_to_f64(rope[where])
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 1e-30)
    # float32 bit model stays within one bf16 ulp of the float64 value
    tab = O.rope_table_f32(16, d_h)
    rope_b, _ = O.append_expected(rope0, lat0, kb, cb, seq, pos, idx, d_h, page_table=table,
                                  page_size=page, table32=tab)
    diff = np.abs(rope_b[where].astype(np.int32) - rope[where].astype(np.int32))
    assert diff.max() <= 1


def test_rotation_preserves_norm_and_composes():
    g = _rng(33)
    x0, x1 = g.standard_normal(50), g.standard_normal(50)
    a, b = g.standard_normal(50) * 10, g.standard_normal(50) * 10
    y0, y1 = O.rotate(x0, x1, a)
    assert np.allclose(y0 ** 2 + y1 ** 2, x0 ** 2 + x1 ** 2, atol=1e-12)
    z0, z1 = O.rotate(y0, y1, b)
    w0, w1 = O.rotate(x0, x1, a + b)
    assert np.allclose(z0, w0, atol=1e-12) and np.allclose(z1, w1, atol=1e-12)
    # quarter turn of (1, 0) is (0, 1) under the row-vector convention
    q0, q1 = O.rotate(np.array(1.0), np.array(0.0), math.pi / 2)
    assert abs(q0) < 1e-15 and abs(q1 - 1) < 1e-15


def test_theta_schedule():
    th = O.rope_theta(128, 10000.0)
    assert th[0] == 1.0 and np.all(np.diff(th) < 0)
    assert abs(th[32] - 10000.0 ** -0.5) < 1e-15
    assert abs(th[63] - 10000.0 ** (-126 / 128)) < 1e-18


def test_projection_with_selector_weights_reduces_to_the_plain_append():
    """Fused projection + append (Section 3.2 projections, Section 3.1 rotation).  With weights
    that merely SELECT coordinates of x (W^k_e and A^kv columns of the identity) the projection is
    exact, so the fused result must equal, bit for bit, the plain append of those coordinates,
    which is pinned on its own above; a swapped weight, a transposed product or a rotation applied
    to the latent part would all break the equality."""
    g = np.random.default_rng(31)
    n_h, d_h, r, d_c = 3, 16, 2, 8
    rope_w = n_h * 2 * r
    d = rope_w + d_c + 5                       # five hidden coordinates feed nothing
    idx = np.stack([g.permutation(d_h // 2)[:r] for _ in range(n_h)])
    T = 9
    xb = O.f64_to_bf16_bits(g.standard_normal((T, d)))
    x = O.bf16_bits_to_f64(xb)
    perm = g.permutation(d)
    W_ke = np.zeros((d, rope_w)); W_ke[perm[:rope_w], np.arange(rope_w)] = 1.0
    W_down = np.zeros((d, d_c)); W_down[perm[rope_w:rope_w + d_c], np.arange(d_c)] = 1.0
    seq = g.integers(0, 2, T); pos = g.permutation(20)[:T]
    rope0 = g.integers(0, 2 ** 15, (40, rope_w)).astype(np.uint16)
    lat0 = g.integers(0, 2 ** 15, (40, d_c)).astype(np.uint16)
    got_r, got_l, rows, c = O.project_append_expected(rope0, lat0, x, W_ke, W_down, seq, pos, idx, d_h, max_ctx=20)
    k_bits = xb[:, perm[:rope_w]].reshape(T, n_h, r, 2)
    c_bits = xb[:, perm[rope_w:rope_w + d_c]]
    want_r, want_l = O.append_expected(rope0, lat0, k_bits, c_bits, seq, pos, idx, d_h, max_ctx=20)
    assert np.array_equal(got_r, want_r) and np.array_equal(got_l, want_l)


def test_projection_properties_that_need_no_second_implementation():
    """Linearity in x before rounding; a token at position 0 is stored un-rotated; rotation keeps
    the norm of every projected pair; the latent part ignores the position."""
    g = np.random.default_rng(32)
    n_h, d_h, r, d_c, d, T = 2, 8, 2, 4, 6, 5
    idx = np.array([[0, 3], [2, 1]])
    W_ke = g.standard_normal((d, n_h * 2 * r)); W_down = g.standard_normal((d, d_c))
    x1, x2 = g.standard_normal((T, d)), g.standard_normal((T, d))
    seq = np.zeros(T, dtype=np.int64); pos = np.array([0, 3, 7, 1, 5])
    z = np.zeros((8, n_h * 2 * r), dtype=np.uint16), np.zeros((8, d_c), dtype=np.uint16)
    _, _, r1, c1 = O.project_append_expected(*z, x1, W_ke, W_down, seq, pos, idx, d_h, max_ctx=8)
    _, _, r2, c2 = O.project_append_expected(*z, x2, W_ke, W_down, seq, pos, idx, d_h, max_ctx=8)
    _, _, r3, c3 = O.project_append_expected(*z, 2 * x1 - 3 * x2, W_ke, W_down, seq, pos, idx, d_h, max_ctx=8)
    assert np.allclose(r3, 2 * r1 - 3 * r2, atol=1e-12) and np.allclose(c3, 2 * c1 - 3 * c2, atol=1e-12)
    # hand-evaluated entries: token 0 sits at position 0 (identity rotation)
    for col in range(n_h * 2 * r):
        assert abs(r1[0, col] - sum(x1[0, k] * W_ke[k, col] for k in range(d))) < 1e-12
    for col in range(d_c):
        assert abs(c1[2, col] - sum(x1[2, k] * W_down[k, col] for k in range(d))) < 1e-12
    # norms of pairs survive the rotation; other positions change the rope row, not the latent
    k_plain = (x1 @ W_ke).reshape(T, n_h * r, 2)
    assert np.allclose(np.linalg.norm(r1.reshape(T, n_h * r, 2), axis=-1), np.linalg.norm(k_plain, axis=-1))
    _, _, r4, c4 = O.project_append_expected(*z, x1, W_ke, W_down, seq, (pos + 2) % 8, idx, d_h, max_ctx=8)
    assert np.allclose(c4, c1) and not np.allclose(r4[1:], r1[1:])
    # quarter turn: theta_0 = 1, so position p = pi/2 cannot be hit by an integer; use the angle law
    # instead: rotating by positions 3 and then reading the pair's angle gives atan2 shifted by 3*theta
    th = O.rope_theta(d_h)[idx.reshape(-1)]
    a_plain = np.arctan2(k_plain[1, :, 1], k_plain[1, :, 0])
    a_rot = np.arctan2(r1.reshape(T, n_h * r, 2)[1, :, 1], r1.reshape(T, n_h * r, 2)[1, :, 0])
    assert np.allclose(np.exp(1j * (a_rot - a_plain)), np.exp(1j * 3 * th))


# ------------------------------------------------------------------ separated latents (S-LRD)
def _slrd_case(seed, n_h=3, d_h=12, r=2, d_ck=7, d_cv=5, n=8):
    g = _rng(seed)
    dn = d_h - 2 * r
    return dict(
        idx=np.stack([g.permutation(d_h // 2)[:r] for _ in range(n_h)]).astype(np.int64),
        q=g.standard_normal((n_h, d_h)), k_e=g.standard_normal((n, n_h, r, 2)),
        c_k=g.standard_normal((n, d_ck)), c_v=g.standard_normal((n, d_cv)),
        W_uk=g.standard_normal((d_ck, n_h * dn)), W_uv=g.standard_normal((d_cv, n_h * d_h)),
        pos=np.sort(g.choice(40, n, replace=False)), q_pos=41, d_h=d_h, n_h=n_h, r=r, dn=dn, n=n)


def test_slrd_is_textbook_rope_attention_on_the_reconstructed_keys_and_values():
    """Section 3.2 (S-LRD): keys of a head = its elite chunks as cached plus c_k . B^k_S,h on the
    other dims (un-rotated), values = c_v . B^v_S,h.  Rebuild full K and V by hand and run the
    complex-number textbook attention with RoPE on the elite chunks only (the others get the
    identity rotation: their positions are set to the query's, so the relative angle is zero)."""
    z = _slrd_case(31)
    n, n_h, d_h, r, dn = z["n"], z["n_h"], z["d_h"], z["r"], z["dn"]
    k_rope = O.rotate_elite_keys(z["k_e"], z["pos"], z["idx"], d_h, 777.0)
    got = O.decode_slrd(z["q"], z["q_pos"], k_rope, z["c_k"], z["c_v"], z["W_uk"], z["W_uv"], z["idx"], d_h,
                        base=777.0)
    want = np.zeros((n_h, d_h))
    for h in range(n_h):
        elite = [int(i) for i in z["idx"][h]]
        rest = [d for d in range(d_h) if d // 2 not in elite]
        Kn = z["c_k"] @ z["W_uk"][:, h * dn:(h + 1) * dn]
        V = z["c_v"] @ z["W_uv"][:, h * d_h:(h + 1) * d_h]
        s = []
        for t in range(n):
            acc = 0.0
            for j, i in enumerate(elite):
                th = 777.0 ** (-2.0 * i / d_h)
                qh = complex(z["q"][h][2 * i], z["q"][h][2 * i + 1]) * cmath.exp(1j * z["q_pos"] * th)
                kh = complex(z["k_e"][t][h][j][0], z["k_e"][t][h][j][1]) * cmath.exp(1j * z["pos"][t] * th)
                acc += (qh * kh.conjugate()).real
            for a, d in enumerate(rest):
                acc += z["q"][h][d] * Kn[t][a]
            s.append(acc / math.sqrt(d_h))
        p = scipy.special.softmax(np.array(s))
        want[h] = p @ V
    assert np.allclose(got, want, atol=1e-12)
    # a head subset, in the order asked for
    sub = O.decode_slrd(z["q"], z["q_pos"], k_rope, z["c_k"], z["c_v"], z["W_uk"], z["W_uv"], z["idx"], d_h,
                        base=777.0, heads=[2, 0])
    assert np.allclose(sub, want[[2, 0]], atol=1e-12)


def test_slrd_equals_the_joint_form_with_block_diagonal_up_projections():
    """[c_k | c_v] with B^kv = diag(B^k_S, B^v_S) is a joint latent whose key half ignores c_v and
    whose value half ignores c_k: the joint oracle on the stacked latent must agree.  Swapping
    the two latents, or the two weights, breaks it."""
    z = _slrd_case(32, d_ck=6, d_cv=9)
    d_h = z["d_h"]
    k_rope = O.rotate_elite_keys(z["k_e"], z["pos"], z["idx"], d_h)
    got = O.decode_slrd(z["q"], z["q_pos"], k_rope, z["c_k"], z["c_v"], z["W_uk"], z["W_uv"], z["idx"], d_h)
    c = np.concatenate([z["c_k"], z["c_v"]], axis=1)
    W_uk = np.concatenate([z["W_uk"], np.zeros((9, z["W_uk"].shape[1]))], axis=0)
    W_uv = np.concatenate([np.zeros((6, z["W_uv"].shape[1])), z["W_uv"]], axis=0)
    want = O.decode(z["q"], z["q_pos"], k_rope, c, W_uk, W_uv, z["idx"], d_h)
    assert np.allclose(got, want, atol=1e-12)
    # equal latents and one shared pair of weights: S-LRD with c_k = c_v = c is J-LRD
    z2 = _random_case(33)
    k2 = O.rotate_elite_keys(z2["k_e"], z2["pos"], z2["idx"], z2["d_h"])
    a = O.decode_slrd(z2["q"], z2["q_pos"], k2, z2["c"], z2["c"], z2["W_uk"], z2["W_uv"], z2["idx"], z2["d_h"])
    b = O.decode(z2["q"], z2["q_pos"], k2, z2["c"], z2["W_uk"], z2["W_uv"], z2["idx"], z2["d_h"])
    assert np.allclose(a, b, atol=1e-12)


def test_slrd_special_cases_and_cache_size():
    z = _slrd_case(34)
    d_h = z["d_h"]
    k_rope = O.rotate_elite_keys(z["k_e"], z["pos"], z["idx"], d_h)
    # one cached token: the output is that token's value, whatever the scores
    one = O.decode_slrd(z["q"], 5, k_rope[:1], z["c_k"][:1], z["c_v"][:1], z["W_uk"], z["W_uv"], z["idx"], d_h)
    assert np.allclose(one, (z["c_v"][0] @ z["W_uv"]).reshape(z["n_h"], d_h), atol=1e-12)
    # zero query: uniform attention, the mean of the values
    flat = O.decode_slrd(np.zeros_like(z["q"]), 5, k_rope, z["c_k"], z["c_v"], z["W_uk"], z["W_uv"], z["idx"], d_h)
    assert np.allclose(flat, (z["c_v"].mean(axis=0) @ z["W_uv"]).reshape(z["n_h"], d_h), atol=1e-12)
    # empty cache
    none = O.decode_slrd(z["q"], 0, k_rope[:0], z["c_k"][:0], z["c_v"][:0], z["W_uk"], z["W_uv"], z["idx"], d_h)
    assert none.shape == (z["n_h"], d_h) and not none.any()
    # cache elements per token (Section 3.2): 2 r n_h + d_ck + d_cv; with d_ck + d_cv = d_c it is the
    # joint count
    assert O.cache_elements_per_token_slrd(32, 8, 512, 1024) == 2 * 8 * 32 + 512 + 1024
    assert O.cache_elements_per_token_slrd(32, 8, 512, 1024) == O.cache_elements_per_token(32, 8, 1536)


# ------------------------------------------------------------------ several query rows, causal
def test_causal_rows_match_the_library_attention_when_every_chunk_is_elite():
    """Every chunk elite, latent = all heads' values, W_uv = I: the method is standard causal
    RoPE attention.  Queries and keys are rotated here with complex arithmetic and handed to
    torch's scaled_dot_product_attention (square causal mask: a prefill of n tokens)."""
    n_h, d_h, n = 2, 8, 7
    g = _rng(41)
    q = g.standard_normal((n, n_h, d_h))
    k = g.standard_normal((n, n_h, d_h))
    v = g.standard_normal((n, n_h, d_h))
    pos = np.arange(n)
    idx = np.stack([g.permutation(d_h // 2) for _ in range(n_h)])
    k_e = np.zeros((n, n_h, d_h // 2, 2))
    for h in range(n_h):
        for j, i in enumerate(idx[h]):
            k_e[:, h, j, 0] = k[:, h, 2 * i]
            k_e[:, h, j, 1] = k[:, h, 2 * i + 1]
    k_rope = O.rotate_elite_keys(k_e, pos, idx, d_h, 300.0)
    got = O.attend_causal(q, pos, k_rope, pos, v.reshape(n, n_h * d_h), np.zeros((n_h * d_h, 0)),
                          np.eye(n_h * d_h), idx, d_h, base=300.0)

    def rot(x):      # [n][n_h][d_h] rotated at its own position, chunk (2i, 2i+1) as a complex number
        z = x[..., 0::2] + 1j * x[..., 1::2]
        th = 300.0 ** (-2.0 * np.arange(d_h // 2) / d_h)
        z = z * np.exp(1j * pos[:, None, None] * th[None, None, :])
        y = np.empty_like(x)
        y[..., 0::2], y[..., 1::2] = z.real, z.imag
        return y
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2) for a in (rot(q), rot(k), v))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True).permute(1, 0, 2).numpy()
    assert np.allclose(got, want, atol=1e-12)


def test_causal_rows_are_single_query_decodes_over_their_prefixes():
    """Row i equals the one-query definition on the tokens it may see; key positions need not be
    sorted or contiguous; a row before every key is zero; with one row and everything visible it
    is `decode` itself."""
    z = _random_case(42, n=11)
    d_h = z["d_h"]
    key_pos = np.array([4, 0, 9, 2, 7, 5, 1, 8, 3, 6, 12])
    k_rope = O.rotate_elite_keys(z["k_e"], key_pos, z["idx"], d_h)
    g = _rng(43)
    q = g.standard_normal((4, 3, d_h))
    q_pos = np.array([5, 9, 12, -1])
    got = O.attend_causal(q, q_pos, k_rope, key_pos, z["c"], z["W_uk"], z["W_uv"], z["idx"], d_h)
    for i in range(3):
        seen = key_pos <= q_pos[i]
        want = O.decode(q[i], int(q_pos[i]), k_rope[seen], z["c"][seen], z["W_uk"], z["W_uv"], z["idx"], d_h)
        assert np.allclose(got[i], want, atol=1e-12)
    assert not got[3].any()
    assert int((key_pos <= 5).sum()) == 6 and int((key_pos <= 9).sum()) == 10     # the masks differ
    assert not np.allclose(got[0], got[1])
    sub = O.attend_causal(q, q_pos, k_rope, key_pos, z["c"], z["W_uk"], z["W_uv"], z["idx"], d_h, heads=[2])
    assert np.allclose(sub[:, 0], got[:, 2], atol=1e-12)
