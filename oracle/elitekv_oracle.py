"""Float64 CPU oracle for EliteKV decode attention (arXiv 2503.01586).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, obviously-correct statement of what
the CUDA library must compute.  It is imported by the test-suite, by the smoke check and by the
CPU-baseline leg of the benchmark, and by nothing else; the CUDA path neither imports it nor
shares any code, table or constant with it.

Everything is numpy float64 and follows the paper's order of operations without absorption,
tiling, splitting or fusion:

  * RoPE (Section 2.2, Eq. 1a): each head's key/query dims are grouped in 2-D chunks
    [2i : 2i+1]; chunk i of the token at position m is multiplied by the rotation R(m*theta_i).
  * RoPElite (Section 3.1, score equation after Algorithm 1): only the chunks of the head's
    elite set I_r^e are rotated; the others enter the score un-rotated.
  * J-LRD (Section 3.2): the un-rotated key dims of all heads and the values of all heads are
    up-projected from one shared latent c = x A^kv, with B^kv = [B^k_J, B^v_J].
  * Attention (Section 2.1): s = q K^T, p = softmax(s / sqrt(d_h)), o = p V.
  * Absorption (Section 5, "SVD for KV Cache Compression"): B^k and B^v can be folded into the
    neighbouring products; `decode_absorbed` is that re-association in float64 and is checked
    against `decode` by the tests.

Readings of points the paper leaves open (each is also listed in the design notes):
  theta_i = base**(-2i/d_h) with base 10000; R(a) acts on a row pair as
  (x0, x1) -> (x0 cos a - x1 sin a, x0 sin a + x1 cos a); the un-rotated ("nope") dims of a head
  are the remaining dims in ascending original index; the softmax scale stays 1/sqrt(d_h) with
  the full d_h; the query attends to its own (just appended) token; an empty context gives zeros.

Shapes (n_h heads, d_h head dim, r elite chunks per head, d_c latent width, n cached tokens):
  idx   int   [n_h][r]            elite chunk ids, distinct per head, each in [0, d_h/2)
  q     f64   [n_h][d_h]          un-rotated query of the decoding token
  k_e   f64   [n][n_h][r][2]      un-rotated elite key chunks, in the order of idx[h]
  c     f64   [n][d_c]            shared latent
  W_uk  f64   [d_c][n_h*(d_h-2r)] B^k_J, head h owns columns [h*(d_h-2r), (h+1)*(d_h-2r))
  W_uv  f64   [d_c][n_h*d_h]      B^v_J, head h owns columns [h*d_h, (h+1)*d_h)
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------------------------
# RoPE (Section 2.2)
# --------------------------------------------------------------------------------------------
def rope_theta(d_h: int, base: float = 10000.0) -> np.ndarray:
    """theta_i for the d_h/2 chunks of Section 2.2; chunk 0 is the highest frequency
    (Figure 2's caption: chunk numbers grow from high to low frequency)."""
    i = np.arange(d_h // 2, dtype=F64)
    return F64(base) ** (-2.0 * i / F64(d_h))


def rotate(x0, x1, angle):
    """Row pair (x0, x1) times the 2-D rotation matrix R(angle) of Eq. 1a."""
    c, s = np.cos(angle), np.sin(angle)
    return x0 * c - x1 * s, x0 * s + x1 * c


def chunk_dims(i, d_h: int, pair_mode: int = 0):
    """The two head dims that form chunk i.  pair_mode 0 is the paper's I = {[2i : 2i+1]};
    pair_mode 1 is the half-split pairing (i, i + d_h/2) used by some checkpoints."""
    i = np.asarray(i)
    if pair_mode == 0:
        return 2 * i, 2 * i + 1
    return i, i + d_h // 2


def nope_dims(idx_h, d_h: int, pair_mode: int = 0) -> np.ndarray:
    """Dims of one head that are NOT in its elite chunks, ascending (the columns of
    W^k_{e-hat,h}, Section 3.2)."""
    a, b = chunk_dims(np.asarray(idx_h, dtype=np.int64), d_h, pair_mode)
    taken = set(a.tolist()) | set(b.tolist())
    return np.array([d for d in range(d_h) if d not in taken], dtype=np.int64)


def rope_table_f32(max_pos: int, d_h: int, base: float = 10000.0) -> np.ndarray:
    """(cos, sin) of pos*theta_i evaluated in float64 and rounded once to float32:
    [max_pos][d_h/2][2].  A caller may hand such a table to the library, which makes the
    append reproducible bit for bit by `rotate_bits_f32`."""
    ang = np.arange(max_pos, dtype=F64)[:, None] * rope_theta(d_h, base)[None, :]
    return np.stack([np.cos(ang), np.sin(ang)], axis=-1).astype(np.float32)


# --------------------------------------------------------------------------------------------
# bf16 rounding (storage format of the cache; round-to-nearest-even)
# --------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern (uint16), round to nearest, ties to even.  Finite inputs."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = u + np.uint64(0x7FFF) + lsb
    return (u >> np.uint64(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(F64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bit pattern with ONE rounding (nearest even), for finite inputs whose
    magnitude is in bf16's normal range or zero.  Works on the float64 bit pattern: bf16 keeps
    the sign, 8 exponent bits and 7 fraction bits; float64 has 52 fraction bits, so 45 are
    dropped."""
    x = np.ascontiguousarray(x, dtype=F64)
    u = x.view(np.uint64)
    sign = (u >> np.uint64(63)).astype(np.uint16) << np.uint16(15)
    mag = u & np.uint64(0x7FFFFFFFFFFFFFFF)
    drop = np.uint64(45)
    lsb = (mag >> drop) & np.uint64(1)
    mag = (mag + ((np.uint64(1) << np.uint64(44)) - np.uint64(1)) + lsb) >> drop
    # mag is now (float64 biased exponent << 7 | 7 fraction bits); re-bias 1023 -> 127.
    rebias = np.uint64((1023 - 127) << 7)
    zero = mag < rebias  # underflows to zero (subnormal bf16 not needed here)
    out = np.where(zero, np.uint64(0), mag - rebias).astype(np.uint16)
    return (out | sign).astype(np.uint16)


# --------------------------------------------------------------------------------------------
# Cache append (Section 3.1, "at the t-th decoding step ... are incorporated into the KV cache")
# --------------------------------------------------------------------------------------------
def token_slot(seq_id, pos, *, max_ctx=None, page_table=None, page_size=64):
    """Index of the cache row (in units of tokens) that holds token `pos` of sequence `seq_id`.
    Contiguous cache: seq*max_ctx + pos.  Paged cache: page_table[seq][pos // page_size] *
    page_size + pos % page_size."""
    seq_id = np.asarray(seq_id, dtype=np.int64)
    pos = np.asarray(pos, dtype=np.int64)
    if page_table is None:
        return seq_id * np.int64(max_ctx) + pos
    pt = np.asarray(page_table, dtype=np.int64)
    return pt[seq_id, pos // page_size] * np.int64(page_size) + pos % page_size


def rotate_elite_keys(k_e, pos, idx, d_h, base=10000.0):
    """k_e [T][n_h][r][2] (un-rotated) at positions pos[T] -> rotated rows [T][n_h][2r]:
    chunk j of head h is multiplied by R(pos * theta_{idx[h][j]}) (Eq. 1a, right factor)."""
    k_e = np.asarray(k_e, dtype=F64)
    T, n_h, r, _ = k_e.shape
    theta = rope_theta(d_h, base)[np.asarray(idx, dtype=np.int64)]  # [n_h][r]
    ang = np.asarray(pos, dtype=F64)[:, None, None] * theta[None, :, :]
    y0, y1 = rotate(k_e[..., 0], k_e[..., 1], ang)
    return np.stack([y0, y1], axis=-1).reshape(T, n_h, 2 * r)


def rotate_bits_f32(x0, x1, cos32, sin32):
    """The append's arithmetic in float32 with every product and sum rounded separately
    (no fused multiply-add): y0 = x0*c - x1*s, y1 = x0*s + x1*c, then bf16 (nearest even).
    With a caller-supplied float32 (cos, sin) table the library must produce these bits."""
    x0 = np.asarray(x0, dtype=np.float32)
    x1 = np.asarray(x1, dtype=np.float32)
    c = np.asarray(cos32, dtype=np.float32)
    s = np.asarray(sin32, dtype=np.float32)
    y0 = (x0 * c).astype(np.float32) - (x1 * s).astype(np.float32)
    y1 = (x0 * s).astype(np.float32) + (x1 * c).astype(np.float32)
    return f32_to_bf16_bits(y0.astype(np.float32)), f32_to_bf16_bits(y1.astype(np.float32))


def append_expected(rope_plane_bits, latent_plane_bits, k_e_bits, c_bits, seq_id, pos, idx, d_h,
                    *, base=10000.0, max_ctx=None, page_table=None, page_size=64, table32=None):
    """Apply one append to copies of the cache planes (uint16 bf16 bit patterns, shaped
    [slots][n_h*2r] and [slots][d_c]) and return them.  Rotated values are float64-exact
    rounded once to bf16, or the float32 bit model when `table32` is given.  Latent rows are
    copied bit for bit."""
    rope = np.array(rope_plane_bits, dtype=np.uint16, copy=True)
    lat = np.array(latent_plane_bits, dtype=np.uint16, copy=True)
    k_e_bits = np.asarray(k_e_bits, dtype=np.uint16)
    T, n_h, r, _ = k_e_bits.shape
    slot = token_slot(seq_id, pos, max_ctx=max_ctx, page_table=page_table, page_size=page_size)
    if table32 is None:
        rows = f64_to_bf16_bits(rotate_elite_keys(bf16_bits_to_f64(k_e_bits), pos, idx, d_h, base))
    else:
        x = bf16_bits_to_f64(k_e_bits).astype(np.float32)
        cs = np.asarray(table32)[np.asarray(pos, dtype=np.int64)][:, np.asarray(idx, dtype=np.int64), :]
        b0, b1 = rotate_bits_f32(x[..., 0], x[..., 1], cs[..., 0], cs[..., 1])
        rows = np.stack([b0, b1], axis=-1).reshape(T, n_h * 2 * r)
    rope[slot] = rows.reshape(T, -1)
    lat[slot] = np.asarray(c_bits, dtype=np.uint16).reshape(T, -1)
    return rope, lat


def project_tokens(x, W_ke, W_down):
    """The projections that feed the cache (Section 3.2): for hidden states x [T][d],
    k_e = x W^k_e  (W^k_e [d][n_h*2r]: the columns of W^k that belong to the elite chunks, head
    by head, Eq. 2) and c = x A^kv (A^kv = W_down [d][d_c]).  Returns float64
    (k_e [T][n_h*2r], c [T][d_c]), not rounded."""
    x = np.asarray(x, dtype=F64)
    return x @ np.asarray(W_ke, dtype=F64), x @ np.asarray(W_down, dtype=F64)


def project_append_expected(rope_plane_bits, latent_plane_bits, x, W_ke, W_down, seq_id, pos, idx,
                            d_h, *, base=10000.0, max_ctx=None, page_table=None, page_size=64):
    """Projection fused with the append: the float64 projections of `project_tokens`, the elite
    chunks rotated at the token's position (Section 3.1), every stored element rounded ONCE to
    bf16.  Returns copies of the planes (uint16 bit patterns) plus the float64 rows before
    rounding (rope rows [T][n_h*2r], latent rows [T][d_c]) for tolerance checks."""
    rope = np.array(rope_plane_bits, dtype=np.uint16, copy=True)
    lat = np.array(latent_plane_bits, dtype=np.uint16, copy=True)
    idx = np.asarray(idx, dtype=np.int64)
    n_h, r = idx.shape
    k_e, c = project_tokens(x, W_ke, W_down)
    T = k_e.shape[0]
    rows = rotate_elite_keys(k_e.reshape(T, n_h, r, 2), pos, idx, d_h, base).reshape(T, n_h * 2 * r)
    slot = token_slot(seq_id, pos, max_ctx=max_ctx, page_table=page_table, page_size=page_size)
    rope[slot] = f64_to_bf16_bits(rows)
    lat[slot] = f64_to_bf16_bits(c)
    return rope, lat, rows, c


# --------------------------------------------------------------------------------------------
# Query side
# --------------------------------------------------------------------------------------------
def query_parts(q, q_pos, idx, d_h, base=10000.0, pair_mode=0):
    """Split one token's query q [n_h][d_h] into q_rope [n_h][2r] (elite chunks rotated at
    q_pos, Eq. 1a left factor) and q_nope [n_h][d_h-2r] (remaining dims, ascending)."""
    q = np.asarray(q, dtype=F64)
    idx = np.asarray(idx, dtype=np.int64)
    n_h, r = idx.shape
    theta = rope_theta(d_h, base)
    q_rope = np.zeros((n_h, 2 * r), dtype=F64)
    q_nope = np.zeros((n_h, d_h - 2 * r), dtype=F64)
    for h in range(n_h):
        a, b = chunk_dims(idx[h], d_h, pair_mode)
        y0, y1 = rotate(q[h, a], q[h, b], F64(q_pos) * theta[idx[h]])
        q_rope[h, 0::2] = y0
        q_rope[h, 1::2] = y1
        q_nope[h] = q[h, nope_dims(idx[h], d_h, pair_mode)]
    return q_rope, q_nope


def absorb_query(q, q_pos, idx, W_uk, d_h, base=10000.0, pair_mode=0):
    """q_rope as above and q_abs[h] = q_nope[h] . W_uk,h^T in R^{d_c} (Section 5: B^k folded
    into the query side)."""
    W_uk = np.asarray(W_uk, dtype=F64)
    q_rope, q_nope = query_parts(q, q_pos, idx, d_h, base, pair_mode)
    n_h, dn = q_nope.shape
    q_abs = np.stack([W_uk[:, h * dn:(h + 1) * dn] @ q_nope[h] for h in range(n_h)])
    return q_rope, q_abs


# --------------------------------------------------------------------------------------------
# Decode attention, un-absorbed (the definition)
# --------------------------------------------------------------------------------------------
def scores(q, q_pos, k_rope, c, W_uk, idx, d_h, base=10000.0, pair_mode=0, heads=None):
    """Pre-softmax scores s[h][t] (not yet scaled) of the RoPElite score equation:
    rotated-elite part + un-rotated part, the latter through K_nope = c . W_uk,h."""
    k_rope = np.asarray(k_rope, dtype=F64)
    c = np.asarray(c, dtype=F64)
    W_uk = np.asarray(W_uk, dtype=F64)
    q_rope, q_nope = query_parts(q, q_pos, idx, d_h, base, pair_mode)
    n_h, dn = q_nope.shape
    heads = range(n_h) if heads is None else heads
    out = []
    for h in heads:
        K_nope = c @ W_uk[:, h * dn:(h + 1) * dn]          # [n][d_h-2r]
        out.append(k_rope[:, h, :] @ q_rope[h] + K_nope @ q_nope[h])
    return np.stack(out)


def softmax_rows(s):
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def decode(q, q_pos, k_rope, c, W_uk, W_uv, idx, d_h, base=10000.0, scale=None, pair_mode=0,
           heads=None):
    """o[h] = softmax(scale * s[h]) . V_h with V_h = c . W_uv,h (Sections 2.1, 3.1, 3.2).
    k_rope [n][n_h][2r] are the cached rotated rows, c [n][d_c] the cached latents.
    Returns [len(heads)][d_h]; zeros when n == 0."""
    c = np.asarray(c, dtype=F64)
    W_uv = np.asarray(W_uv, dtype=F64)
    n_h = np.asarray(idx).shape[0]
    heads = list(range(n_h)) if heads is None else list(heads)
    if c.shape[0] == 0:
        return np.zeros((len(heads), d_h), dtype=F64)
    scale = 1.0 / np.sqrt(F64(d_h)) if scale is None else F64(scale)
    s = scores(q, q_pos, k_rope, c, W_uk, idx, d_h, base, pair_mode, heads)
    p = softmax_rows(scale * s)
    out = []
    for j, h in enumerate(heads):
        V = c @ W_uv[:, h * d_h:(h + 1) * d_h]              # [n][d_h]
        out.append(p[j] @ V)
    return np.stack(out)


def decode_absorbed(q, q_pos, k_rope, c, W_uk, W_uv, idx, d_h, base=10000.0, scale=None,
                    pair_mode=0, heads=None):
    """The same result with B^k and B^v folded outwards (Section 5): scores through
    q_abs . c, output through (sum_t p_t c_t) . W_uv,h.  Float64; equality with `decode` is a
    test, after which this cheaper form serves for long contexts."""
    k_rope = np.asarray(k_rope, dtype=F64)
    c = np.asarray(c, dtype=F64)
    W_uv = np.asarray(W_uv, dtype=F64)
    n_h = np.asarray(idx).shape[0]
    heads = list(range(n_h)) if heads is None else list(heads)
    if c.shape[0] == 0:
        return np.zeros((len(heads), d_h), dtype=F64)
    scale = 1.0 / np.sqrt(F64(d_h)) if scale is None else F64(scale)
    q_rope, q_abs = absorb_query(q, q_pos, idx, W_uk, d_h, base, pair_mode)
    out = []
    for h in heads:
        s = k_rope[:, h, :] @ q_rope[h] + c @ q_abs[h]
        p = softmax_rows(scale * s[None, :])[0]
        out.append((p @ c) @ W_uv[:, h * d_h:(h + 1) * d_h])
    return np.stack(out)


def decode_from_raw(q, q_pos, k_e, pos, c, W_uk, W_uv, idx, d_h, base=10000.0, scale=None,
                    heads=None):
    """End-to-end form: rotate the raw elite keys at their positions, then `decode`."""
    k_rope = rotate_elite_keys(k_e, pos, idx, d_h, base)
    return decode(q, q_pos, k_rope, c, W_uk, W_uv, idx, d_h, base, scale, 0, heads)


# --------------------------------------------------------------------------------------------
# Separated low-rank decomposition (S-LRD, Section 3.2): keys and values have their own latents
# --------------------------------------------------------------------------------------------
def decode_slrd(q, q_pos, k_rope, c_k, c_v, W_uk_S, W_uv_S, idx, d_h, base=10000.0, scale=None,
                pair_mode=0, heads=None):
    """Decode attention when W^k_e ~ A^k B^k_S and W^v ~ A^v B^v_S are factorised separately:
    the cache holds c_k = x A^k [n][d_ck] and c_v = x A^v [n][d_cv] beside the rotated elite
    rows; the un-rotated key dims of head h are c_k . B^k_S,h and its values c_v . B^v_S,h.
    W_uk_S [d_ck][n_h (d_h-2r)], W_uv_S [d_cv][n_h d_h].  Returns [len(heads)][d_h]."""
    k_rope = np.asarray(k_rope, dtype=F64)
    c_k = np.asarray(c_k, dtype=F64)
    c_v = np.asarray(c_v, dtype=F64)
    W_uk_S = np.asarray(W_uk_S, dtype=F64)
    W_uv_S = np.asarray(W_uv_S, dtype=F64)
    n_h = np.asarray(idx).shape[0]
    heads = list(range(n_h)) if heads is None else list(heads)
    if c_k.shape[0] == 0:
        return np.zeros((len(heads), d_h), dtype=F64)
    scale = 1.0 / np.sqrt(F64(d_h)) if scale is None else F64(scale)
    q_rope, q_nope = query_parts(q, q_pos, idx, d_h, base, pair_mode)
    dn = q_nope.shape[1]
    out = []
    for h in heads:
        K_nope = c_k @ W_uk_S[:, h * dn:(h + 1) * dn]        # [n][d_h-2r]
        V = c_v @ W_uv_S[:, h * d_h:(h + 1) * d_h]           # [n][d_h]
        s = k_rope[:, h, :] @ q_rope[h] + K_nope @ q_nope[h]
        p = softmax_rows(scale * s[None, :])[0]
        out.append(p @ V)
    return np.stack(out)


def cache_elements_per_token_slrd(n_h, r, d_ck, d_cv):
    """KV-cache elements per token per layer under S-LRD (Section 3.2)."""
    return 2 * r * n_h + d_ck + d_cv


# --------------------------------------------------------------------------------------------
# Several query rows over the cache (prefill chunk, speculative tokens): causal attention
# --------------------------------------------------------------------------------------------
def attend_causal(q, q_pos, k_rope, key_pos, c, W_uk, W_uv, idx, d_h, base=10000.0, scale=None,
                  pair_mode=0, heads=None):
    """The score equation of Section 3.1 for general query position m and key position n, with
    the causal rule of a decoder: query row i (q[i] at position q_pos[i]) sees the cached tokens
    whose position key_pos[t] <= q_pos[i].  q [m][n_h][d_h], k_rope [n][n_h][2r] (cached rotated
    rows), c [n][d_c].  Returns [m][len(heads)][d_h]; a row that sees no token is zero."""
    q = np.asarray(q, dtype=F64)
    k_rope = np.asarray(k_rope, dtype=F64)
    c = np.asarray(c, dtype=F64)
    W_uk = np.asarray(W_uk, dtype=F64)
    W_uv = np.asarray(W_uv, dtype=F64)
    key_pos = np.asarray(key_pos)
    n_h = np.asarray(idx).shape[0]
    heads = list(range(n_h)) if heads is None else list(heads)
    m, n = q.shape[0], c.shape[0]
    scale = 1.0 / np.sqrt(F64(d_h)) if scale is None else F64(scale)
    out = np.zeros((m, len(heads), d_h), dtype=F64)
    parts = [query_parts(q[i], int(q_pos[i]), idx, d_h, base, pair_mode) for i in range(m)]
    for j, h in enumerate(heads):
        dn = parts[0][1].shape[1]
        K_nope = c @ W_uk[:, h * dn:(h + 1) * dn]              # [n][d_h-2r]
        V = c @ W_uv[:, h * d_h:(h + 1) * d_h]                 # [n][d_h]
        S = np.empty((m, n), dtype=F64)
        for i in range(m):
            q_rope, q_nope = parts[i]
            S[i] = k_rope[:, h, :] @ q_rope[h] + K_nope @ q_nope[h]
        for i in range(m):
            seen = key_pos <= int(q_pos[i])
            if not seen.any():
                continue
            p = softmax_rows((scale * S[i, seen])[None, :])[0]
            out[i, j] = p @ V[seen]
    return out


# --------------------------------------------------------------------------------------------
# Uncompressed RoPE multi-head attention (Section 2.1 + 2.2): the comparator's definition
# --------------------------------------------------------------------------------------------
def mha_decode(q_hat, K_hat, V, scale=None, heads=None):
    """q_hat [n_h][d_h] rotated query, K_hat [n][n_h][d_h] rotated keys, V [n][n_h][d_h]."""
    q_hat = np.asarray(q_hat, dtype=F64)
    K_hat = np.asarray(K_hat, dtype=F64)
    V = np.asarray(V, dtype=F64)
    n_h, d_h = q_hat.shape
    heads = list(range(n_h)) if heads is None else list(heads)
    if K_hat.shape[0] == 0:
        return np.zeros((len(heads), d_h), dtype=F64)
    scale = 1.0 / np.sqrt(F64(d_h)) if scale is None else F64(scale)
    out = []
    for h in heads:
        p = softmax_rows((scale * (K_hat[:, h, :] @ q_hat[h]))[None, :])[0]
        out.append(p @ V[:, h, :])
    return np.stack(out)


def cache_elements_per_token(n_h, r, d_c):
    """KV-cache elements per token per layer under J-LRD (end of Section 3.2)."""
    return 2 * r * n_h + d_c
