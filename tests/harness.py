"""Test/bench scaffolding: lays a workload out on the GPU through the C ABI and evaluates the
float64 oracle on chosen (sequence, head) units of the same bytes."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import elitekv_oracle as O
from paper_2503_01586_b200 import binding as ek
from paper_2503_01586_b200 import inputs as gen

REL_L2_TOL = 1e-2     # ||o_gpu - o_ref||_2 / ||o_ref||_2
MAX_ABS_TOL = 3e-2    # max |o_gpu - o_ref|


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16)


@dataclass
class State:
    w: gen.Workload
    idx: torch.Tensor            # cpu int32 [n_h][r]
    W_uk: torch.Tensor           # cuda bf16
    W_uv: torch.Tensor
    lens: torch.Tensor           # cpu int32 [B] tokens per sequence INCLUDING the decoded one
    starts: np.ndarray           # [B+1] offsets of each sequence in the token stream
    k_e: torch.Tensor            # cuda bf16 [N][n_h][r][2]
    c: torch.Tensor              # cuda bf16 [N][d_c]
    seq_id: torch.Tensor         # cuda int32 [N]
    pos: torch.Tensor            # cuda int32 [N]
    q: torch.Tensor              # cuda bf16 [B][n_h][d_h]
    q_pos: torch.Tensor          # cuda int32 [B]
    layer: ek.Layer
    cache: ek.CacheDesc
    rope_plane: torch.Tensor
    latent_plane: torch.Tensor
    page_table: Optional[torch.Tensor]
    lens_dev: torch.Tensor
    workspace: torch.Tensor
    pos_offset: int = 0
    d_ck: int = 0                # > 0: separated latents, a latent row is [c_k (d_ck) | c_v]


def setup(w: gen.Workload, *, lens: Optional[Sequence[int]] = None, decode_kernel: int = 0,
          pos_offset: int = 0, cos_sin=None, fill: bool = True, device="cuda",
          q_scale: float = 1.0, edit_tokens=None, d_ck: int = 0) -> State:
    """Builds layer, cache planes and the token stream; when `fill`, appends every token of
    every sequence (so the cache holds lens[b] tokens, the last being the decoding token).
    `q_scale` multiplies the drawn queries (exactly, for a power of two); `edit_tokens(st)` may
    overwrite rows of st.k_e / st.c before they are appended."""
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, device)
    d_ck = d_ck or w.d_ck
    if d_ck:
        # S-LRD: B^k_S reads the first d_ck latent columns, B^v_S the remaining ones
        W_uk, W_uv = W_uk[:d_ck].contiguous(), W_uv[d_ck:].contiguous()
    lens_t = gen.sequence_lengths(w) if lens is None else torch.tensor(list(lens), dtype=torch.int32)
    B = w.B
    assert lens_t.numel() == B
    starts = np.concatenate([[0], np.cumsum(lens_t.numpy().astype(np.int64))])
    N = int(starts[-1])
    k_e, c = gen.tokens(w, N, device)
    seq_id = torch.repeat_interleave(torch.arange(B, dtype=torch.int32), lens_t.to(torch.int64))
    pos = torch.cat([torch.arange(int(n), dtype=torch.int32) for n in lens_t.tolist()]) if N else \
        torch.zeros(0, dtype=torch.int32)
    q = gen.queries(w, device)
    if q_scale != 1.0:
        q = (q.float() * q_scale).to(torch.bfloat16)
    q_pos = (lens_t - 1).clamp(min=0)
    max_pos = int(lens_t.max().item()) + 2 if B else 2
    if pos_offset:
        # RoPE positions shifted by a constant while cache slots stay put: hand the layer a
        # (cos, sin) table that starts at pos_offset
        tab = O.rope_table_f32(max_pos + pos_offset, w.d_h, w.rope_base)[pos_offset:]
        cos_sin = torch.from_numpy(np.ascontiguousarray(tab)).to(device)
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, max_pos, rope_base=w.rope_base,
                     cos_sin=cos_sin, decode_kernel=decode_kernel, d_ck=d_ck)
    rope_w = w.n_h * 2 * w.r
    if w.paged:
        table, num_pages = gen.page_table(w, lens_t, headroom_tokens=1)
        rows = num_pages * w.page_size
        page_table = table.to(device)
        max_ctx = 0
    else:
        page_table = None
        max_ctx = int(lens_t.max().item()) + 1
        rows = B * max_ctx
    rope_plane = (torch.zeros((rows, rope_w), dtype=torch.bfloat16, device=device) if rope_w > 0
                  else torch.zeros((8,), dtype=torch.bfloat16, device=device))   # r = 0: never read
    latent_plane = torch.zeros((rows, w.d_c), dtype=torch.bfloat16, device=device)
    cache = ek.make_cache(rope_plane, latent_plane, n_seqs=B, max_ctx=max_ctx,
                          page_table=page_table, page_size=w.page_size)
    ws = torch.empty(ek.elitekv_decode_workspace_size(layer, B), dtype=torch.uint8, device=device)
    st = State(w, idx, W_uk, W_uv, lens_t, starts, k_e, c, seq_id.to(device), pos.to(device), q,
               q_pos.to(torch.int32).to(device), layer, cache, rope_plane, latent_plane, page_table,
               lens_t.to(device), ws, pos_offset, d_ck)
    if edit_tokens is not None:
        edit_tokens(st)
    if fill and N:
        ek.elitekv_append(layer, cache, st.k_e, st.c, st.seq_id, st.pos)
    return st


def run_decode(st: State) -> torch.Tensor:
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
    out = ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, st.lens_dev, st.workspace)
    torch.cuda.synchronize()
    code = ek.elitekv_check_status(st.layer)
    assert code == 0, ek.strerror(code)
    return out


def oracle_units(st: State, units: Sequence[Tuple[int, int]]) -> np.ndarray:
    """Float64 oracle output [len(units)][d_h] from the RAW inputs (end-to-end parity)."""
    w = st.w
    idx = st.idx.numpy().astype(np.int64)
    W_uk, W_uv = f64(st.W_uk), f64(st.W_uv)
    out = []
    by_seq = {}
    for u, (b, h) in enumerate(units):
        by_seq.setdefault(b, []).append((u, h))
    res = [None] * len(units)
    for b, lst in by_seq.items():
        lo, hi = int(st.starts[b]), int(st.starts[b + 1])
        k_e = f64(st.k_e[lo:hi])
        c = f64(st.c[lo:hi])
        posv = np.arange(hi - lo) + st.pos_offset
        q = f64(st.q[b])
        heads = [h for _, h in lst]
        q_pos = int(max(hi - lo - 1, 0)) + st.pos_offset
        if st.d_ck:
            k_rope = O.rotate_elite_keys(k_e, posv, idx, w.d_h, w.rope_base)
            o = O.decode_slrd(q, q_pos, k_rope, c[:, :st.d_ck], c[:, st.d_ck:], W_uk, W_uv, idx, w.d_h,
                              base=w.rope_base, heads=heads)
        else:
            o = O.decode_from_raw(q, q_pos, k_e, posv, c, W_uk, W_uv, idx, w.d_h, base=w.rope_base, heads=heads)
        for (u, _), row in zip(lst, o):
            res[u] = row
    return np.stack(res)


def all_units(st: State) -> List[Tuple[int, int]]:
    return [(b, h) for b in range(st.w.B) for h in range(st.w.n_h)]


def sample_units(st: State, k: int, seed: int = 0) -> List[Tuple[int, int]]:
    g = np.random.default_rng(seed + 17 * st.w.seed)
    total = st.w.B * st.w.n_h
    pick = g.choice(total, size=min(k, total), replace=False)
    return [(int(p // st.w.n_h), int(p % st.w.n_h)) for p in pick]


def errors(got: np.ndarray, want: np.ndarray) -> Tuple[float, float]:
    d = got - want
    denom = float(np.linalg.norm(want))
    rel = float(np.linalg.norm(d)) / denom if denom > 0 else float(np.linalg.norm(d))
    return rel, float(np.max(np.abs(d))) if d.size else 0.0


def check_parity(st: State, out: torch.Tensor, units: Sequence[Tuple[int, int]]) -> Tuple[float, float]:
    want = oracle_units(st, units)
    o = f64(out)
    got = np.stack([o[b, h] for b, h in units])
    rel, mx = errors(got, want)
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, (rel, mx)
    return rel, mx
