"""Seeded synthetic inputs with the shapes of LLaMA2-7B/13B EliteKV layers.

This module only draws random tensors, index sets, lengths and page permutations.  It holds
none of the method's arithmetic (no RoPE, no attention, no cache layout) so that both the CUDA
library's tests and the CPU oracle's tests can be fed the same bytes from here.

All floating-point tensors are bf16 (the storage type of the cache and of the weights); index
tensors are int32.  `device` may be "cpu" or "cuda"; the same seed gives different streams on
the two device types, so callers generate once and copy.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    n_h: int            # heads
    d_h: int            # head dim
    r: int              # elite RoPE chunks per head
    d_c: int            # latent width
    d: int              # model width (only sets the weight variance 1/d)
    B: int              # sequences decoded per step
    ctx: int            # context per sequence (upper bound when ctx_lo is set)
    ctx_lo: Optional[int] = None   # if set, lengths are uniform in [ctx_lo, ctx]
    paged: bool = False
    page_size: int = 64
    rope_base: float = 10000.0
    seed: int = 0
    d_ck: int = 0       # > 0: separated latents, a latent row is [c_k (d_ck) | c_v (d_c - d_ck)]

    @property
    def cache_elems_per_token(self) -> int:
        return 2 * self.r * self.n_h + self.d_c

    @property
    def d_nope(self) -> int:
        return self.d_h - 2 * self.r


# The five benchmark configurations (index = configuration number - 1).
TINY = Workload("tiny", n_h=4, d_h=64, r=2, d_c=64, d=256, B=1, ctx=256, seed=1001)
LLAMA7B_75 = Workload("7b-75pct-b16-ctx4096", n_h=32, d_h=128, r=8, d_c=1536, d=4096, B=16,
                      ctx=4096, seed=1002)
LLAMA7B_75_PAGED = Workload("7b-75pct-paged-b64-ragged", n_h=32, d_h=128, r=8, d_c=1536, d=4096,
                            B=64, ctx=32768, ctx_lo=1024, paged=True, seed=1003)
LLAMA13B_75 = Workload("13b-75pct-b32-ctx16384", n_h=40, d_h=128, r=8, d_c=1920, d=5120, B=32,
                       ctx=16384, seed=1004)
SWEEP_50 = Workload("7b-50pct-b32-ctx8192", n_h=32, d_h=128, r=16, d_c=3072, d=4096, B=32,
                    ctx=8192, seed=1005)
SWEEP_75 = replace(SWEEP_50, name="7b-75pct-b32-ctx8192", r=8, d_c=1536)
SWEEP_875 = replace(SWEEP_50, name="7b-87.5pct-b32-ctx8192", r=4, d_c=768)
# the 75 % cache split into a key latent of 512 and a value latent of 1024 (S-LRD)
SWEEP_75_SLRD = replace(SWEEP_75, name="7b-75pct-slrd512+1024-b32-ctx8192", d_ck=512)

CONFIGS = {w.name: w for w in
           (TINY, LLAMA7B_75, LLAMA7B_75_PAGED, LLAMA13B_75, SWEEP_50, SWEEP_75, SWEEP_875, SWEEP_75_SLRD)}


def shrink(w: Workload, *, B: int, ctx: int, ctx_lo: Optional[int] = None) -> Workload:
    """Same layer shape, smaller batch/context (for parity cases the oracle finishes quickly)."""
    return replace(w, name=f"{w.name}-small", B=B, ctx=ctx,
                   ctx_lo=ctx_lo if w.ctx_lo is not None else None)


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal_bf16(shape, std: float, gen: torch.Generator, device) -> torch.Tensor:
    """N(0, std^2) drawn in fp32, rounded to bf16.  Large tensors are drawn in slabs."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    step = 1 << 26
    for lo in range(0, flat.numel(), step):
        hi = min(flat.numel(), lo + step)
        flat[lo:hi] = (torch.randn(hi - lo, generator=gen, device=device,
                                   dtype=torch.float32) * std).to(torch.bfloat16)
    return out


def elite_index_sets(w: Workload) -> torch.Tensor:
    """int32 [n_h][r]: per head r distinct chunk ids out of d_h/2, in random order
    (stand-in for the searched per-head frequency preferences)."""
    g = _gen(w.seed * 7 + 1, "cpu")
    rows = [torch.randperm(w.d_h // 2, generator=g)[: w.r] for _ in range(w.n_h)]
    return torch.stack(rows).to(torch.int32) if w.r > 0 else torch.zeros((w.n_h, 0), dtype=torch.int32)


def up_projections(w: Workload, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """W_uk bf16 [d_c][n_h*(d_h-2r)], W_uv bf16 [d_c][n_h*d_h], entries N(0, 1/d)."""
    g = _gen(w.seed * 7 + 2, device)
    std = (1.0 / w.d) ** 0.5
    W_uk = _normal_bf16((w.d_c, w.n_h * w.d_nope), std, g, device)
    W_uv = _normal_bf16((w.d_c, w.n_h * w.d_h), std, g, device)
    return W_uk, W_uv


def sequence_lengths(w: Workload) -> torch.Tensor:
    """int32 [B]: every sequence `ctx` tokens, or uniform in [ctx_lo, ctx] by seed."""
    if w.ctx_lo is None:
        return torch.full((w.B,), w.ctx, dtype=torch.int32)
    g = _gen(w.seed * 7 + 3, "cpu")
    return torch.randint(w.ctx_lo, w.ctx + 1, (w.B,), generator=g).to(torch.int32)


def page_table(w: Workload, lens: torch.Tensor, headroom_tokens: int = 1):
    """Paged layout: each sequence owns ceil((len+headroom)/page_size) pages; physical page ids
    are one seeded random permutation of [0, num_pages).  Returns (int32 [B][max_pages] padded
    with -1, num_pages)."""
    need = [(int(n) + headroom_tokens + w.page_size - 1) // w.page_size for n in lens.tolist()]
    num_pages = sum(need)
    g = _gen(w.seed * 7 + 4, "cpu")
    perm = torch.randperm(num_pages, generator=g).to(torch.int32)
    table = torch.full((w.B, max(need)), -1, dtype=torch.int32)
    at = 0
    for b, k in enumerate(need):
        table[b, :k] = perm[at:at + k]
        at += k
    return table, num_pages


def tokens(w: Workload, T: int, device="cpu", stream: int = 0):
    """T cached tokens' raw material: un-rotated elite key chunks bf16 [T][n_h][r][2] and
    latents bf16 [T][d_c], iid N(0,1) (the law of x.W for x~N(0,1), W~N(0,1/d))."""
    g = _gen(w.seed * 7 + 5 + 1000 * stream, device)
    k_e = _normal_bf16((T, w.n_h, w.r, 2), 1.0, g, device)
    c = _normal_bf16((T, w.d_c), 1.0, g, device)
    return k_e, c


def queries(w: Workload, device="cpu") -> torch.Tensor:
    """bf16 [B][n_h][d_h] un-rotated queries, iid N(0,1)."""
    g = _gen(w.seed * 7 + 6, device)
    return _normal_bf16((w.B, w.n_h, w.d_h), 1.0, g, device)


def mha_cache(w: Workload, T: int, device="cpu"):
    """Uncompressed comparator cache: rotated keys and values, bf16 [T][n_h][d_h] each,
    iid N(0,1) (a rotation leaves the law of an iid Gaussian pair unchanged)."""
    g = _gen(w.seed * 7 + 7, device)
    K = _normal_bf16((T, w.n_h, w.d_h), 1.0, g, device)
    V = _normal_bf16((T, w.n_h, w.d_h), 1.0, g, device)
    return K, V


def projected_chain(w: Workload, idx: torch.Tensor, T: int):
    """Small configurations only: hidden states x ~ N(0,1) [T][d] pushed through random
    projections W^q, W^k_e (the elite key columns) and W_down ~ N(0, 1/d) in float64, each
    result rounded to bf16.  Returns q_all bf16 [T][n_h][d_h], k_e bf16 [T][n_h][r][2],
    c bf16 [T][d_c].  Plain matrix products, no positional or attention arithmetic."""
    g = _gen(w.seed * 7 + 8, "cpu")
    std = (1.0 / w.d) ** 0.5
    x = torch.randn(T, w.d, generator=g, dtype=torch.float64)
    Wq = torch.randn(w.d, w.n_h * w.d_h, generator=g, dtype=torch.float64) * std
    Wke = torch.randn(w.d, w.n_h * w.r * 2, generator=g, dtype=torch.float64) * std
    Wdown = torch.randn(w.d, w.d_c, generator=g, dtype=torch.float64) * std
    q = (x @ Wq).to(torch.bfloat16).view(T, w.n_h, w.d_h)
    k_e = (x @ Wke).to(torch.bfloat16).view(T, w.n_h, w.r, 2)
    c = (x @ Wdown).to(torch.bfloat16).view(T, w.d_c)
    return q, k_e, c
