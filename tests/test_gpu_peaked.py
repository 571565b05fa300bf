"""GPU parity on PEAKED attention.  With iid N(0,1) inputs the scores of a head differ by a
couple of units between tiles, so the running maximum of the online softmax (paper Section 2.1,
evaluated tile by tile) hardly ever moves after the first tile, and the branch that rescales the
running sum and the accumulated output never runs.  Real attention is peaked; these cases make
it so, at contexts long enough that a worker's plan item spans several tiles:

  scaled   queries multiplied by 8: score spread ~8x, the maximum keeps moving upwards
  planted  tokens whose latent is aligned with one head's absorbed query, with scores that climb
           in runs along the sequence: an outlier in the first tile of an item (later tiles negligible),
           in a later tile of an item (everything before it is rescaled away), and several in
           one item (repeated rescales)

The tensor-core kernels move their reference maximum lazily (only when a tile maximum exceeds it
by more than 8 in base-2 units); the tests replay that rule on the oracle's scores over the
library's own work plan and insist that it fires in a tile other than an item's first.
Outputs are O(1) here, so the absolute tolerance binds as well as the relative one."""
import math
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import elitekv_oracle as O
from paper_2503_01586_b200 import inputs as gen

from . import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ek():
    from paper_2503_01586_b200 import binding
    binding.lib()
    return binding


def _plant(st, plants):
    """plants: (sequence, token, head, score in natural-log units).  Overwrites the token's
    latent with the multiple of q_abs[b, h] that gives that head exactly this latent score."""
    w = st.w
    idx = st.idx.numpy().astype(np.int64)
    W_uk = H.f64(st.W_uk)
    scale = 1.0 / math.sqrt(w.d_h)
    cache = {}
    for b, t, h, score in plants:
        if b not in cache:
            cache[b] = O.absorb_query(H.f64(st.q[b]), int(st.lens[b]) - 1, idx, W_uk, w.d_h, w.rope_base)[1]
        qa = cache[b][h]
        c_new = (score / scale) * qa / float(qa @ qa)
        st.c[int(st.starts[b]) + t] = torch.from_numpy(c_new).to(torch.bfloat16).to(st.c.device)


def _moves_after_first_tile(ek, st, units):
    """Replays the lazy reference-maximum rule on the oracle's scores: number of (unit, item,
    tile > 0) triples in which the reference moves."""
    w = st.w
    kernel, tile, n_workers, max_items, overhead = ek.elitekv_decode_plan_info(st.layer, st.cache, w.B)
    if n_workers == 0:
        items, first = ek.elitekv_plan(st.lens_dev, tile, max_items)
    else:
        items, first, _ = ek.elitekv_plan_workers(st.lens_dev, tile, n_workers, max_items, overhead)
    torch.cuda.synchronize()
    items, first = items.cpu().numpy(), first.cpu().numpy()
    idx = st.idx.numpy().astype(np.int64)
    W_uk = H.f64(st.W_uk)
    log2e_scale = math.log2(math.e) / math.sqrt(w.d_h)
    moves = 0
    by_seq = {}
    for b, h in units:
        by_seq.setdefault(b, []).append(h)
    for b, heads in by_seq.items():
        lo, hi = int(st.starts[b]), int(st.starts[b + 1])
        k_rope = O.rotate_elite_keys(H.f64(st.k_e[lo:hi]), np.arange(hi - lo), idx, w.d_h, w.rope_base)
        s = O.scores(H.f64(st.q[b]), hi - lo - 1, k_rope, H.f64(st.c[lo:hi]), W_uk, idx, w.d_h,
                     w.rope_base, heads=heads) * log2e_scale
        for row in s:
            for seq, t0, cnt, _ in items[first[b]:first[b + 1]]:
                assert seq == b
                m_ref = -np.inf
                for k, a in enumerate(range(t0, t0 + cnt, tile)):
                    tm = row[a:min(a + tile, t0 + cnt)].max()
                    if tm > m_ref + 8.0:
                        moves += k > 0
                        m_ref = tm
    return kernel, moves


SHAPES = {
    # name: (workload, lengths); long enough that every persistent worker gets several tiles
    "7b": (gen.LLAMA7B_75, [20000, 14001]),
    "7b-paged": (replace(gen.LLAMA7B_75, paged=True, page_size=64), [19999, 14100]),
    "13b": (gen.LLAMA13B_75, [9000, 4100]),
    "50pct": (gen.SWEEP_50, [12000, 8100]),
    "87.5pct": (gen.SWEEP_875, [20000, 14001]),
}


def _plants_for(lens, n_h):
    plants = []
    for b, n in enumerate(lens):
        k = 0
        t = 70 + 31 * b
        while t < n - 1:
            # scores climb in runs of four (14, 21, 28, 35 natural units = 20 ... 50 base-2 units
            # above the crowd), so inside an item each outlier tops the previous one by far
            plants.append((b, t, (5 + 3 * b + k // 4) % n_h, 14.0 + 7.0 * (k % 4)))
            k += 1
            t += 197 + 61 * (k % 5)       # 1.5 - 3.5 tiles apart: first, middle and last tiles of items
    return plants


def _run(ek, shape, mode, kernel):
    w0, lens = SHAPES[shape]
    w = replace(w0, name=f"{w0.name}-peaked", B=len(lens), ctx=max(lens), ctx_lo=None, seed=w0.seed + 400)
    plants = _plants_for(lens, w.n_h) if mode == "planted" else []
    st = H.setup(w, lens=lens, decode_kernel=kernel, q_scale=8.0 if mode == "scaled" else 1.0,
                 edit_tokens=(lambda s: _plant(s, plants)) if plants else None)
    out = H.run_decode(st)
    assert torch.isfinite(out.float()).all()
    if mode == "planted":
        # the heads that own the last outliers of each sequence, plus a few bystanders
        owners = sorted({(b, h) for b, _, h, _ in plants})
        units = sorted(set(owners[::max(1, len(owners) // 8)]) | set(H.sample_units(st, 4, seed=9)))
    else:
        units = H.sample_units(st, 12, seed=9)
    want = H.oracle_units(st, units)
    o = H.f64(out)
    got = np.stack([o[b, h] for b, h in units])
    rel, mx = H.errors(got, want)
    assert np.max(np.abs(want)) > 0.5          # O(1) outputs: the absolute bound is a real one
    assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL, (rel, mx)
    # element by element, relative to the size of the unit's output row
    rows = np.max(np.abs(want), axis=1, keepdims=True)
    assert np.all(np.abs(got - want) <= 4e-2 * rows), float(np.max(np.abs(got - want) / rows))
    used, moves = _moves_after_first_tile(ek, st, units)
    if used != 1:
        assert moves > 0, "the inputs did not move the reference maximum after an item's first tile"
    return used


@pytest.mark.parametrize("mode", ["scaled", "planted"])
@pytest.mark.parametrize("kernel", [1, 2, 3], ids=["generic", "two-pass", "resident"])
def test_peaked_7b_shape_each_kernel(ek, mode, kernel):
    assert _run(ek, "7b", mode, kernel) == kernel


@pytest.mark.parametrize("mode", ["scaled", "planted"])
@pytest.mark.parametrize("shape", ["7b-paged", "13b", "50pct", "87.5pct"])
def test_peaked_other_shapes_default_kernel(ek, shape, mode):
    _run(ek, shape, mode, 0)
