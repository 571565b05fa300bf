"""GPU parity of elitekv_attend_rows: several query rows per sequence over the cache with the
causal rule (the score equation of paper Section 3.1 for general query and key positions).
Every case compares all query rows of the sampled heads with the float64 oracle's
`attend_causal` on the same bytes."""
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


def _run_rows(ek, st, m, seed):
    """m query rows per sequence at the last m positions; returns (q, out)."""
    w = st.w
    B = w.B
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = torch.randn((B, m, w.n_h, w.d_h), generator=g).to(torch.bfloat16).cuda()
    q_pos = (st.lens_dev.view(B, 1) - m + torch.arange(m, device="cuda", dtype=torch.int32).view(1, m)).to(torch.int32)
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, q.view(B * m, w.n_h, w.d_h), q_pos.reshape(-1).contiguous())
    ws = torch.empty(ek.elitekv_attend_rows_workspace_size(st.layer, B, m), dtype=torch.uint8, device="cuda")
    out = ek.elitekv_attend_rows(st.layer, st.cache, q_rope, q_abs, st.lens_dev, m, ws)
    torch.cuda.synchronize()
    code = ek.elitekv_check_status(st.layer)
    assert code == 0, ek.strerror(code)
    return q, out


def _check_rows(st, q, out, m, heads):
    w = st.w
    idx = st.idx.numpy().astype(np.int64)
    W_uk, W_uv = H.f64(st.W_uk), H.f64(st.W_uv)
    worst = (0.0, 0.0)
    for b in range(w.B):
        lo, hi = int(st.starts[b]), int(st.starts[b + 1])
        n = hi - lo
        key_pos = np.arange(n)
        k_rope = O.rotate_elite_keys(H.f64(st.k_e[lo:hi]), key_pos, idx, w.d_h, w.rope_base)
        c = H.f64(st.c[lo:hi])
        q_pos = n - m + np.arange(m)
        if st.d_ck:
            want = np.stack([O.decode_slrd(H.f64(q[b, i]), int(q_pos[i]), k_rope[:q_pos[i] + 1], c[:q_pos[i] + 1, :st.d_ck],
                                           c[:q_pos[i] + 1, st.d_ck:], W_uk, W_uv, idx, w.d_h, base=w.rope_base, heads=heads)
                             for i in range(m)])
        else:
            want = O.attend_causal(H.f64(q[b]), q_pos, k_rope, key_pos, c, W_uk, W_uv, idx, w.d_h,
                                   base=w.rope_base, heads=heads)
        got = H.f64(out[b])[:, heads, :]
        rel, mx = H.errors(got.reshape(-1, w.d_h), want.reshape(-1, w.d_h))
        assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL, (b, rel, mx)
        worst = max(worst, (rel, mx))
    return worst


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("m", [2, 5])
def test_rows_7b_shape(ek, m, paged):
    """Tile edges inside the last m tokens: a length of 128 + 2 puts the rows' causal limits on
    both sides of a tile boundary; a length of m makes row 0 see a single token; 700 spans
    several tiles and several plan items."""
    w = gen.shrink(gen.LLAMA7B_75, B=5, ctx=700)
    if paged:
        w = replace(w, paged=True, page_size=64)
    st = H.setup(w, lens=[700, 130, 129, m, 64 + m - 1])
    q, out = _run_rows(ek, st, m, 700 + m)
    _check_rows(st, q, out, m, [0, 7, 31])
    # the rows differ (a shared, unmasked result would pass a weak check)
    assert not torch.equal(out[:, 0], out[:, m - 1])


def test_rows_other_shapes(ek):
    """40 heads (two head groups per query row), a narrow latent, separated latents, m = 16."""
    st = H.setup(gen.shrink(gen.LLAMA13B_75, B=2, ctx=300), lens=[300, 67])
    q, out = _run_rows(ek, st, 3, 11)
    _check_rows(st, q, out, 3, [0, 31, 32, 39])
    st = H.setup(gen.shrink(gen.SWEEP_875, B=2, ctx=400), lens=[400, 16])
    q, out = _run_rows(ek, st, 16, 12)
    _check_rows(st, q, out, 16, [3, 30])
    st = H.setup(gen.shrink(gen.LLAMA7B_75, B=2, ctx=260), lens=[260, 131], d_ck=512)
    q, out = _run_rows(ek, st, 4, 13)
    _check_rows(st, q, out, 4, [1, 18])


def test_one_row_is_the_decode_call(ek):
    w = gen.shrink(gen.LLAMA7B_75, B=3, ctx=500)
    st = H.setup(w, lens=[500, 128, 1], decode_kernel=2)
    want = H.run_decode(st)
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
    ws = torch.empty(ek.elitekv_attend_rows_workspace_size(st.layer, 3, 1), dtype=torch.uint8, device="cuda")
    got = ek.elitekv_attend_rows(st.layer, st.cache, q_rope, q_abs, st.lens_dev, 1, ws)
    torch.cuda.synchronize()
    assert torch.equal(got.view_as(want), want)


def test_rows_argument_checks(ek):
    w = gen.shrink(gen.LLAMA7B_75, B=1, ctx=40)
    st = H.setup(w, lens=[40])
    for m in (0, 17):
        with pytest.raises(ek.ElitekvError) as e:
            ek.elitekv_attend_rows_workspace_size(st.layer, 1, m)
        assert e.value.code == ek.ERR_INVALID_ARG
    st1 = H.setup(w, lens=[40], decode_kernel=1)
    q_rope, q_abs = ek.elitekv_absorb_query(st1.layer, torch.zeros((2, w.n_h, w.d_h), dtype=torch.bfloat16, device="cuda"),
                                            torch.tensor([38, 39], dtype=torch.int32, device="cuda"))
    ws = torch.empty(ek.elitekv_attend_rows_workspace_size(st1.layer, 1, 2), dtype=torch.uint8, device="cuda")
    with pytest.raises(ek.ElitekvError) as e:      # the layer insists on the generic kernel, which serves one row
        ek.elitekv_attend_rows(st1.layer, st1.cache, q_rope, q_abs, st1.lens_dev, 2, ws)
    assert e.value.code == ek.ERR_UNSUPPORTED_SHAPE
    small = H.setup(gen.TINY, lens=[40])               # a shape the tensor-core kernel does not cover
    with pytest.raises(ek.ElitekvError) as e:
        ek.elitekv_attend_rows_workspace_size(small.layer, 1, 2)
    assert e.value.code == ek.ERR_UNSUPPORTED_SHAPE
