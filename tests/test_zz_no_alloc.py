"""elitekv_decode_static -- the decode entry point for callers that may not allocate device
memory (arena-only serving engines, plugins inside another framework's step).  It must give
what elitekv_decode gives, call after call, while keeping its scratch inside the library.
Collected last on purpose: a failure here leaves every other test already run."""
import ctypes as C
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2503_01586_b200 import inputs as gen

from . import harness as H

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_workspace_decode_twice():
    from paper_2503_01586_b200 import binding as ek
    w = gen.shrink(gen.LLAMA7B_75, B=3, ctx=400)
    st = H.setup(w, lens=[400, 129, 64])
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
    want = ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, st.lens_dev, st.workspace)
    torch.cuda.synchronize()
    want = H.f64(want)
    out = torch.empty((w.B, w.n_h, w.d_h), dtype=torch.bfloat16, device="cuda")
    for call in range(2):
        out.fill_(float("nan"))
        ek.elitekv_decode_static(st.layer, st.cache, q_rope, q_abs, st.lens_dev, out)
        torch.cuda.synchronize()
        assert ek.elitekv_check_status(st.layer) == 0
        rel, mx = H.errors(H.f64(out), want)
        assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL, (call, rel, mx)
        # a different batch in between must not leak into the next call through the shared array
        if call == 0:
            other = H.setup(replace(w, seed=w.seed + 1), lens=[70, 300, 5])
            qr2, qa2 = ek.elitekv_absorb_query(other.layer, other.q, other.q_pos)
            o2 = torch.empty_like(out)
            ek.elitekv_decode_static(other.layer, other.cache, qr2, qa2, other.lens_dev, o2)
            ref2 = ek.elitekv_decode(other.layer, other.cache, qr2, qa2, other.lens_dev, other.workspace)
            torch.cuda.synchronize()
            rel2, mx2 = H.errors(H.f64(o2), H.f64(ref2))
            assert rel2 <= H.REL_L2_TOL and mx2 <= H.MAX_ABS_TOL
    # and against the oracle, like every other decode test
    H.check_parity(st, out, H.sample_units(st, 12))


def test_static_scratch_rejects_oversized_requests():
    from paper_2503_01586_b200 import binding as ek
    w = gen.shrink(gen.LLAMA7B_75, B=512, ctx=2)
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, "cuda")
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, 8)
    assert ek.elitekv_decode_workspace_size(layer, w.B) > ek.STATIC_SCRATCH_BYTES
    rope = torch.zeros((w.B * 2, w.n_h * 2 * w.r), dtype=torch.bfloat16, device="cuda")
    lat = torch.zeros((w.B * 2, w.d_c), dtype=torch.bfloat16, device="cuda")
    cache = ek.make_cache(rope, lat, n_seqs=w.B, max_ctx=2)
    q_rope = torch.zeros((w.B, w.n_h, 2 * w.r), dtype=torch.bfloat16, device="cuda")
    q_abs = torch.zeros((w.B, w.n_h, w.d_c), dtype=torch.bfloat16, device="cuda")
    lens = torch.ones((w.B,), dtype=torch.int32, device="cuda")
    out = torch.empty((w.B, w.n_h, w.d_h), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(ek.ElitekvError) as e:
        ek.elitekv_decode_static(layer, cache, q_rope, q_abs, lens, out)
    assert e.value.code == ek.ERR_STATIC_SCRATCH_EXCEEDED
    assert "scratch" in ek.strerror(e.value.code)
