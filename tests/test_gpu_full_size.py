"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the five
workload configurations, checked on seeded samples of (sequence, head) units that the float64
oracle evaluates one by one at full context (units are independent: everything is per head and
sequences never interact)."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2503_01586_b200 import inputs as gen

from . import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ek():
    from paper_2503_01586_b200 import binding
    binding.lib()
    return binding


def _free():
    import gc
    gc.collect()
    torch.cuda.empty_cache()


def _run(ek, w, n_units, two_step_append=False):
    if not two_step_append:
        st = H.setup(w)
    else:
        # cache holds len-1 tokens; the step appends one token per sequence, then decodes
        st = H.setup(w, fill=False)
        last = torch.from_numpy(st.starts[1:] - 1).to(torch.int64).cuda()
        keep = torch.ones(st.c.shape[0], dtype=torch.bool, device="cuda")
        keep[last] = False
        idx_pre = torch.nonzero(keep).squeeze(1)
        ek.elitekv_append(st.layer, st.cache, st.k_e[idx_pre].contiguous(), st.c[idx_pre].contiguous(),
                          st.seq_id[idx_pre].contiguous(), st.pos[idx_pre].contiguous())
        ek.elitekv_append(st.layer, st.cache, st.k_e[last].contiguous(), st.c[last].contiguous(),
                          st.seq_id[last].contiguous(), st.pos[last].contiguous())
        del idx_pre, keep
    out = H.run_decode(st)
    units = H.sample_units(st, n_units)
    rel, mx = H.check_parity(st, out, units)
    # outputs are finite everywhere, not only on the sampled units
    assert torch.isfinite(out.float()).all()
    del st, out
    _free()
    return rel, mx


def test_config2_7b_75pct_b16_ctx4096(ek):
    """The benchmark workload: every one of its 16 x 32 (sequence, head) units."""
    _run(ek, gen.LLAMA7B_75, 16 * 32)


def test_config2_all_three_kernels_agree(ek):
    """The CUDA-core kernel and the tcgen05 kernels on the same full-size inputs."""
    outs = []
    for kernel in (1, 2, 3):
        st = H.setup(gen.LLAMA7B_75, decode_kernel=kernel)
        outs.append(H.f64(H.run_decode(st)))
        del st
        _free()
    for o in outs[1:]:
        rel, mx = H.errors(o, outs[0])
        assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL, (rel, mx)


def test_config3_7b_75pct_ragged_paged_b64(ek):
    _run(ek, gen.LLAMA7B_75_PAGED, 8, two_step_append=True)


def test_config4_13b_75pct_b32_ctx16384(ek):
    _run(ek, gen.LLAMA13B_75, 8)


@pytest.mark.parametrize("w", [gen.SWEEP_50, gen.SWEEP_75, gen.SWEEP_875], ids=["50pct", "75pct", "87.5pct"])
def test_config5_sweep_b32_ctx8192(ek, w):
    _run(ek, w, 8)


def test_config5_prefill_append_4096_tokens_bit_exact(ek):
    """A 4096-token prefill append into a paged cache: every written row checked against the
    float32 bit model with a caller-supplied table; every other row untouched."""
    from oracle import elitekv_oracle as O
    w = replace(gen.SWEEP_75, B=2, ctx=4096, paged=True, seed=1777)
    table32 = torch.from_numpy(O.rope_table_f32(4100, w.d_h, w.rope_base)).cuda()
    st = H.setup(w, lens=[4096, 700], cos_sin=table32, fill=False)
    st.rope_plane.fill_(1.5)
    st.latent_plane.fill_(-2.0)
    rope0, lat0 = H.bits(st.rope_plane), H.bits(st.latent_plane)
    ek.elitekv_append(st.layer, st.cache, st.k_e, st.c, st.seq_id, st.pos)
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == 0
    rope_exp, lat_exp = O.append_expected(rope0, lat0, H.bits(st.k_e), H.bits(st.c), st.seq_id.cpu().numpy(),
                                          st.pos.cpu().numpy(), st.idx.numpy(), w.d_h, base=w.rope_base,
                                          page_table=st.page_table.cpu().numpy(), page_size=w.page_size,
                                          table32=table32.cpu().numpy())
    assert np.array_equal(H.bits(st.latent_plane), lat_exp)
    assert np.array_equal(H.bits(st.rope_plane), rope_exp)


def test_separated_latents_b32_ctx8192(ek):
    """The sweep's S-LRD configuration (key latent 512, value latent 1024) at full size."""
    _run(ek, gen.SWEEP_75_SLRD, 8)


def test_query_rows_on_the_benchmark_workload(ek):
    """Four causal query rows per sequence over the benchmark workload's cache (the shape
    bench.py times for elitekv_attend_rows): sampled (sequence, head) units, all four rows each,
    against the oracle's causal definition at full context."""
    from oracle import elitekv_oracle as O
    w, m = gen.LLAMA7B_75, 4
    st = H.setup(w)
    g = torch.Generator(device="cpu").manual_seed(77)
    q = torch.randn((w.B, m, w.n_h, w.d_h), generator=g).to(torch.bfloat16).cuda()
    q_pos = (st.lens_dev.view(-1, 1) - m + torch.arange(m, device="cuda", dtype=torch.int32).view(1, m)).to(torch.int32)
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, q.view(w.B * m, w.n_h, w.d_h), q_pos.reshape(-1).contiguous())
    ws = torch.empty(ek.elitekv_attend_rows_workspace_size(st.layer, w.B, m), dtype=torch.uint8, device="cuda")
    out = ek.elitekv_attend_rows(st.layer, st.cache, q_rope, q_abs, st.lens_dev, m, ws)
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == 0
    assert torch.isfinite(out.float()).all()
    idx = st.idx.numpy().astype(np.int64)
    W_uk, W_uv = H.f64(st.W_uk), H.f64(st.W_uv)
    for b, h in H.sample_units(st, 6, seed=21):
        lo, hi = int(st.starts[b]), int(st.starts[b + 1])
        n = hi - lo
        key_pos = np.arange(n)
        k_rope = O.rotate_elite_keys(H.f64(st.k_e[lo:hi]), key_pos, idx, w.d_h, w.rope_base)
        want = O.attend_causal(H.f64(q[b]), n - m + np.arange(m), k_rope, key_pos, H.f64(st.c[lo:hi]), W_uk, W_uv,
                               idx, w.d_h, base=w.rope_base, heads=[h])[:, 0]
        rel, mx = H.errors(H.f64(out[b, :, h]), want)
        assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL, (b, h, rel, mx)
    del st, out
    _free()
