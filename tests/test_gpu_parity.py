"""GPU parity: the CUDA library, called through its C ABI, against the float64 oracle on the
same seeded bytes.  Integer/layout work must match bit for bit; floating-point outputs within
relative L2 error 1e-2 and max abs error 3e-2 (bf16 inputs, fp32 accumulation)."""
import ctypes as C
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


SMALL = gen.Workload("small", n_h=6, d_h=32, r=3, d_c=72, d=192, B=3, ctx=150, seed=41)


# ------------------------------------------------------------------ append
@pytest.mark.parametrize("paged", [False, True])
def test_append_layout_and_bits(ek, paged):
    w = replace(SMALL, paged=paged, page_size=16, seed=42 + paged)
    lens = [37, 1, 100]
    table32 = torch.from_numpy(O.rope_table_f32(128, w.d_h, w.rope_base)).cuda()
    st = H.setup(w, lens=lens, cos_sin=table32, fill=False)
    # canary pattern in both planes; append must touch only the addressed rows
    g = torch.Generator(device="cpu").manual_seed(5)
    rope0 = torch.randint(0, 2 ** 15, tuple(st.rope_plane.shape), generator=g, dtype=torch.int16)
    lat0 = torch.randint(0, 2 ** 15, tuple(st.latent_plane.shape), generator=g, dtype=torch.int16)
    st.rope_plane.copy_(rope0.view(torch.bfloat16))
    st.latent_plane.copy_(lat0.view(torch.bfloat16))
    # append in two calls with a shuffled token order
    N = st.c.shape[0]
    perm = torch.randperm(N, generator=g).cuda()
    half = N // 2
    for sel in (perm[:half], perm[half:]):
        ek.elitekv_append(st.layer, st.cache, st.k_e[sel].contiguous(), st.c[sel].contiguous(),
                          st.seq_id[sel].contiguous(), st.pos[sel].contiguous())
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == 0
    pt = st.page_table.cpu().numpy() if paged else None
    max_ctx = st.cache.max_ctx if not paged else None
    rope_exp, lat_exp = O.append_expected(
        rope0.numpy().view(np.uint16), lat0.numpy().view(np.uint16), H.bits(st.k_e), H.bits(st.c),
        st.seq_id.cpu().numpy(), st.pos.cpu().numpy(), st.idx.numpy(), w.d_h, base=w.rope_base,
        max_ctx=max_ctx, page_table=pt, page_size=w.page_size, table32=table32.cpu().numpy())
    assert np.array_equal(H.bits(st.latent_plane), lat_exp)
    assert np.array_equal(H.bits(st.rope_plane), rope_exp)


@pytest.mark.parametrize("paged", [False, True])
def test_append_prefill_sized_call_bits(ek, paged):
    """A call of thousands of tokens takes the staged form (groups of tokens through a
    shared-memory ring with bulk copies).  7B shape, 4200 tokens in shuffled order in one call
    (groups of 8: a ragged last group), a token with a position outside the table in the middle:
    reported, not written, everything else bit for bit as the oracle's append says."""
    w = replace(gen.shrink(gen.LLAMA7B_75, B=3, ctx=2100), paged=paged, seed=48 + paged)
    lens = [2100, 2000, 100]
    table32 = torch.from_numpy(O.rope_table_f32(2104, w.d_h, w.rope_base)).cuda()
    st = H.setup(w, lens=lens, cos_sin=table32, fill=False)
    g = torch.Generator(device="cpu").manual_seed(6)
    rope0 = torch.randint(0, 2 ** 15, tuple(st.rope_plane.shape), generator=g, dtype=torch.int16)
    lat0 = torch.randint(0, 2 ** 15, tuple(st.latent_plane.shape), generator=g, dtype=torch.int16)
    st.rope_plane.copy_(rope0.view(torch.bfloat16))
    st.latent_plane.copy_(lat0.view(torch.bfloat16))
    N = st.c.shape[0]
    assert N == 4200
    perm = torch.randperm(N, generator=g).cuda()
    pos = st.pos[perm].contiguous()
    bad = 1234
    good = torch.ones(N, dtype=torch.bool)
    good[bad] = False
    pos_bad = pos.clone()
    pos_bad[bad] = 1_000_000
    ek.elitekv_append(st.layer, st.cache, st.k_e[perm].contiguous(), st.c[perm].contiguous(),
                      st.seq_id[perm].contiguous(), pos_bad)
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == ek.ERR_BAD_POSITION
    sel = perm.cpu()[good]
    pt = st.page_table.cpu().numpy() if paged else None
    max_ctx = st.cache.max_ctx if not paged else None
    rope_exp, lat_exp = O.append_expected(
        rope0.numpy().view(np.uint16), lat0.numpy().view(np.uint16), H.bits(st.k_e)[sel], H.bits(st.c)[sel],
        st.seq_id.cpu().numpy()[sel], st.pos.cpu().numpy()[sel], st.idx.numpy(), w.d_h, base=w.rope_base,
        max_ctx=max_ctx, page_table=pt, page_size=w.page_size, table32=table32.cpu().numpy())
    assert np.array_equal(H.bits(st.latent_plane), lat_exp)
    assert np.array_equal(H.bits(st.rope_plane), rope_exp)


def test_append_own_table_within_one_ulp(ek):
    w = replace(SMALL, seed=44)
    st = H.setup(w, lens=[64, 65, 129])
    torch.cuda.synchronize()
    rope0 = np.zeros(tuple(st.rope_plane.shape), dtype=np.uint16)
    lat0 = np.zeros(tuple(st.latent_plane.shape), dtype=np.uint16)
    rope_exp, lat_exp = O.append_expected(rope0, lat0, H.bits(st.k_e), H.bits(st.c),
                                          st.seq_id.cpu().numpy(), st.pos.cpu().numpy(),
                                          st.idx.numpy(), w.d_h, base=w.rope_base,
                                          max_ctx=st.cache.max_ctx)
    assert np.array_equal(H.bits(st.latent_plane), lat_exp)
    got = H.bits(st.rope_plane).astype(np.int32)
    # same sign/exponent neighbourhood: compare as ordered integers of the magnitude
    assert np.max(np.abs(got - rope_exp.astype(np.int32))) <= 1
    # rows never written stay zero
    written = O.token_slot(st.seq_id.cpu().numpy(), st.pos.cpu().numpy(), max_ctx=st.cache.max_ctx)
    mask = np.ones(got.shape[0], dtype=bool)
    mask[written] = False
    assert not got[mask].any()


def test_append_bad_position_is_reported_not_written(ek):
    w = replace(SMALL, seed=45)
    st = H.setup(w, lens=[4, 4, 4], fill=False)
    k_e, c = gen.tokens(w, 2, "cuda")
    seq = torch.tensor([0, 1], dtype=torch.int32, device="cuda")
    pos = torch.tensor([2, 10_000], dtype=torch.int32, device="cuda")
    ek.elitekv_append(st.layer, st.cache, k_e, c, seq, pos)
    assert ek.elitekv_check_status(st.layer) == ek.ERR_BAD_POSITION
    assert ek.elitekv_check_status(st.layer) == 0          # cleared by the read
    lat = H.bits(st.latent_plane)
    assert np.array_equal(lat[2], H.bits(c)[0])
    assert np.count_nonzero(lat.any(axis=1)) == 1


# ------------------------------------------------------------------ fused projection + append
def _projection_case(ek, w, d, lens, paged, seed):
    """Hidden states through elitekv_project_append into a canary-filled cache, against the
    float64 oracle: untouched rows stay bit for bit, written rows match the single-rounded float64
    result within bf16 rounding of an fp32-accumulated product."""
    w = replace(w, paged=paged, seed=seed)
    g = torch.Generator(device="cpu").manual_seed(seed)
    rope_w = w.n_h * 2 * w.r
    W_ke = (torch.randn(d, rope_w, generator=g) / d ** 0.5).to(torch.bfloat16).cuda()
    W_down = (torch.randn(d, w.d_c, generator=g) / d ** 0.5).to(torch.bfloat16).cuda()
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, "cuda")
    max_ctx = max(lens) + 1
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, max_ctx + 1, W_ke=W_ke, W_down=W_down)
    lens_t = torch.tensor(lens, dtype=torch.int32)
    B = len(lens)
    if paged:
        table, num_pages = gen.page_table(replace(w, B=B), lens_t, headroom_tokens=1)
        rows, page_table, mc = num_pages * w.page_size, table.cuda(), 0
    else:
        rows, page_table, mc = B * max_ctx, None, max_ctx
    rope0 = torch.randint(0, 2 ** 15, (rows, rope_w), generator=g, dtype=torch.int16)
    lat0 = torch.randint(0, 2 ** 15, (rows, w.d_c), generator=g, dtype=torch.int16)
    rope_plane = rope0.view(torch.bfloat16).cuda()
    latent_plane = lat0.view(torch.bfloat16).cuda()
    cache = ek.make_cache(rope_plane, latent_plane, n_seqs=B, max_ctx=mc, page_table=page_table, page_size=w.page_size)
    T = int(sum(lens))
    x = torch.randn(T, d, generator=g).to(torch.bfloat16).cuda()
    seq = torch.repeat_interleave(torch.arange(B, dtype=torch.int32), lens_t.to(torch.int64))
    pos = torch.cat([torch.arange(n, dtype=torch.int32) for n in lens])
    perm = torch.randperm(T, generator=g)
    ek.elitekv_project_append(layer, cache, x[perm.cuda()].contiguous(), seq[perm].cuda(), pos[perm].cuda())
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(layer) == 0
    exp_r, exp_l, rows64, c64 = O.project_append_expected(
        rope0.numpy().view(np.uint16), lat0.numpy().view(np.uint16), H.f64(x), H.f64(W_ke), H.f64(W_down),
        seq.numpy(), pos.numpy(), idx.numpy(), w.d_h, base=w.rope_base, max_ctx=mc if not paged else None,
        page_table=page_table.cpu().numpy() if paged else None, page_size=w.page_size)
    slot = O.token_slot(seq.numpy(), pos.numpy(), max_ctx=mc if not paged else None,
                        page_table=page_table.cpu().numpy() if paged else None, page_size=w.page_size)
    got_r, got_l = H.bits(rope_plane), H.bits(latent_plane)
    untouched = np.ones(rows, dtype=bool)
    untouched[slot] = False
    assert np.array_equal(got_r[untouched], rope0.numpy().view(np.uint16)[untouched])
    assert np.array_equal(got_l[untouched], lat0.numpy().view(np.uint16)[untouched])
    for got, want in ((O.bf16_bits_to_f64(got_r[slot]), rows64), (O.bf16_bits_to_f64(got_l[slot]), c64)):
        # one bf16 rounding (2^-9 relative) plus fp32 accumulation over d terms
        assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -8 + 2e-5 * d ** 0.5), float(np.max(np.abs(got - want)))
        rel = np.linalg.norm(got - want) / np.linalg.norm(want)
        assert rel < 3e-3, rel


@pytest.mark.parametrize("paged", [False, True])
def test_project_append_7b_shape(ek, paged):
    """d = 4096: 64 depth stages through a 4-stage ring; 700 tokens = 5 full token tiles and a
    ragged sixth; rope part 4 column tiles, latent part 12."""
    _projection_case(ek, gen.shrink(gen.LLAMA7B_75, B=3, ctx=400), 4096, [400, 237, 63], paged, 91 + paged)


def test_project_append_other_shapes(ek):
    _projection_case(ek, gen.shrink(gen.SWEEP_875, B=2, ctx=100), 1024, [100, 29], False, 93)
    _projection_case(ek, gen.shrink(gen.LLAMA13B_75, B=2, ctx=140), 5120, [1, 140], False, 94)


@pytest.mark.parametrize("paged", [False, True])
@pytest.mark.parametrize("lens", [[1] * 16, [40, 37, 51], [1], [17, 100]], ids=["b16", "128tok", "1tok", "117tok"])
def test_project_append_decode_batches_split_depth(ek, lens, paged):
    """At most 128 tokens (a decode step's batch): the call runs as clusters of 8 blocks that
    split the depth d and exchange partial sums through distributed shared memory.  One token,
    a batch of 16 one-token sequences, a full tile of 128 and a ragged 117 (the rows a block
    finishes, 16 per block, end inside block 7)."""
    _projection_case(ek, gen.shrink(gen.LLAMA7B_75, B=len(lens), ctx=max(lens) + 1), 4096, lens, paged, 96 + paged)


def test_project_append_split_depth_uneven_shares(ek):
    """d = 5120: 80 depth stages over 8 blocks (10 each); d = 1024 at d_c = 768: 16 stages, 2 each;
    d = 576: 9 stages, shares of 1 and 2."""
    _projection_case(ek, gen.shrink(gen.LLAMA13B_75, B=2, ctx=30), 5120, [30, 9], False, 97)
    _projection_case(ek, gen.shrink(gen.SWEEP_875, B=2, ctx=60), 1024, [60, 60], False, 98)
    _projection_case(ek, gen.shrink(gen.SWEEP_875, B=1, ctx=5), 576, [5], False, 99)


@pytest.mark.parametrize("paged", [False, True])
def test_project_append_prefill_sized_call(ek, paged):
    """1000+ tokens with an output width of whole 256-column tiles take the 256 x 256 form (two
    accumulators sharing every weight tile).  7B shape: 1400 tokens = 5 full token tiles and a
    ragged sixth, shuffled order."""
    _projection_case(ek, gen.shrink(gen.LLAMA7B_75, B=3, ctx=1000), 4096, [1000, 337, 63], paged, 101 + paged)


def test_project_append_prefill_form_rope_boundary_inside_a_tile(ek):
    """13B shape: 640 rope columns + 1920 latent columns = ten 256-column tiles, the third of
    which holds rope columns and latent columns side by side."""
    _projection_case(ek, gen.shrink(gen.LLAMA13B_75, B=2, ctx=900), 5120, [900, 300], False, 103)


def test_project_append_needs_projection_weights_and_a_covered_shape(ek):
    w = replace(SMALL, seed=95)
    st = H.setup(w, lens=[5, 5, 5])
    x = torch.zeros((2, 192), dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(2, dtype=torch.int32, device="cuda")
    with pytest.raises(ek.ElitekvError) as e:          # layer without W_ke / W_down
        ek.elitekv_project_append(st.layer, st.cache, x, z, z)
    assert e.value.code == ek.ERR_INVALID_ARG
    W_ke = torch.zeros((192, w.n_h * 2 * w.r), dtype=torch.bfloat16, device="cuda")
    W_down = torch.zeros((192, w.d_c), dtype=torch.bfloat16, device="cuda")
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, st.idx, st.W_uk, st.W_uv, 64, W_ke=W_ke, W_down=W_down)
    with pytest.raises(ek.ElitekvError) as e:          # 36 rope columns and d_c = 72: not 128-column tiles
        ek.elitekv_project_append(layer, st.cache, x, z, z)
    assert e.value.code == ek.ERR_UNSUPPORTED_SHAPE


# ------------------------------------------------------------------ separated latents (S-LRD)
@pytest.mark.parametrize("kernel", [1, 2], ids=["generic", "two-pass"])
@pytest.mark.parametrize("d_ck", [512, 1024, 128])
@pytest.mark.parametrize("paged", [False, True])
def test_decode_separated_latents_7b_shape(ek, kernel, d_ck, paged):
    """S-LRD (Section 3.2) at the 7B 75 % cache size: a latent row is [c_k (d_ck) | c_v (1536 - d_ck)],
    scores read c_k through B^k_S, outputs read c_v through B^v_S.  All (sequence, head) units
    against the float64 oracle; several tiles, ragged tails, a one-token and an empty sequence."""
    w = gen.shrink(gen.LLAMA7B_75, B=5, ctx=700)
    if paged:
        w = replace(w, paged=True, page_size=64)
    st = H.setup(w, lens=[700, 385, 128, 1, 0], decode_kernel=kernel, d_ck=d_ck)
    assert ek.elitekv_decode_plan_info(st.layer, st.cache, 5)[0] == kernel
    out = H.run_decode(st)
    assert not out[4].any()
    H.check_parity(st, out, [(b, h) for b in range(4) for h in range(w.n_h)])


def test_decode_separated_latents_choice_and_other_shapes(ek):
    """Left to itself the library serves separated latents with the two-pass kernel (nothing is
    read twice there); the resident-tile kernel refuses them; widths the tensor-core kernel does
    not cover (multiples of 8, not of 128) go to the generic kernel.  13B-like: 40 heads."""
    w = gen.shrink(gen.LLAMA7B_75, B=2, ctx=300)
    st = H.setup(w, lens=[300, 77], d_ck=768)
    assert ek.elitekv_decode_plan_info(st.layer, st.cache, 2)[0] == 2
    H.check_parity(st, H.run_decode(st), H.sample_units(st, 24, seed=2))
    with pytest.raises(ek.ElitekvError) as e:
        H.run_decode(H.setup(w, lens=[300, 77], d_ck=768, decode_kernel=3))
    assert e.value.code == ek.ERR_UNSUPPORTED_SHAPE
    st = H.setup(w, lens=[300, 77], d_ck=200)
    assert ek.elitekv_decode_plan_info(st.layer, st.cache, 2)[0] == 1
    H.check_parity(st, H.run_decode(st), H.sample_units(st, 24, seed=3))
    w13 = gen.shrink(gen.LLAMA13B_75, B=2, ctx=260)
    st = H.setup(w13, lens=[260, 129], d_ck=640)
    H.check_parity(st, H.run_decode(st), H.sample_units(st, 40, seed=4))


def test_separated_latents_bad_widths_are_rejected(ek):
    w = gen.shrink(gen.LLAMA7B_75, B=1, ctx=10)
    for d_ck, code in ((1536, "ERR_INVALID_ARG"), (-8, "ERR_INVALID_ARG"), (100, "ERR_UNSUPPORTED_SHAPE")):
        with pytest.raises(ek.ElitekvError) as e:
            H.setup(w, lens=[10], d_ck=d_ck, fill=False)
        assert e.value.code == getattr(ek, code)


# ------------------------------------------------------------------ query preparation
@pytest.mark.parametrize("pair_mode", [0, 1])
def test_absorb_query(ek, pair_mode):
    w = replace(SMALL, B=19, seed=46)
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, "cuda")
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, 4096, pair_mode=pair_mode)
    q = gen.queries(w, "cuda")
    q_pos = torch.randint(0, 4096, (w.B,), dtype=torch.int32).cuda()
    q_rope, q_abs = ek.elitekv_absorb_query(layer, q, q_pos)
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(layer) == 0
    for b in range(w.B):
        r_ref, a_ref = O.absorb_query(H.f64(q[b]), int(q_pos[b]), idx.numpy(), H.f64(W_uk), w.d_h,
                                      w.rope_base, pair_mode)
        # bf16 output of an fp32 computation: half an ulp plus accumulation noise
        assert np.all(np.abs(H.f64(q_rope[b]) - r_ref) <= np.abs(r_ref) * 2.0 ** -8 + 1e-6)
        assert np.all(np.abs(H.f64(q_abs[b]) - a_ref) <= np.abs(a_ref) * 2.0 ** -8 + 1e-4)


# ------------------------------------------------------------------ decode
def test_decode_tiny_config_all_units(ek):
    """Configuration 1: the whole chain from hidden states, every (sequence, head) unit."""
    w = gen.TINY
    st = H.setup(w, fill=False)
    idx = st.idx
    q_all, k_e, c = gen.projected_chain(w, idx, w.ctx)
    st.k_e, st.c = k_e.cuda(), c.cuda()
    st.q = q_all[-1:].contiguous().cuda()
    ek.elitekv_append(st.layer, st.cache, st.k_e, st.c, st.seq_id, st.pos)
    out = H.run_decode(st)
    rel, mx = H.check_parity(st, out, H.all_units(st))
    assert rel < 5e-3


CASES = [
    # name, workload, lens
    ("ragged", replace(SMALL, seed=51), [150, 1, 77]),
    ("tile-edges", replace(SMALL, seed=52), [64, 65, 63]),
    ("paged", replace(SMALL, paged=True, page_size=64, seed=53), [130, 64, 1]),
    ("paged-small-pages", replace(SMALL, paged=True, page_size=16, seed=54), [100, 17, 48]),
    ("one-head-odd", gen.Workload("odd", n_h=1, d_h=8, r=1, d_c=8, d=8, B=2, ctx=20, seed=55), [20, 3]),
    ("nine-heads", gen.Workload("nine", n_h=9, d_h=64, r=4, d_c=264, d=576, B=2, ctx=90, seed=56), [90, 33]),
    ("no-rope", gen.Workload("r0", n_h=4, d_h=16, r=0, d_c=40, d=64, B=2, ctx=50, seed=57), [50, 9]),
    ("all-rope", gen.Workload("rfull", n_h=4, d_h=16, r=8, d_c=64, d=64, B=2, ctx=50, seed=58), [50, 9]),
    ("wide-latent", gen.Workload("wide", n_h=2, d_h=32, r=2, d_c=3072, d=3072, B=1, ctx=70, seed=59), [70]),
]


@pytest.mark.parametrize("name,w,lens", CASES, ids=[c[0] for c in CASES])
def test_decode_small_cases(ek, name, w, lens):
    st = H.setup(w, lens=lens)
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


def test_decode_empty_sequence_gives_zero_row(ek):
    w = replace(SMALL, seed=60)
    st = H.setup(w, lens=[40, 0, 5])
    out = H.run_decode(st)
    assert not H.bits(out[1]).any()
    H.check_parity(st, out, [(b, h) for b in (0, 2) for h in range(w.n_h)])


def test_decode_single_token_equals_up_projected_latent(ek):
    w = replace(SMALL, seed=61)
    st = H.setup(w, lens=[1, 1, 1])
    out = H.f64(H.run_decode(st))
    c, W_uv = H.f64(st.c), H.f64(st.W_uv)
    for b in range(3):
        want = (c[b] @ W_uv).reshape(w.n_h, w.d_h)
        assert np.max(np.abs(out[b] - want)) <= 2.0 ** -8 * np.max(np.abs(want)) + 1e-3


def test_decode_shift_invariance_on_gpu(ek):
    w = replace(SMALL, seed=62)
    a = H.f64(H.run_decode(H.setup(w, lens=[90, 20, 64])))
    b = H.f64(H.run_decode(H.setup(w, lens=[90, 20, 64], pos_offset=777)))
    rel, mx = H.errors(b, a)
    assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL


def test_decode_page_permutation_is_bit_identical(ek):
    """Where pages sit physically must not matter: same logical cache, other permutation."""
    w1 = replace(SMALL, paged=True, seed=63)
    st1 = H.setup(w1, lens=[130, 70, 64])
    o1 = H.bits(H.run_decode(st1))
    # rebuild with the page table reversed, same tokens
    st2 = H.setup(w1, lens=[130, 70, 64], fill=False)
    num_pages = st2.cache.num_pages
    flipped = torch.where(st2.page_table >= 0, num_pages - 1 - st2.page_table, st2.page_table)
    st2.page_table.copy_(flipped)
    ek.elitekv_append(st2.layer, st2.cache, st2.k_e, st2.c, st2.seq_id, st2.pos)
    o2 = H.bits(H.run_decode(st2))
    assert np.array_equal(o1, o2)


def test_decode_7b_shape_small_context(ek):
    """Layer shape of configuration 2 at a context the oracle finishes quickly: spans several
    64-token tiles with ragged tails; all heads of every sequence."""
    w = gen.shrink(gen.LLAMA7B_75, B=3, ctx=700)
    st = H.setup(w, lens=[700, 333, 65])
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


def test_decode_7b_shape_batch_not_a_multiple_of_16(ek):
    """37 sequences: the absorb and combine kernels work on chunks of 16 sequences (one MMA row
    tile), so the last chunk has 5 live rows; lengths from 1 token to a few tiles."""
    B = 37
    lens = [1 + (53 * i * i + 17 * i) % 330 for i in range(B)]
    w = gen.shrink(gen.LLAMA7B_75, B=B, ctx=max(lens))
    st = H.setup(w, lens=lens)
    out = H.run_decode(st)
    assert torch.isfinite(out.float()).all()
    H.check_parity(st, out, H.sample_units(st, 96, seed=3))


def test_step_replays_from_a_cuda_graph(ek):
    """The calls only enqueue work and read lengths, positions and the plan on the device, so a
    step (query preparation + attention, programmatic launches included) can be captured once
    and replayed; after the queries change in place the replay gives the new result."""
    w = gen.shrink(gen.LLAMA7B_75, B=4, ctx=600)
    st = H.setup(w, lens=[600, 257, 128, 31])
    eager1 = H.run_decode(st).clone()
    q_live = st.q.clone()
    q_rope = torch.empty((4, w.n_h, 2 * w.r), dtype=torch.bfloat16, device="cuda")
    q_abs = torch.empty((4, w.n_h, w.d_c), dtype=torch.bfloat16, device="cuda")
    out = torch.empty((4, w.n_h, w.d_h), dtype=torch.bfloat16, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(2):   # warm-up outside capture (attribute calls, lazy module loading)
            ek.elitekv_absorb_query(st.layer, q_live, st.q_pos, q_rope, q_abs)
            ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, st.lens_dev, st.workspace, out)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ek.elitekv_absorb_query(st.layer, q_live, st.q_pos, q_rope, q_abs)
        ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, st.lens_dev, st.workspace, out)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager1)
    q2 = torch.flip(st.q, dims=[1]).contiguous()
    eager2 = H.run_decode(replace(st, q=q2)).clone()
    q_live.copy_(q2)
    graph.replay()
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == 0
    assert torch.equal(out, eager2)


def test_back_to_back_steps_share_one_workspace(ek):
    """Two steps queued without a synchronisation in between, same workspace, different queries:
    the plan / split-K / combine kernels of the second step are launched with programmatic
    serialisation, so they must still wait for the first step's combine before they touch the
    shared plan arrays and partial results.  Each output must equal the one the same step gives
    when run alone, bit for bit, and match the oracle."""
    w = gen.shrink(gen.LLAMA7B_75, B=4, ctx=900)
    st = H.setup(w, lens=[900, 641, 130, 64])
    q2 = torch.flip(st.q, dims=[0]).contiguous()
    alone1 = H.run_decode(st).clone()
    st2 = replace(st, q=q2)
    alone2 = H.run_decode(st2).clone()
    for _ in range(5):
        qr1, qa1 = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
        o1 = ek.elitekv_decode(st.layer, st.cache, qr1, qa1, st.lens_dev, st.workspace)
        qr2, qa2 = ek.elitekv_absorb_query(st.layer, q2, st.q_pos)
        o2 = ek.elitekv_decode(st.layer, st.cache, qr2, qa2, st.lens_dev, st.workspace)
        torch.cuda.synchronize()
        assert ek.elitekv_check_status(st.layer) == 0
        assert torch.equal(o1, alone1)
        assert torch.equal(o2, alone2)
    H.check_parity(st, alone1, H.all_units(st))


def _step_state(ek, paged):
    """A cache filled up to, not including, the decoding tokens, and the step's own inputs."""
    w = gen.shrink(gen.LLAMA7B_75, B=4, ctx=700)
    if paged:
        w = replace(w, paged=True, page_size=64)
    lens = [700, 257, 129, 1]
    st = H.setup(w, lens=lens, fill=False)
    last = torch.tensor([int(st.starts[b + 1]) - 1 for b in range(4)], device="cuda")
    keep = torch.ones(int(st.starts[-1]), dtype=torch.bool, device="cuda")
    keep[last] = False
    ek.elitekv_append(st.layer, st.cache, st.k_e[keep], st.c[keep], st.seq_id[keep], st.pos[keep])
    new = {"k_e": st.k_e[last].contiguous(), "c": st.c[last].contiguous(),
           "seq_id": st.seq_id[last].contiguous(), "pos": st.pos[last].contiguous()}
    return w, st, new


@pytest.mark.parametrize("paged", [False, True])
def test_single_call_step_equals_the_three_calls(ek, paged):
    """elitekv_decode_step (append and plan on the layer's second stream, joined before the
    attention kernel) against append -> absorb -> decode on one stream: same cache rows, same
    output bits, several steps queued back to back without a synchronisation, and parity with the
    oracle from the raw inputs."""
    w, st, new = _step_state(ek, paged)
    q_rope = torch.empty((4, w.n_h, 2 * w.r), dtype=torch.bfloat16, device="cuda")
    q_abs = torch.empty((4, w.n_h, w.d_c), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((4, w.n_h, w.d_h), dtype=torch.bfloat16, device="cuda")
    for _ in range(3):
        ek.elitekv_decode_step(st.layer, st.cache, new["k_e"], new["c"], new["seq_id"], new["pos"], st.q,
                               st.lens_dev, q_rope, q_abs, st.workspace, out)
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == 0
    rope_rows, lat_rows = st.rope_plane.clone(), st.latent_plane.clone()
    # the three calls on a cache that is built the same way
    w2, st2, new2 = _step_state(ek, paged)
    ek.elitekv_append(st2.layer, st2.cache, new2["k_e"], new2["c"], new2["seq_id"], new2["pos"])
    want = H.run_decode(st2)
    assert torch.equal(st2.rope_plane, rope_rows) and torch.equal(st2.latent_plane, lat_rows)
    assert torch.equal(out, want)
    H.check_parity(st, out, H.sample_units(st, 48, seed=5))


def test_single_call_step_replays_from_a_cuda_graph(ek):
    """The fork to the layer's second stream and the join are event edges, so the whole step
    can be captured from the caller's stream alone."""
    w, st, new = _step_state(ek, False)
    q_live = st.q.clone()
    q_rope = torch.empty((4, w.n_h, 2 * w.r), dtype=torch.bfloat16, device="cuda")
    q_abs = torch.empty((4, w.n_h, w.d_c), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((4, w.n_h, w.d_h), dtype=torch.bfloat16, device="cuda")

    def one():
        ek.elitekv_decode_step(st.layer, st.cache, new["k_e"], new["c"], new["seq_id"], new["pos"], q_live,
                               st.lens_dev, q_rope, q_abs, st.workspace, out)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        one()
        one()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    eager = out.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        one()
    out.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, eager)
    q_live.copy_(torch.flip(st.q, dims=[1]))
    graph.replay()
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(st.layer) == 0
    want = H.run_decode(replace(st, q=q_live))
    assert torch.equal(out, want)


def test_step_runner_host_to_host(ek):
    """The host-to-host runner (one packed copy in, the single-call step, one copy out; eager and
    as a replayed CUDA graph) returns the bits of the same step made call by call."""
    w, st, new = _step_state(ek, False)
    runners = [ek.DecodeStepRunner(st.layer, st.cache, 4, "cuda", graph=g) for g in (False, True)]
    w2, st2, new2 = _step_state(ek, False)
    ek.elitekv_append(st2.layer, st2.cache, new2["k_e"], new2["c"], new2["seq_id"], new2["pos"])
    want = H.run_decode(st2).cpu()
    for r in runners:
        assert r.h2d_bytes >= sum(v.numel() * v.element_size() for v in r.host.values())
        for k, v in (("k_e", new["k_e"]), ("c", new["c"]), ("seq_id", new["seq_id"]), ("pos", new["pos"]),
                     ("q", st.q), ("lens", st.lens_dev)):
            r.host[k].copy_(v.cpu().view(r.host[k].shape))
        for _ in range(3):       # eager, capture + replay, replay
            r.out_host.zero_()
            got = r.run()
            assert torch.equal(got, want)
    assert runners[0].graph is None and runners[1].graph is not None
    assert ek.elitekv_check_status(st.layer) == 0


KERNELS = [1, 2, 3]
KERNEL_IDS = ["generic", "two-pass", "resident"]
TC_KERNELS, TC_KERNEL_IDS = KERNELS[1:], KERNEL_IDS[1:]


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_decode_7b_shape_ragged_tails_both_kernels(ek, kernel):
    """Same inputs through the CUDA-core kernel and the tcgen05 kernel: lengths around the
    16-token MMA step and the 128-token tile."""
    w = gen.shrink(gen.LLAMA7B_75, B=8, ctx=400)
    st = H.setup(w, lens=[1, 15, 16, 17, 127, 128, 129, 400], decode_kernel=kernel)
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


@pytest.mark.parametrize("kernel", TC_KERNELS, ids=TC_KERNEL_IDS)
@pytest.mark.parametrize("page_size", [64, 128])
def test_decode_7b_shape_paged_tensor_core(ek, page_size, kernel):
    w = replace(gen.shrink(gen.LLAMA7B_75, B=3, ctx=700), paged=True, page_size=page_size)
    st = H.setup(w, lens=[700, 64, 193], decode_kernel=kernel)
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


@pytest.mark.parametrize("kernel", TC_KERNELS, ids=TC_KERNEL_IDS)
def test_tensor_core_kernels_many_items_per_worker(ek, kernel):
    """Many short sequences: workers walk several items, some of them a few tiles long, and
    sequences are cut at tile boundaries that fall anywhere."""
    w = gen.shrink(gen.LLAMA7B_75, B=300, ctx=300)
    lens = [1 + (37 * i) % 300 for i in range(300)]
    st = H.setup(w, lens=lens, decode_kernel=kernel)
    out = H.run_decode(st)
    assert torch.isfinite(out.float()).all()
    H.check_parity(st, out, H.sample_units(st, 96))


@pytest.mark.parametrize("kernel", TC_KERNELS, ids=TC_KERNEL_IDS)
def test_tensor_core_kernels_87_5pct_shape(ek, kernel):
    w = gen.shrink(gen.SWEEP_875, B=3, ctx=500)
    st = H.setup(w, lens=[500, 33, 160], decode_kernel=kernel)
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


# ------------------------------------------------------------------ faults the device reports
@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_decode_overlong_length_is_reported_and_clamped(ek, kernel):
    """A length beyond the rows a sequence owns must not reach into the next sequence's rows:
    the plan records BAD_POSITION (sequence, length), clamps, and the other sequences' outputs
    are bit for bit what they are without the fault."""
    w = gen.shrink(gen.LLAMA7B_75, B=3, ctx=200)
    st = H.setup(w, lens=[200, 150, 90], decode_kernel=kernel)
    good = H.run_decode(st).clone()
    bad_lens = st.lens_dev.clone()
    bad_lens[1] = st.cache.max_ctx + 77
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
    out = ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, bad_lens, st.workspace)
    assert ek.elitekv_check_status(st.layer) == ek.ERR_BAD_POSITION
    assert ek.elitekv_last_status_detail(st.layer)[:2] == (1, st.cache.max_ctx + 77)
    assert torch.equal(out[0], good[0]) and torch.equal(out[2], good[2])
    assert torch.isfinite(out.float()).all()
    assert torch.equal(H.run_decode(st), good)        # the layer is usable afterwards


@pytest.mark.parametrize("kernel", KERNELS, ids=KERNEL_IDS)
def test_decode_bad_page_id_is_reported(ek, kernel):
    w = replace(gen.shrink(gen.LLAMA7B_75, B=3, ctx=300), paged=True, page_size=64)
    st = H.setup(w, lens=[300, 200, 100], decode_kernel=kernel)
    good = H.run_decode(st).clone()
    keep = st.page_table[1, 1].item()
    st.page_table[1, 1] = st.cache.num_pages + 5
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
    out = ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, st.lens_dev, st.workspace)
    assert ek.elitekv_check_status(st.layer) == ek.ERR_BAD_PAGE
    assert ek.elitekv_last_status_detail(st.layer)[:2] == (1, st.cache.num_pages + 5)
    assert torch.equal(out[0], good[0]) and torch.equal(out[2], good[2])
    st.page_table[1, 1] = keep
    assert torch.equal(H.run_decode(st), good)


def test_bounded_waits_give_up_and_report(ek):
    """A wait that cannot complete must end with TIMEOUT in the status word, for every wait
    helper the tensor-core kernels use; the context stays usable."""
    w = gen.shrink(gen.LLAMA7B_75, B=2, ctx=200)
    st = H.setup(w, lens=[200, 67])
    good = H.run_decode(st).clone()
    for limit in (1, 100, 5000):
        ek.elitekv_selftest_bounded_wait(st.layer, limit)
        assert ek.elitekv_check_status(st.layer) == ek.ERR_TIMEOUT
        assert ek.elitekv_last_status_detail(st.layer) == (7, limit, 1)
    assert ek.elitekv_check_status(st.layer) == 0
    assert torch.equal(H.run_decode(st), good)


def test_tensor_core_kernel_refuses_uncovered_shapes(ek):
    w = replace(SMALL, seed=64)
    st = H.setup(w, lens=[5, 5, 5], decode_kernel=0)
    idx = gen.elite_index_sets(w)
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, st.W_uk, st.W_uv, 64, decode_kernel=2)
    with pytest.raises(ek.ElitekvError) as e:
        ek.elitekv_decode_workspace_size(layer, 3)
    assert e.value.code == ek.ERR_UNSUPPORTED_SHAPE


def test_decode_only_parity_from_the_gpu_cache(ek):
    """Decode in isolation: the oracle reads the rope rows the GPU appended (bf16, downloaded)
    instead of rotating the raw keys itself, so append rounding cannot mask a decode error."""
    w = gen.shrink(gen.LLAMA7B_75, B=2, ctx=300)
    lens = [300, 131]
    st = H.setup(w, lens=lens)
    out = H.f64(H.run_decode(st))
    W_uk, W_uv, idx = H.f64(st.W_uk), H.f64(st.W_uv), st.idx.numpy().astype(np.int64)
    max_ctx = st.cache.max_ctx
    for b, n in enumerate(lens):
        rows = slice(b * max_ctx, b * max_ctx + n)
        k_rope = H.f64(st.rope_plane[rows]).reshape(n, w.n_h, 2 * w.r)
        c = H.f64(st.latent_plane[rows])
        want = O.decode(H.f64(st.q[b]), n - 1, k_rope, c, W_uk, W_uv, idx, w.d_h, base=w.rope_base)
        rel, mx = H.errors(out[b], want)
        assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL, (b, rel, mx)


def test_decode_13b_shape_small_context(ek):
    w = gen.shrink(gen.LLAMA13B_75, B=2, ctx=300)
    st = H.setup(w, lens=[300, 129])
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


@pytest.mark.parametrize("w", [gen.SWEEP_50, gen.SWEEP_875], ids=["50pct", "87.5pct"])
def test_decode_sweep_shapes_small_context(ek, w):
    ws = gen.shrink(w, B=2, ctx=200)
    st = H.setup(ws, lens=[200, 70])
    out = H.run_decode(st)
    H.check_parity(st, out, H.all_units(st))


# ------------------------------------------------------------------ plan
@pytest.mark.parametrize("lens,max_items", [([1], 5), ([64, 65, 0, 1000], 9), ([4096] * 16, 164),
                                             (list(range(1, 300, 7)), 80), ([100000, 3], 40)])
def test_plan_partitions_every_sequence(ek, lens, max_items):
    t = torch.tensor(lens, dtype=torch.int32, device="cuda")
    max_items = max(max_items, len(lens) + 1)
    items, first = ek.elitekv_plan(t, 64, max_items)
    torch.cuda.synchronize()
    items, first = items.cpu().numpy(), first.cpu().numpy()
    assert first[0] == 0 and first[-1] <= max_items
    sizes = []
    for b, n in enumerate(lens):
        rows = items[first[b]:first[b + 1]]
        at = 0
        for s, t0, cnt, _ in rows:
            assert s == b and t0 == at and cnt > 0 and t0 % 64 == 0
            at += cnt
            sizes.append(cnt)
        assert at == n
    assert np.all(items[first[-1]:, 0] == -1)
    if sizes:   # near-equal pieces: no piece more than one tile above the ideal share
        total_tiles = sum((n + 63) // 64 for n in lens)
        budget = max_items - len(lens)
        target = max(1, -(-total_tiles // budget))
        assert max(sizes) <= target * 64


def _plan_cases():
    return [([4096] * 16, 128, 148), ([4096] * 16, 64, 148), ([1], 64, 148), ([64, 65, 0, 1000], 64, 7),
            (list(range(1, 3000, 37)), 128, 49), ([100000, 3], 64, 148), ([0, 0, 5], 128, 3),
            ([1024 + (7919 * i) % 31744 for i in range(64)], 64, 148)]


@pytest.mark.parametrize("overhead", [0, 1, 3])
@pytest.mark.parametrize("lens,tile,n_workers", _plan_cases())
def test_worker_plan_structure(ek, lens, tile, n_workers, overhead):
    """The persistent-worker plan.  The batch's tile list carries `overhead` empty tiles in front
    of every non-empty sequence; worker w owns positions [w*total/n, (w+1)*total/n) of that list, n = min(workers, total).
    Every sequence is partitioned into consecutive items that start on tile boundaries; items are
    ordered by worker and lie inside their worker's range; worker_first is monotone and covers
    all items; with overhead 0 every worker holds exactly the tiles of its range."""
    B = len(lens)
    t = torch.tensor(lens, dtype=torch.int32, device="cuda")
    max_items = B + n_workers
    items, first, wfirst = ek.elitekv_plan_workers(t, tile, n_workers, max_items, overhead)
    torch.cuda.synchronize()
    items, first, wfirst = items.cpu().numpy(), first.cpu().numpy(), wfirst.cpu().numpy()
    n_items = int(first[-1])
    assert first[0] == 0 and n_items <= max_items
    assert np.all(items[n_items:, 0] == -1)
    tiles_of = [(n + tile - 1) // tile for n in lens]
    slots_of = [k + overhead if k else 0 for k in tiles_of]
    total = max(1, sum(slots_of))
    n_used = min(n_workers, total)
    bound = [min(w, n_used) * total // n_used for w in range(n_workers + 1)]
    g0 = np.concatenate([[0], np.cumsum(slots_of)])
    # sequences: consecutive, tile-aligned, complete
    for b, n in enumerate(lens):
        at = 0
        for s, t0, cnt, wk in items[first[b]:first[b + 1]]:
            assert s == b and t0 == at and cnt > 0 and t0 % tile == 0
            at += cnt
        assert at == n
    # workers: monotone boundaries that cover all items; each item lies inside its worker's range
    assert wfirst[0] == 0 and wfirst[-1] == n_items and np.all(np.diff(wfirst) >= 0)
    per_worker = np.zeros(n_workers, dtype=np.int64)
    for w_id in range(n_workers):
        for s, t0, cnt, wk in items[wfirst[w_id]:wfirst[w_id + 1]]:
            assert wk == w_id
            ga = g0[s] + overhead + t0 // tile
            gb = g0[s] + overhead + (t0 + cnt + tile - 1) // tile
            assert bound[w_id] <= ga and gb <= bound[w_id + 1]
            per_worker[w_id] += gb - ga
    assert per_worker.sum() == sum(tiles_of)
    if overhead == 0 and sum(tiles_of) > 0:
        assert np.array_equal(per_worker, np.diff(bound))


# ------------------------------------------------------------------ comparator
@pytest.mark.parametrize("n_h,d_h,lens", [(3, 64, [100, 1, 64]), (32, 128, [300, 77]), (9, 16, [50, 0])])
def test_mha_comparator(ek, n_h, d_h, lens):
    B, max_ctx = len(lens), max(lens) + 3
    g = torch.Generator(device="cuda").manual_seed(7)
    q = torch.randn(B, n_h, d_h, generator=g, device="cuda").to(torch.bfloat16)
    K = torch.randn(B, max_ctx, n_h, d_h, generator=g, device="cuda").to(torch.bfloat16)
    V = torch.randn(B, max_ctx, n_h, d_h, generator=g, device="cuda").to(torch.bfloat16)
    ws = torch.empty(ek.elitekv_mha_workspace_size(B, n_h, d_h), dtype=torch.uint8, device="cuda")
    out = ek.elitekv_mha_decode(q, K, V, torch.tensor(lens, dtype=torch.int32, device="cuda"), ws)
    torch.cuda.synchronize()
    for b, n in enumerate(lens):
        want = O.mha_decode(H.f64(q[b]), H.f64(K[b, :n]), H.f64(V[b, :n]))
        rel, mx = H.errors(H.f64(out[b]), want)
        assert rel <= H.REL_L2_TOL and mx <= H.MAX_ABS_TOL


# ------------------------------------------------------------------ argument checking
def test_invalid_arguments_are_rejected_before_launch(ek):
    w = SMALL
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, "cuda")
    bad = idx.clone()
    bad[0, 1] = bad[0, 0]                      # duplicate chunk in one head
    with pytest.raises(ek.ElitekvError) as e:
        ek.Layer(w.n_h, w.d_h, w.r, w.d_c, bad, W_uk, W_uv, 64)
    assert e.value.code == ek.ERR_INVALID_ARG
    bad = idx.clone()
    bad[1, 0] = w.d_h // 2                     # out of range
    with pytest.raises(ek.ElitekvError):
        ek.Layer(w.n_h, w.d_h, w.r, w.d_c, bad, W_uk, W_uv, 64)
    with pytest.raises(ek.ElitekvError) as e:   # latent width not a multiple of 8
        ek.Layer(w.n_h, w.d_h, w.r, 76, idx, W_uk, W_uv, 64)
    assert e.value.code == ek.ERR_UNSUPPORTED_SHAPE
    st = H.setup(w, lens=[5, 5, 5])
    q_rope, q_abs = ek.elitekv_absorb_query(st.layer, st.q, st.q_pos)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(ek.ElitekvError) as e:
        ek.elitekv_decode(st.layer, st.cache, q_rope, q_abs, st.lens_dev, small)
    assert e.value.code == ek.ERR_WORKSPACE_TOO_SMALL
    lib = ek.lib()
    assert lib.elitekv_decode(None, None, None, None, None, 1, None, 0, None, None) == ek.ERR_INVALID_ARG
    assert lib.elitekv_append(None, None, None, None, None, None, 1, None) == ek.ERR_INVALID_ARG
