// Tensor-core split-K decode kernel for sm_100a (tcgen05 + TMEM + TMA).
//
// All heads of a layer read the SAME latent row (J-LRD, Section 3.2), so for one sequence the
// two latent contractions are dense GEMMs against a tile of T = 128 cached tokens:
//     S   [T x n_h]    = C[T x d_c] . Q_abs^T[d_c x n_h]          (score equation of Section
//                                                                   3.1 with B^k absorbed)
//     acc [d_c x n_h] += C^T[d_c x T] . P[T x n_h]                 (sum_t p_t c_t, Section 2.1;
//                                                                   B^v applied later)
// Both run as tcgen05.mma (M = 128, N = n_h, K = 16, bf16 in, fp32 accumulate in TMEM) straight
// from the 128-byte-swizzled shared-memory tiles that TMA writes; the narrow per-head rope dot
// product stays on FP32 FMA in the softmax threads.
//
// The absorbed queries of a sequence (n_h x d_c bf16, 96 KB at d_c = 1536) and a whole
// 128 x d_c token tile do not fit in shared memory together, so nothing is kept resident: the
// tile is streamed twice through a ring of slots, each slot holding one [128 tokens x 64 coords]
// latent chunk and, in pass A, the matching [n_h x 64] chunk of the absorbed queries (which
// stays L2-resident).  Pass A accumulates S over the latent axis, the softmax threads turn S
// (+ rope part) into P, pass B streams the same latent chunks again and accumulates P-weighted
// latents into the TMEM-resident output.  L2 eviction hints (keep after pass A, drop after pass
// B) make the second read an L2 hit, so HBM sees every cache byte once per step.
//
// With separated latents (S-LRD, Section 3.2: a latent row is [c_k | c_v]) pass A streams only
// the key latent's chunks and pass B only the value latent's, so nothing is read twice.
//
// Layers whose fp32 output is too wide for TMEM even with 32 heads (d_c = 3072) split the
// OUTPUT columns between two blocks instead of the heads: both blocks compute the scores of all
// 32 heads (pass A over the whole latent), each accumulates its half of the latent columns in
// pass B, so a block streams a tile one and a half times instead of twice.
//
// A block is a persistent worker: it walks the items of the balanced plan that fall into its
// share of the batch's tiles and writes one partial result (m, l, acc) per item.  Layers with
// more than 32 heads run as several head groups (and with 16 heads per block where even half the
// output is too wide for 32); the head groups of an item are
// adjacent blocks so that they share L2.
//
// Roles (288 threads):
//   warps 0,7,8  latent TMA producers (ring uses dealt round-robin)
//   warp 6       rope TMA producer
//   warp 1       TMEM allocation and MMA issue.  The tensor core finishes a 128 x N x 16 MMA in
//                about 40 clocks (the time to read the 4 KB A operand from shared memory); the
//                issuing code keeps up only when it runs warp-uniformly with the tcgen05.mma
//                itself under an elected lane and the descriptor words built from precomputed
//                halves plus small immediates (measured: 42 clocks per MMA, against 61 when a
//                single diverged lane runs the same loop and ~100 with per-MMA 64-bit
//                descriptor assembly).  The warp also zero-fills token rows past the end of
//                the sequence.  Producer warps issue TMA the same way.
//   warps 2-5    one thread per token row: rope dot products, S from TMEM, masking, running
//                max / sum in base 2 with a lazily moved reference max, P to shared memory in the
//                layout the second GEMM wants, TMEM rescale when the reference moves, epilogue
//                (output blocks transposed through shared memory and written by TMA stores)
// Every wait is bounded: when a limit is hit the block records ELITEKV_ERR_TIMEOUT in the
// layer's status word, stops issuing work, frees its TMEM and leaves.
#include "tc_ptx.cuh"

namespace {

constexpr int kTile = 128;            // tokens per tile
constexpr int kChunkBytes = 16384;    // [128 tokens][64 bf16] with 128-byte rows
constexpr int kLatSlots = 8;          // ring slots: one latent chunk + the matching query chunk each
constexpr int kRopeSlots = 3;
constexpr int kThreads = 288;         // warps 0,7,8 latent loads, 1 MMA, 2-5 softmax, 6 rope loads
constexpr int kProdWarps = 3;         // latent-load warps: 0, 7, 8
constexpr int kSoftmaxThreads = 128;
constexpr int kOutBufs = 12;          // [N heads][128 coords] fp32 staging tiles of the epilogue (ring + rope area)

struct TcArgs {
  const int32_t* items;
  const int32_t* worker_first;
  const int32_t* page_table;
  float* part_acc;
  float* part_ml;
  const bf16* q_rope;       // [B][n_h][2r]
  int32_t* status;
  long long max_ctx;
  long long num_pages;
  int page_shift, page_mask, max_pages_per_seq;
  int n_h, d_c;
  int kw, voff, vw;         // latent columns of the scores [0, kw) and of the outputs [voff, voff + vw)
  int n_groups;             // blocks per worker: query rows x head groups of N heads; blockIdx.x = worker * n_groups + group
  int rows, gpr, nv;        // query rows per sequence, head groups per row, rows * n_h
  int vparts;               // blocks that share a head group by splitting the OUTPUT columns between them
  const int32_t* seq_lens;  // rows > 1: row i of sequence b sees seq_lens[b] - (rows - 1 - i) tokens
  float scale_log2e;
};

struct __align__(8) TcBarriers {
  uint64_t lat_full[kLatSlots], lat_empty[kLatSlots];
  uint64_t rope_full[kRopeSlots], rope_empty[kRopeSlots];
  uint64_t s_full, p_ready, pv_done;
};

// shared-memory carve-up (offsets from a 1024-byte aligned base)
template <int N>
struct Smem {
  // a ring slot holds a latent chunk [128 tokens][64] and, behind it, the absorbed-query chunk
  // [N heads][64] of the same latent coordinates (used by pass A only)
  static constexpr int slot_bytes = kChunkBytes + N * 128;
  __host__ __device__ static constexpr int lat_off(int) { return 0; }
  __host__ __device__ static constexpr int rope_off(int d_c) { return lat_off(d_c) + kLatSlots * slot_bytes; }
  __host__ __device__ static constexpr int p_off(int d_c) { return rope_off(d_c) + kRopeSlots * kChunkBytes; }
  static constexpr int p_bytes = kTile * N * 2;
  __host__ __device__ static constexpr int misc_off(int d_c) { return p_off(d_c) + p_bytes; }
  // misc: q_rope fp32 [N][R2max=32] 4 KB | wmax [4][N] | corr [N] | barriers | tmem base | abort |
  // the two outcome words of the group waits
  static constexpr int misc_bytes = N * 32 * 4 + 4 * N * 4 + N * 4 + (int)sizeof(TcBarriers) + 64;
  __host__ __device__ static constexpr int total(int d_c) { return misc_off(d_c) + misc_bytes + 1024; }
};

template <int N, int R2>
__global__ void __launch_bounds__(kThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap map_lat, const __grid_constant__ CUtensorMap map_rope,
                 const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_lat128,
                 const __grid_constant__ CUtensorMap map_rope128, const __grid_constant__ CUtensorMap map_part,
                 const TcArgs a) {
  extern __shared__ unsigned char smem_raw[];
  const int worker = blockIdx.x / a.n_groups;         // persistent worker: walks its plan items
  const int grp = (blockIdx.x % a.n_groups) / a.vparts;
  const int vpart = (blockIdx.x % a.n_groups) % a.vparts;   // which share of the output columns this block accumulates
  const int qrow = grp / a.gpr;                       // query row of this block (0 when decoding)
  const int h0 = (grp % a.gpr) * N;                   // first head of this block's group
  const int vh0 = qrow * a.n_h + h0;                  // the same in the [rows][n_h] layout of queries and results
  const int nh_here = min(N, a.n_h - h0);
  const int d_c = a.d_c;
  const int NKC = a.kw >> 6;     // 64-wide latent chunks of pass A
  const int vw_blk = a.vw / a.vparts;                 // output columns of this block
  const int NB = vw_blk >> 7;    // 128-row output blocks = slot pairs of pass B
  const int NUSE = NKC + 2 * NB; // ring uses per tile
  const int vc0 = (a.voff + vpart * vw_blk) >> 6;     // first 64-wide chunk of the columns pass B reads
  const bool reread = a.voff == 0;   // joint latent: pass B reads what pass A read
  constexpr int NRB = N * R2 / 64;   // rope boxes per tile
  constexpr int HPB = 64 / R2;       // heads per rope box

  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  constexpr int kSlot = Smem<N>::slot_bytes;
  unsigned char* s_lat = base + Smem<N>::lat_off(d_c);
  unsigned char* s_rope = base + Smem<N>::rope_off(d_c);
  unsigned char* s_p = base + Smem<N>::p_off(d_c);
  unsigned char* s_misc = base + Smem<N>::misc_off(d_c);
  float* s_qrope = (float*)s_misc;                         // [N][R2]
  float* s_wmax = (float*)(s_misc + N * 32 * 4);           // [4][N]
  float* s_corr = s_wmax + 4 * N;                          // [N]
  TcBarriers* bars = (TcBarriers*)(s_corr + N);
  uint32_t* s_tmem = (uint32_t*)(bars + 1);
  volatile int* s_abort = (volatile int*)(s_tmem + 1);
  volatile int* s_verdict = s_abort + 1;     // [2] outcome words of the softmax threads' group waits

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_lat128) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_rope128) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_lat) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_rope) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_part) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kLatSlots; ++i) {
      mbar_init(smem_u32(&bars->lat_full[i]), 1);
      mbar_init(smem_u32(&bars->lat_empty[i]), 1);
    }
    for (int i = 0; i < kRopeSlots; ++i) {
      mbar_init(smem_u32(&bars->rope_full[i]), 1);
      mbar_init(smem_u32(&bars->rope_empty[i]), kSoftmaxThreads / 32);
    }
    mbar_init(smem_u32(&bars->s_full), 1);
    mbar_init(smem_u32(&bars->p_ready), kSoftmaxThreads);
    mbar_init(smem_u32(&bars->pv_done), 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  const int tmem_cols_needed = NB * N + N;
  uint32_t tmem_cols = 32;
  while ((int)tmem_cols < tmem_cols_needed) tmem_cols <<= 1;
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t tmem_s = tmem_base + NB * N;     // S columns after the NB output blocks
  // Everything above touched only this block's own state; the plan, the queries and the cache
  // come from kernels earlier in the stream.  A worker without items falls through to the
  // teardown (it has allocated tensor memory like everybody else).
  ekv_pdl_wait();
  ekv_pdl_trigger();
  const int item_lo = a.worker_first[worker], item_hi = a.worker_first[worker + 1];

  // running counters (each role advances its own copies identically): ring uses, tiles, items
  unsigned lat_n = 0, rope_n = 0, tbase = 0;
  unsigned gw_turn = 0;      // group waits taken so far by the softmax threads
  int seq = -1;
  for (int item = item_lo; item < item_hi; ++item) {
  seq = a.items[4 * item + 0];
  const int tok0 = a.items[4 * item + 1];
  const int ntok = a.items[4 * item + 2];
  const int n_tiles = (ntok + kTile - 1) / kTile;
  // rotated query chunks of this sequence as fp32 (broadcast operand of the rope dot products):
  // filled and used by the softmax warps only, so nobody else waits for it
  if (warp >= 2 && warp <= 5) {
    for (int e = threadIdx.x - 64; e < N * R2; e += kSoftmaxThreads) {
      const int h = e / R2;
      s_qrope[e] = h < nh_here ? __bfloat162float(a.q_rope[((size_t)seq * a.nv + vh0 + h) * R2 + (e % R2)]) : 0.f;
    }
    named_bar_sync(1, kSoftmaxThreads);
  }

  // ============================================================== warps 0, 7, 8: latent TMA producers; warp 6: rope
  // Each producer warp runs its loop warp-uniformly and one elected lane issues expect_tx and the
  // TMA loads.  One warp can issue a box only every ~0.17 us, so the latent ring uses are dealt
  // round-robin to kProdWarps warps.
  if (warp == 0 || warp >= 6) {
    const bool rope_role = warp == 6;
    const int prod = warp == 0 ? 0 : warp - 6;          // latent producer index
    // L2 priorities: a latent chunk read in pass A is read again soon (pass B) -> keep; after
    // pass B, and for rope rows, the data is dead -> first to go; the queries are re-read by
    // every tile of the sequence -> keep
    const uint64_t pol_keep = make_l2_policy_evict_last(), pol_drop = make_l2_policy_evict_first();
    bool ok = true;
    for (int tile = 0; tile < n_tiles && ok; ++tile) {
      // cache rows of the two 64-token halves of the tile; `whole` = adjacent (one 128-row box)
      const int t_abs = tok0 + tile * kTile;
      const int nvalid = min(kTile, ntok - tile * kTile);
      const int halves = nvalid > 64 ? 2 : 1;
      long long row[2];
      for (int hf = 0; hf < 2; ++hf) {
        const int t = t_abs + 64 * hf;
        if (a.page_table == nullptr) {
          row[hf] = (long long)seq * a.max_ctx + t;
        } else {
          const int pi = t >> a.page_shift;
          int page = (hf < halves && pi < a.max_pages_per_seq)
                         ? a.page_table[(long long)seq * a.max_pages_per_seq + pi] : 0;
          if (page < 0 || page >= a.num_pages) {
            if (hf < halves && rope_role && lane == 0) ekv_record(a.status, ELITEKV_ERR_BAD_PAGE, seq, page);
            page = 0;
          }
          row[hf] = ((long long)page << a.page_shift) + (t & a.page_mask);
        }
      }
      const bool whole = halves == 2 && row[1] == row[0] + 64;
      if (!rope_role) {
        // ring uses of this tile: NKC chunks of pass A (each with its query chunk), then the
        // 2 NB chunks of pass B (joint latent: the same chunks again, served by L2)
        for (int u = prod; u < NUSE; u += kProdWarps) {
          const bool with_q = u < NKC;
          const int kc = with_q ? u : vc0 + u - NKC;
          const unsigned n = lat_n + (unsigned)u, slot = n % kLatSlots;
          const uint32_t eb = smem_u32(&bars->lat_empty[slot]), epar = ((n / kLatSlots) & 1) ^ 1;
          ok = warp_wait(eb, epar, s_abort, 1);
          if (!ok) break;
          if (elect_one()) {
            const uint32_t fb = smem_u32(&bars->lat_full[slot]);
            mbar_expect_tx(fb, (uint32_t)(halves * 8192 + (with_q ? N * 128 : 0)));
            if (with_q)   // the sequence's absorbed queries for these 64 latent coordinates (L2-resident)
              tma_load_2d_hint(smem_u32(s_lat + slot * kSlot + kChunkBytes), &map_q, kc * 64, seq * a.nv + vh0, fb, pol_keep);
            const uint64_t pol = (with_q && reread) ? pol_keep : pol_drop;
            if (whole) {
              tma_load_2d_hint(smem_u32(s_lat + slot * kSlot), &map_lat128, kc * 64, (int)row[0], fb, pol);
            } else {
              for (int hf = 0; hf < halves; ++hf)
                tma_load_2d_hint(smem_u32(s_lat + slot * kSlot + hf * 8192), &map_lat, kc * 64, (int)row[hf], fb, pol);
            }
          }
          __syncwarp();
        }
        lat_n += (unsigned)NUSE;
      } else {
        // warp 6: the rope boxes of the tile
        for (int cb = 0; cb < NRB; ++cb) {
          const unsigned slot = rope_n % kRopeSlots;
          const uint32_t eb = smem_u32(&bars->rope_empty[slot]), epar = ((rope_n / kRopeSlots) & 1) ^ 1;
          ok = warp_wait(eb, epar, s_abort, 2);
          if (!ok) break;
          if (elect_one()) {
            const uint32_t fb = smem_u32(&bars->rope_full[slot]);
            mbar_expect_tx(fb, (uint32_t)(halves * 8192));
            if (whole) {
              tma_load_2d_hint(smem_u32(s_rope + slot * kChunkBytes), &map_rope128, h0 * R2 + cb * 64, (int)row[0], fb, pol_drop);
            } else {
              for (int hf = 0; hf < halves; ++hf)
                tma_load_2d_hint(smem_u32(s_rope + slot * kChunkBytes + hf * 8192), &map_rope, h0 * R2 + cb * 64, (int)row[hf], fb, pol_drop);
            }
          }
          __syncwarp();
          ++rope_n;
        }
      }
    }
  }
  // ============================================================== warp 1: MMA issuer
  // The whole warp walks the ring (waits, descriptor arithmetic, slot bookkeeping are
  // warp-uniform) and an elected lane issues the MMAs and the commits that free ring slots;
  // all lanes help to zero a ragged tail.
  else if (warp == 1) {
    constexpr uint32_t idesc_s = make_idesc(128, N, 0, 0);    // S = C . Q^T   (both K-major)
    constexpr uint32_t idesc_pv = make_idesc(128, N, 1, 1);   // acc = C^T . P (both MN-major)
    constexpr uint32_t hi_sw = desc_hi(1024, 2);              // 128-byte swizzle, 1024 bytes between 8-row groups
    constexpr uint32_t hi_p = desc_hi(2048, 0);               // P tile: no swizzle, 2048 bytes between 8-head groups
    constexpr uint32_t kSlot16 = kSlot >> 4;
    const uint32_t lat16 = smem_u32(s_lat) >> 4;              // ring base in 16-byte units
    const uint32_t lo_p = desc_lo(smem_u32(s_p), 128);
    const uint32_t full0 = smem_u32(&bars->lat_full[0]), empty0 = smem_u32(&bars->lat_empty[0]);
    bool ok = true;
    for (int tile = 0; tile < n_tiles && ok; ++tile) {
      const int nvalid = min(kTile, ntok - tile * kTile);
      const int ksteps = (nvalid + 15) >> 4;
      const int zero_from = nvalid, zero_to = ksteps * 16;
      const unsigned n0 = lat_n;                 // first ring use of this tile
      // ---- pass A: NKC chunks, 4 K-steps of 16 latent coordinates each
      unsigned slot = n0 % kLatSlots, par = (n0 / kLatSlots) & 1;
      for (int kc = 0; kc < NKC; ++kc) {
        const uint32_t fb = full0 + slot * 8;
        ok = warp_wait(fb, par, s_abort, 3);
        if (!ok) break;
        const uint32_t la = (lat16 + slot * kSlot16) | (1u << 16), lb = la + (kChunkBytes >> 4);
        if (elect_one()) {
          tc_mma_w(tmem_s, la, hi_sw, lb, hi_sw, idesc_s, kc != 0);
          tc_mma_w(tmem_s, la + 2, hi_sw, lb + 2, hi_sw, idesc_s, 1);     // +32 bytes along K per step
          tc_mma_w(tmem_s, la + 4, hi_sw, lb + 4, hi_sw, idesc_s, 1);
          tc_mma_w(tmem_s, la + 6, hi_sw, lb + 6, hi_sw, idesc_s, 1);
          tc_commit(empty0 + slot * 8);
        }
        __syncwarp();
        if (++slot == kLatSlots) { slot = 0; par ^= 1; }
      }
      if (!ok) break;
      if (elect_one()) tc_commit(smem_u32(&bars->s_full));
      __syncwarp();
      // ---- wait for P (and the rescaled output) of this tile
      ok = warp_wait(smem_u32(&bars->p_ready), (tbase + tile) & 1, s_abort, 4);
      if (!ok) break;
      tc_fence_after();
      // ---- pass B: NB output blocks of 128 latent coordinates = one even/odd slot pair each
      const unsigned nb0 = n0 + NKC;
      slot = nb0 % kLatSlots;
      par = (nb0 / kLatSlots) & 1;
      for (int blk = 0; blk < NB; ++blk) {
        const uint32_t fb = full0 + slot * 8;
        ok = warp_wait(fb, par, s_abort, 5) && warp_wait(fb + 8, par, s_abort, 5);
        if (!ok) break;
        if (zero_to > zero_from) {
          // ragged end of a sequence: rows past its last token inside the last 16-token step are
          // made exact zeros so that zero-probability rows cannot inject NaN/Inf bit patterns
          for (int e = lane; e < (zero_to - zero_from) * 16; e += 32) {
            const int rrow = zero_from + (e >> 4), c16 = e & 15;
            unsigned char* p = s_lat + (slot + (c16 >> 3)) * kSlot + rrow * 128 + (c16 & 7) * 16;
            *(uint4*)p = make_uint4(0, 0, 0, 0);
          }
          fence_proxy_async();
          __syncwarp();
        }
        // A: two 64-coordinate atoms one slot apart; +16 tokens = +2048 bytes in A, +256 bytes in P
        const uint32_t la = (lat16 + slot * kSlot16) | (kSlot16 << 16);
        const uint32_t d = tmem_base + blk * N;
        if (elect_one()) {
          if (ksteps == 8) {
            tc_mma_w(d, la, hi_sw, lo_p, hi_p, idesc_pv, tile != 0);
            tc_mma_w(d, la + 128, hi_sw, lo_p + 16, hi_p, idesc_pv, 1);
            tc_mma_w(d, la + 256, hi_sw, lo_p + 32, hi_p, idesc_pv, 1);
            tc_mma_w(d, la + 384, hi_sw, lo_p + 48, hi_p, idesc_pv, 1);
            tc_mma_w(d, la + 512, hi_sw, lo_p + 64, hi_p, idesc_pv, 1);
            tc_mma_w(d, la + 640, hi_sw, lo_p + 80, hi_p, idesc_pv, 1);
            tc_mma_w(d, la + 768, hi_sw, lo_p + 96, hi_p, idesc_pv, 1);
            tc_mma_w(d, la + 896, hi_sw, lo_p + 112, hi_p, idesc_pv, 1);
          } else {      // short last tile: only the loaded token rows
            for (int k = 0; k < ksteps; ++k)
              tc_mma_w(d, la + 128 * k, hi_sw, lo_p + 16 * k, hi_p, idesc_pv, (tile | k) != 0);
          }
          tc_commit(empty0 + slot * 8);
          tc_commit(empty0 + slot * 8 + 8);
        }
        __syncwarp();
        slot += 2;
        if (slot >= kLatSlots) { slot -= kLatSlots; par ^= 1; }
      }
      if (!ok) break;
      if (elect_one()) tc_commit(smem_u32(&bars->pv_done));
      __syncwarp();
      lat_n = n0 + (unsigned)NUSE;
    }
  }
  // ============================================================== warps 2-5: softmax
  else {
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may access
    const int trow = quarter * 32 + lane;         // token row inside the tile / output row inside a block
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    float l_part[N];                              // per-thread partial softmax denominators
#pragma unroll
    for (int h = 0; h < N; ++h) l_part[h] = 0.f;
    // lane h holds head h's reference max (N <= 32 per group).  With several query rows a row
    // may see nothing of an item (its causal limit lies before it): a finite start keeps
    // exp2(-inf - m_ref) at zero instead of NaN.
    float m_ref = a.rows > 1 ? -1e30f : -INFINITY;
    // tokens of this item the block's query row may see (causal rule; all of them when decoding)
    int vis = ntok;
    if (a.rows > 1) vis = max(0, min(ntok, a.seq_lens[seq] - (a.rows - 1 - qrow) - tok0));
    bool ok = true;
    const bool leader = threadIdx.x == 64;
    static_assert(N == 16 || N == 32, "softmax threads keep one head per lane (lanes >= N idle)");

    for (int tile = 0; tile < n_tiles && ok; ++tile) {
      const int nvis = min(kTile, vis - tile * kTile);     // rows of the tile this query row sees (may be <= 0)
      float s[N];
#pragma unroll
      for (int h = 0; h < N; ++h) s[h] = 0.f;
      // ---- rope part of the score (FP32 FMA)
#pragma unroll
      for (int cb = 0; cb < NRB; ++cb) {
        if (!ok) break;
        const unsigned slot = rope_n % kRopeSlots;
        ok = mbar_wait_group(smem_u32(&bars->rope_full[slot]), (rope_n / kRopeSlots) & 1, s_abort, s_verdict, gw_turn, leader, 2, kSoftmaxThreads, 6);
        if (!ok) break;
        const unsigned char* rowp = s_rope + slot * kChunkBytes + trow * 128;
        float part[HPB];
#pragma unroll
        for (int hh = 0; hh < HPB; ++hh) part[hh] = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          const uint4 v = *(const uint4*)(rowp + ((c ^ (trow & 7)) << 4));
          const bf162* k2 = (const bf162*)&v;
          const int hh = (c * 8) / R2;                       // head inside the box
          const float* qq = s_qrope + (cb * HPB + hh) * R2 + (c * 8) % R2;
          const float4 q0 = *(const float4*)qq, q1 = *(const float4*)(qq + 4);
          const float2 k0 = __bfloat1622float2(k2[0]), k1 = __bfloat1622float2(k2[1]);
          const float2 k2f = __bfloat1622float2(k2[2]), k3 = __bfloat1622float2(k2[3]);
          float acc = part[hh];
          acc = fmaf(q0.x, k0.x, acc); acc = fmaf(q0.y, k0.y, acc);
          acc = fmaf(q0.z, k1.x, acc); acc = fmaf(q0.w, k1.y, acc);
          acc = fmaf(q1.x, k2f.x, acc); acc = fmaf(q1.y, k2f.y, acc);
          acc = fmaf(q1.z, k3.x, acc); acc = fmaf(q1.w, k3.y, acc);
          part[hh] = acc;
        }
#pragma unroll
        for (int hh = 0; hh < HPB; ++hh) s[cb * HPB + hh] = part[hh];
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->rope_empty[slot]));
        ++rope_n;
      }
      if (!ok) break;
      // ---- latent part from TMEM
      ok = mbar_wait_group(smem_u32(&bars->s_full), (tbase + tile) & 1, s_abort, s_verdict, gw_turn, leader, 2, kSoftmaxThreads, 7);
      if (!ok) break;
      tc_fence_after();
      {
        float sv[N];
        tc_ld_cols<N>(tmem_s + lane_base, sv);
        tc_wait_ld();
#pragma unroll
        for (int h = 0; h < N; ++h) {
          const float x = (s[h] + sv[h]) * a.scale_log2e;
          s[h] = trow < nvis ? x : -INFINITY;
        }
      }
      // ---- per-head max over the 128 tokens of the tile
      float wm = -INFINITY;
#pragma unroll
      for (int h = 0; h < N; ++h) {
        const float v = ord2f(__reduce_max_sync(0xffffffffu, f2ord(s[h])));
        if (lane == h) wm = v;
      }
      if (lane < N) s_wmax[quarter * N + lane] = wm;
      named_bar_sync(1, kSoftmaxThreads);
      const int hl = lane & (N - 1);
      float tm = fmaxf(fmaxf(s_wmax[hl], s_wmax[N + hl]), fmaxf(s_wmax[2 * N + hl], s_wmax[3 * N + hl]));
      // reference max moves only when the tile max exceeds it by more than 2^8
      const bool move = tm > m_ref + 8.f;
      const float m_new = move ? tm : m_ref;
      const float corr = move ? exp2f(m_ref - m_new) : 1.f;      // 0 on the first tile
      m_ref = m_new;
      const bool any_move = __any_sync(0xffffffffu, move);       // same in all four warps
      if (any_move && quarter == 0 && lane < N) s_corr[lane] = corr;
      // ---- probabilities, partial sums, P tile in the no-swizzle MN-major layout
#pragma unroll
      for (int j = 0; j < N / 8; ++j) {
        uint32_t packed[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int h0 = j * 8 + 2 * e;
          const float mh0 = __shfl_sync(0xffffffffu, m_new, h0), mh1 = __shfl_sync(0xffffffffu, m_new, h0 + 1);
          const float p0 = exp2f(s[h0] - mh0), p1 = exp2f(s[h0 + 1] - mh1);
          if (any_move) {
            l_part[h0] *= __shfl_sync(0xffffffffu, corr, h0);
            l_part[h0 + 1] *= __shfl_sync(0xffffffffu, corr, h0 + 1);
          }
          const bf162 pb = __floats2bfloat162_rn(p0, p1);
          // sum what the tensor core will actually see (bf16-rounded probabilities)
          const float2 pr = __bfloat1622float2(pb);
          l_part[h0] += pr.x;
          l_part[h0 + 1] += pr.y;
          packed[e] = *(const uint32_t*)&pb;
        }
        *(uint4*)(s_p + j * 2048 + (trow >> 3) * 128 + (trow & 7) * 16) =
            make_uint4(packed[0], packed[1], packed[2], packed[3]);
      }
      // ---- rescale the TMEM-resident output when a reference moved (skip on the first tile:
      //      the first pass-B MMA overwrites)
      if (any_move && tile > 0) {
        named_bar_sync(1, kSoftmaxThreads);      // s_corr visible
        for (int blk = 0; blk < NB; ++blk) {
          float v[N];
          tc_ld_cols<N>(tmem_base + blk * N + lane_base, v);
          tc_wait_ld();
#pragma unroll
          for (int h = 0; h < N; ++h) v[h] *= s_corr[h];
          tc_st_cols<N>(tmem_base + blk * N + lane_base, v);
        }
        tc_wait_st();
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(smem_u32(&bars->p_ready));
    }

    // ---- epilogue: softmax statistics of this item (while the last pass B still runs) ...
    if (ok) {
      float wl = 0.f;
#pragma unroll
      for (int h = 0; h < N; ++h) {
        const float v = warp_sum(l_part[h]);
        if (lane == h) wl = v;
      }
      named_bar_sync(1, kSoftmaxThreads);
      if (lane < N) s_wmax[quarter * N + lane] = wl;
      named_bar_sync(1, kSoftmaxThreads);
      if (quarter == 0 && lane < nh_here && vpart == 0) {     // the blocks of a head group hold the same statistics
        const float lsum = s_wmax[lane] + s_wmax[N + lane] + s_wmax[2 * N + lane] + s_wmax[3 * N + lane];
        a.part_ml[((size_t)item * a.nv + vh0 + lane) * 2 + 0] = m_ref;
        a.part_ml[((size_t)item * a.nv + vh0 + lane) * 2 + 1] = lsum;
      }
    }
    // ---- ... and its partial output
    ok = mbar_wait_group(smem_u32(&bars->pv_done), (tbase + n_tiles - 1) & 1, s_abort, s_verdict, gw_turn, leader, 2, kSoftmaxThreads, 8) && ok;
    if (ok) {
      tc_fence_after();
      // The output block [128 coords x N heads] leaves TMEM with one thread per coordinate; it is
      // turned into [N heads][128 coords] tiles in shared memory (the ring is idle by now) and
      // written with one TMA store per block: part_acc[item][query row][h0 + h][blk*128 ...].
      // Rows of a last, partly filled head group fall outside the head axis of the tensor and
      // are clipped by the store.
      float* stage = (float*)s_lat;
      for (int blk = 0; blk < NB; ++blk) {
        float v[N];
        tc_ld_cols<N>(tmem_base + blk * N + lane_base, v);
        tc_wait_ld();
        if (blk >= kOutBufs) {     // a staging buffer comes round again: its store must have read it
          if (threadIdx.x == 64) bulk_wait_group_read<kOutBufs - 1>();
          named_bar_sync(1, kSoftmaxThreads);
        }
        float* tile_s = stage + (size_t)(blk % kOutBufs) * N * 128;
#pragma unroll
        for (int h = 0; h < N; ++h) tile_s[h * 128 + trow] = v[h];
        fence_proxy_async();
        named_bar_sync(1, kSoftmaxThreads);
        if (threadIdx.x == 64) {
          tma_store_4d(&map_part, vpart * vw_blk + blk * 128, h0, qrow, item, smem_u32(tile_s));
          bulk_commit_group();
        }
      }
      if (threadIdx.x == 64) bulk_wait_group_all();     // stores done before the ring is reused or the block leaves
    }
  }

  // ---- end of item: every role is done with the queries, the P tile and the output columns
  tbase += (unsigned)n_tiles;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (*s_abort) break;      // same value in every thread: nobody is inside a wait here
  }

  // ============================================================== teardown
  if (*s_abort) drain_after_abort();
  tc_fence_before();
  __syncthreads();
  // detail: worker in the low 16 bits, the code of the wait that gave up above them
  if (threadIdx.x == 0 && *s_abort) ekv_record(a.status, ELITEKV_ERR_TIMEOUT, worker | (*s_abort << 16), seq);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

// Heads per block: 32 when 32 fp32 output columns per 128 latent coordinates of the block's
// output share plus the score columns fit TMEM's 512 columns, else 16.  A layer with more heads
// than that runs as head groups (the last one partly filled: 40 heads = 32 + 8); each group
// streams the token tile itself, and the blocks of an item are adjacent so that the later readers
// hit L2.
// Output-column shares per head group: 1, or 2 when only half of the output fits TMEM beside
// the scores of 32 heads.
static int tc_pick_parts(const elitekv_layer* L) {
  const int nb = L->vw / 128;
  if ((nb + 1) * 32 <= 512) return 1;
  if (L->n_h <= 32 && nb % 2 == 0 && (nb / 2 + 1) * 32 <= 512) return 2;
  return 1;
}
static int tc_pick_n(const elitekv_layer* L) {
  const int nb = L->vw / 128 / tc_pick_parts(L);
  if ((nb + 1) * 32 <= 512) return 32;
  if ((nb + 1) * 16 <= 512) return 16;
  return 0;
}

int ekv_tc_supported(const elitekv_layer* L, const elitekv_cache* cache) {
  const int r2 = 2 * L->r;
  // pass A takes 64-wide chunks, pass B slot pairs that must start on an even ring use
  if (L->kw % 128 != 0 || L->vw % 128 != 0) return 0;
  if (!(r2 == 8 || r2 == 16 || r2 == 32)) return 0;
  const int n = tc_pick_n(L);
  if (n == 0) return 0;
  if ((L->n_h * r2) % 64 != 0 || L->n_h % 8 != 0) return 0;
  if ((n == 32 ? Smem<32>::total(L->d_c) : Smem<16>::total(L->d_c)) > L->smem_optin) return 0;
  // the epilogue cycles through kOutBufs staging tiles of [n][128] floats in the ring + rope area
  if ((size_t)kOutBufs * n * 128 * 4 > (size_t)kLatSlots * (kChunkBytes + n * 128) + (size_t)kRopeSlots * kChunkBytes) return 0;
  if (cache && cache->page_table && (cache->page_size % 64 != 0)) return 0;
  return 1;
}

static int tc_groups(const elitekv_layer* L) {      // head groups per query row
  const int n = tc_pick_n(L);
  return n ? (L->n_h + n - 1) / n : 1;
}

// One persistent worker (a block per query row and head group) per SM share; items = workers +
// sequences at most.
int ekv_tc_workers(const elitekv_layer* L, int rows) {
  const int per = tc_groups(L) * tc_pick_parts(L) * (rows > 0 ? rows : 1);
  return L->sm_count / per > 0 ? L->sm_count / per : 1;
}
int ekv_tc_max_items(const elitekv_layer* L, int B, int rows) { return ekv_tc_workers(L, rows) + B; }

int ekv_launch_decode_tc(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                         const void* q_rope, const void* q_abs, int B, const DecodeScratch& ws,
                         cudaStream_t st) {
  if (!ekv_tc_supported(L, cache)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  const unsigned long long rows =
      cv.page_table ? (unsigned long long)cv.num_pages << cv.page_shift : (unsigned long long)cv.max_ctx * cv.n_seqs;
  if (rows >= (1ull << 31)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap m_lat, m_rope, m_q, m_lat128, m_rope128, m_part;
  int rc = make_map(&m_lat, cache->latent, rows, L->d_c, 64);
  if (rc == ELITEKV_OK) rc = make_map(&m_rope, cache->rope, rows, (unsigned long long)L->n_h * 2 * L->r, 64);
  if (rc == ELITEKV_OK) rc = make_map(&m_lat128, cache->latent, rows, L->d_c, 128);
  if (rc == ELITEKV_OK) rc = make_map(&m_rope128, cache->rope, rows, (unsigned long long)L->n_h * 2 * L->r, 128);
  const int N = tc_pick_n(L);
  const int rows_q = ws.rows > 0 ? ws.rows : 1;
  if (rc == ELITEKV_OK) rc = make_map(&m_q, q_abs, (unsigned long long)B * rows_q * L->n_h, L->kw, N);
  if (rc == ELITEKV_OK) rc = make_map_f32_4d(&m_part, ws.part_acc, L->vw, L->n_h, rows_q, (unsigned long long)ws.max_items, N);
  if (rc != ELITEKV_OK) return rc;
  TcArgs a;
  a.items = ws.items;
  a.worker_first = ws.worker_first;
  a.page_table = cv.page_table;
  a.part_acc = ws.part_acc;
  a.part_ml = ws.part_ml;
  a.q_rope = (const bf16*)q_rope;
  a.status = L->d_status;
  a.max_ctx = cv.max_ctx;
  a.num_pages = cv.num_pages;
  a.page_shift = cv.page_shift;
  a.page_mask = cv.page_mask;
  a.max_pages_per_seq = cv.max_pages_per_seq;
  a.n_h = L->n_h;
  a.d_c = L->d_c;
  a.kw = L->kw;
  a.voff = L->voff;
  a.vw = L->vw;
  a.rows = rows_q;
  a.gpr = tc_groups(L);
  a.vparts = tc_pick_parts(L);
  a.n_groups = a.gpr * rows_q * a.vparts;
  a.nv = rows_q * L->n_h;
  a.seq_lens = ws.seq_lens;
  a.scale_log2e = L->scale * 1.4426950408889634f;
  const int smem = N == 32 ? Smem<32>::total(L->d_c) : Smem<16>::total(L->d_c);
  auto launch = [&](auto kern) -> int {
    EKV_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    EKV_CUDA_OK(ekv_launch_pdl(kern, dim3(ws.n_workers * a.n_groups), dim3(kThreads), (size_t)smem, st, m_lat, m_rope,
                               m_q, m_lat128, m_rope128, m_part, a));
    EKV_CUDA_OK(cudaGetLastError());
    return ELITEKV_OK;
  };
  if (N == 32) {
    switch (2 * L->r) {
      case 8: return launch(decode_tc_kernel<32, 8>);
      case 16: return launch(decode_tc_kernel<32, 16>);
      default: return launch(decode_tc_kernel<32, 32>);
    }
  }
  switch (2 * L->r) {
    case 8: return launch(decode_tc_kernel<16, 8>);
    case 16: return launch(decode_tc_kernel<16, 16>);
    default: return launch(decode_tc_kernel<16, 32>);
  }
}
