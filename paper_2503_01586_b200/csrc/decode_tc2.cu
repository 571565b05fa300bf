// Paired tensor-core split-K decode kernel for sm_100a: a cluster of two thread blocks splits
// the latent axis, so every cache byte goes through shared memory exactly once.
//
// Why a pair.  The absorbed queries of a sequence (n_h x d_c bf16) must sit in shared memory as
// the B operand of the score GEMM, and a token tile must stay there from the score GEMM until
// the value GEMM has used it.  With the whole latent width in one block the two do not fit
// together with any prefetch depth.  Block c of the pair therefore owns latent coordinates
// [c*d_c/2, (c+1)*d_c/2): half of the queries (48 KB at d_c = 1536), half of every token row,
// and half of the output rows.  Per 32-token tile each block
//   1. computes its PARTIAL scores  S_c[32 x n_h] = C[:, half_c] . Q_abs[:, half_c]^T
//      (tcgen05.mma, M = 64 with the upper 32 rows ignored, fp32 in TMEM),
//   2. adds the rope dot products (score equation of Section 3.1) of the 16 tokens it is
//      responsible for, and sends the 4 KB partial to its peer through distributed shared
//      memory while keeping a copy,
//   3. after the peer's partial has arrived both blocks hold the same full scores and run the
//      same online softmax (base 2, lazily moved reference max, Section 2.1),
//   4. accumulates  acc_c[d_c/2 x n_h] += C[:, half_c]^T . P  into its TMEM-resident output
//      (the latent is both key and value source, Section 3.2).
// The tile ring holds about 2.5 tiles, the score GEMM of tile i+1 is issued before the value
// GEMM of tile i, and the softmax threads send tile i+1's partial before they finish tile i, so
// the exchange latency is off the critical path.
//
// A pair is a persistent worker: it walks the items of the balanced plan that fall into its
// share of the batch's tiles, writing one partial result (m, l, acc) per item.
//
// Roles per block (192 threads): warp 0 lane 0 = TMA producer, warp 1 = MMA issuer and TMEM
// owner, warps 2-5 = rope / exchange / softmax / epilogue.  Every wait is bounded; on a timeout
// the block records ELITEKV_ERR_TIMEOUT, stops issuing work and leaves through the common exit.
#include "tc_ptx.cuh"

namespace {

constexpr int kT2 = 32;               // tokens per tile
constexpr int kUnitBytes = 8192;      // ring unit: [2 chunks][32 tokens][64 bf16]
constexpr int kThreads2 = 192;
constexpr int kSm2 = 128;             // softmax threads
constexpr int kMaxUnits = 16;

struct Tc2Args {
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
  int n_units;              // ring depth
  float scale_log2e;
};

struct __align__(8) Tc2Barriers {
  uint64_t full[kMaxUnits], empty[kMaxUnits];
  uint64_t rope_full[2], rope_empty[2];
  uint64_t q_full, p_ready;
  uint64_t s_full[2], pv_done[2];
  uint64_t x_full[2], x_free[2];
};

// shared-memory carve-up (offsets from a 1024-byte aligned base), N = 32 heads
struct Smem2 {
  int q, ring, rope, p, xbuf, srope, qrope, wmax, corr, bars, total;
};
__host__ __device__ inline Smem2 smem2_layout(int d_c, int r2, int n_units) {
  Smem2 s;
  const int dh = d_c / 2;
  int o = 0;
  s.q = o;     o += (dh / 64) * 32 * 128;
  s.ring = o;  o += n_units * kUnitBytes + 4096;      // + slack read by the M = 64 score MMA
  s.rope = o;  o += 2 * 16 * 32 * r2 * 2;             // two stages of [16 tokens][n_h * 2r]
  s.p = o;     o += 2 * kT2 * 32 * 2;
  s.xbuf = o;  o += 2 * 2 * kT2 * 32 * 4;
  s.srope = o; o += 16 * 32 * 4;
  s.qrope = o; o += 32 * r2 * 4;
  s.wmax = o;  o += 2 * 4 * 32 * 4;
  s.corr = o;  o += 2 * 32 * 4;
  s.bars = o;  o += (int)sizeof(Tc2Barriers) + 64;
  s.total = o + 1024;
  return s;
}

template <int R2>
__global__ void __launch_bounds__(kThreads2, 1)
decode_tc2_kernel(const __grid_constant__ CUtensorMap map_lat, const __grid_constant__ CUtensorMap map_rope,
                  const __grid_constant__ CUtensorMap map_q, const Tc2Args a) {
  constexpr int N = 32;
  constexpr int NRBOX = N * R2 / 64;    // rope boxes ([16 tokens][64 elements]) per stage
  constexpr int HPB = 64 / R2;          // heads per rope box
  extern __shared__ unsigned char smem_raw[];
  const int worker = blockIdx.x >> 1;
  const uint32_t rank = cluster_ctarank();
  const uint32_t peer = rank ^ 1;
  const int item_lo = a.worker_first[worker], item_hi = a.worker_first[worker + 1];
  const int d_c = a.d_c, DH = d_c >> 1;
  const int NBh = DH >> 7;              // ring units per tile = output blocks of this CTA
  const int NKCh = DH >> 6;
  const int NU = a.n_units;
  const Smem2 L = smem2_layout(d_c, R2, NU);

  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* s_q = base + L.q;
  unsigned char* s_ring = base + L.ring;
  unsigned char* s_ropeb = base + L.rope;
  unsigned char* s_p = base + L.p;
  float* s_x = (float*)(base + L.xbuf);          // [parity][source: 0 own, 1 peer][32][32]
  float* s_srope = (float*)(base + L.srope);     // [16][32]
  float* s_qrope = (float*)(base + L.qrope);     // [32][R2]
  float* s_wmax = (float*)(base + L.wmax);       // [4][32]
  float* s_corr = (float*)(base + L.corr);       // [32]
  Tc2Barriers* bars = (Tc2Barriers*)(base + L.bars);
  uint32_t* s_tmem = (uint32_t*)(bars + 1);
  volatile int* s_abort = (volatile int*)(s_tmem + 1);
  constexpr int kRopeStage = 16 * N * R2 * 2;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxUnits; ++i) {
      mbar_init(smem_u32(&bars->full[i]), 1);
      mbar_init(smem_u32(&bars->empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->rope_full[i]), 1);
      mbar_init(smem_u32(&bars->rope_empty[i]), kSm2 / 32);
      mbar_init(smem_u32(&bars->s_full[i]), 1);
      mbar_init(smem_u32(&bars->pv_done[i]), 1);
      mbar_init(smem_u32(&bars->x_full[i]), 64);     // 32 own + 32 peer row writers
      mbar_init(smem_u32(&bars->x_free[i]), 1);
    }
    mbar_init(smem_u32(&bars->q_full), 1);
    mbar_init(smem_u32(&bars->p_ready), kSm2);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  constexpr uint32_t tmem_cols = 256;   // NBh*32 output columns (<= 192) + two 32-column score buffers
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                   // peer's barriers are initialised before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t tmem_s0 = tmem_base + NBh * N;

  unsigned gt_base = 0;                 // tiles processed by this worker before the current item
  for (int item = item_lo; item < item_hi; ++item) {
    const int seq = a.items[4 * item + 0];
    const int tok0 = a.items[4 * item + 1];
    const int ntok = a.items[4 * item + 2];
    const int n_tiles = (ntok + kT2 - 1) / kT2;
    const unsigned item_n = (unsigned)(item - item_lo);

    // ============================================================ warp 0: TMA producer
    if (warp == 0) {
      if (lane == 0) {
        bool ok = true;
        {
          // this block's half of the sequence's absorbed queries
          const uint32_t qbar = smem_u32(&bars->q_full);
          mbar_expect_tx(qbar, (uint32_t)(NKCh * N * 128));
          for (int kc = 0; kc < NKCh; ++kc)
            tma_load_2d(smem_u32(s_q + kc * N * 128), &map_q, (int)rank * DH + kc * 64, seq * a.n_h, qbar);
        }
        for (int tile = 0; tile < n_tiles && ok; ++tile) {
          const unsigned gt = gt_base + tile;
          const int t_abs = tok0 + tile * kT2;
          long long row;
          if (a.page_table == nullptr) {
            row = (long long)seq * a.max_ctx + t_abs;
          } else {
            const int pi = t_abs >> a.page_shift;
            int page = pi < a.max_pages_per_seq ? a.page_table[(long long)seq * a.max_pages_per_seq + pi] : -1;
            if (page < 0 || page >= a.num_pages) {
              ekv_record(a.status, ELITEKV_ERR_BAD_PAGE, seq, page);
              page = 0;
            }
            row = ((long long)page << a.page_shift) + (t_abs & a.page_mask);
          }
          {
            // rope rows of the 16 tokens this block adds to the scores
            const unsigned st = gt & 1;
            ok = mbar_wait(smem_u32(&bars->rope_empty[st]), ((gt >> 1) & 1) ^ 1, s_abort);
            if (!ok) break;
            const uint32_t fb = smem_u32(&bars->rope_full[st]);
            mbar_expect_tx(fb, (uint32_t)(NRBOX * 2048));
            for (int box = 0; box < NRBOX; ++box)
              tma_load_2d(smem_u32(s_ropeb + st * kRopeStage + box * 2048), &map_rope, box * 64,
                          (int)(row + 16 * (int)rank), fb);
          }
          for (int u = 0; u < NBh && ok; ++u) {
            const unsigned cnt = gt * (unsigned)NBh + u, slot = cnt % (unsigned)NU;
            ok = mbar_wait(smem_u32(&bars->empty[slot]), ((cnt / (unsigned)NU) & 1) ^ 1, s_abort);
            if (!ok) break;
            const uint32_t fb = smem_u32(&bars->full[slot]);
            mbar_expect_tx(fb, (uint32_t)kUnitBytes);
            for (int c = 0; c < 2; ++c)
              tma_load_2d(smem_u32(s_ring + slot * kUnitBytes + c * 4096), &map_lat,
                          (int)rank * DH + (2 * u + c) * 64, (int)row, fb);
          }
        }
      }
    }
    // ============================================================ warp 1: MMA issuer
    else if (warp == 1) {
      constexpr uint32_t idesc_s = make_idesc(64, N, 0, 0);     // partial S = C_half . Q_half^T
      constexpr uint32_t idesc_pv = make_idesc(128, N, 1, 1);   // acc_half += C_half^T . P
      bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->q_full), item_n & 1, s_abort));
      auto issue_scores = [&](int tile) -> bool {
        const unsigned gt = gt_base + tile;
        const uint32_t d_tmem = tmem_s0 + (gt & 1) * N;
        for (int u = 0; u < NBh; ++u) {
          const unsigned cnt = gt * (unsigned)NBh + u, slot = cnt % (unsigned)NU;
          if (!__all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->full[slot]), (cnt / (unsigned)NU) & 1, s_abort)))
            return false;
          tc_fence_after();
          if (lane == 0) {
            const uint32_t a_addr = smem_u32(s_ring + slot * kUnitBytes);
            const uint32_t b_addr = smem_u32(s_q + (2 * u) * N * 128);
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
              for (int k = 0; k < 4; ++k)
                tc_mma(d_tmem, make_desc(a_addr + c * 4096 + k * 32, 16, 1024, 2),
                       make_desc(b_addr + c * N * 128 + k * 32, 16, 1024, 2), idesc_s, (u | c | k) != 0);
          }
          __syncwarp();
        }
        if (lane == 0) tc_commit(smem_u32(&bars->s_full[gt & 1]));
        __syncwarp();
        return true;
      };
      if (ok && n_tiles > 0) ok = issue_scores(0);
      for (int tile = 0; tile < n_tiles && ok; ++tile) {
        if (tile + 1 < n_tiles) {
          ok = issue_scores(tile + 1);
          if (!ok) break;
        }
        const unsigned gt = gt_base + tile;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->p_ready), gt & 1, s_abort));
        if (!ok) break;
        tc_fence_after();
        const int nvalid = min(kT2, ntok - tile * kT2);
        const int ksteps = (nvalid + 15) >> 4;
        const int zero_from = nvalid, zero_to = ksteps * 16;
        for (int u = 0; u < NBh; ++u) {
          const unsigned cnt = gt * (unsigned)NBh + u, slot = cnt % (unsigned)NU;
          unsigned char* unit = s_ring + slot * kUnitBytes;
          if (zero_to > zero_from) {
            // rows past the end of the sequence inside the last 16-token step become exact zeros,
            // so that zero-probability rows cannot inject NaN/Inf bit patterns
            for (int e = lane; e < (zero_to - zero_from) * 16; e += 32) {
              const int rrow = zero_from + (e >> 4), c16 = e & 15;
              *(uint4*)(unit + (c16 >> 3) * 4096 + rrow * 128 + (c16 & 7) * 16) = make_uint4(0, 0, 0, 0);
            }
            fence_proxy_async();
            __syncwarp();
          }
          if (lane == 0) {
            const uint32_t a_addr = smem_u32(unit);
            const uint32_t b_addr = smem_u32(s_p + (gt & 1) * (kT2 * N * 2));
            for (int k = 0; k < ksteps; ++k)
              tc_mma(tmem_base + u * N, make_desc(a_addr + k * 2048, 4096, 1024, 2),
                     make_desc(b_addr + k * 256, 128, 512, 0), idesc_pv, (tile | k) != 0);
            tc_commit(smem_u32(&bars->empty[slot]));
          }
          __syncwarp();
        }
        if (lane == 0) tc_commit(smem_u32(&bars->pv_done[gt & 1]));
        __syncwarp();
      }
    }
    // ============================================================ warps 2-5: rope, exchange, softmax
    else {
      const int sid = threadIdx.x - 64, tg = sid >> 5, quarter = warp & 3;
      const int h = lane;                                   // head this thread owns in the softmax
      const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
      for (int e = sid; e < N * R2; e += kSm2)
        s_qrope[e] = __bfloat162float(a.q_rope[((size_t)seq * a.n_h + e / R2) * R2 + (e % R2)]);
      named_bar_sync(1, kSm2);
      float m_ref = -INFINITY, l_part = 0.f;
      bool ok = true;

      // rope scores of this block's 16 tokens, then partial scores out of TMEM to both blocks
      auto rope_and_send = [&](int tile) -> bool {
        const unsigned gt = gt_base + tile, par = gt & 1, k = gt >> 1;
        bool w = mbar_wait(smem_u32(&bars->rope_full[par]), k & 1, s_abort);
        if (w) {
          for (int task = sid; task < 16 * NRBOX; task += kSm2) {
            const int tt = task / NRBOX, box = task % NRBOX;
            const unsigned char* rowp = s_ropeb + par * kRopeStage + box * 2048 + tt * 128;
            float part[HPB];
#pragma unroll
            for (int hh = 0; hh < HPB; ++hh) part[hh] = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 v = *(const uint4*)(rowp + ((c ^ (tt & 7)) << 4));
              const bf162* k2 = (const bf162*)&v;
              const int hh = (c * 8) / R2;
              const float* qq = s_qrope + (box * HPB + hh) * R2 + (c * 8) % R2;
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
            for (int hh = 0; hh < HPB; ++hh) s_srope[tt * N + box * HPB + hh] = part[hh];
          }
        }
        named_bar_sync(1, kSm2);
        if (lane == 0) mbar_arrive(smem_u32(&bars->rope_empty[par]));
        if (quarter < 2) {       // the warps whose TMEM lanes hold token rows 0-15 / 16-31
          const bool w2 = mbar_wait(smem_u32(&bars->s_full[par]), k & 1, s_abort);
          w = w && w2;
          tc_fence_after();
          float sv[32];
          tc_ld32(tmem_s0 + par * N + lane_base, sv);
          tc_wait_ld();
          if (lane < 16 && w) {
            const int t = quarter * 16 + lane;
            if ((uint32_t)(t >> 4) == rank) {
#pragma unroll
              for (int j = 0; j < N; ++j) sv[j] += s_srope[(t & 15) * N + j];
            }
            // the peer must have consumed what this buffer held two tiles ago
            if (k > 0) w = mbar_wait_cluster(smem_u32(&bars->x_free[par]), (k - 1) & 1, s_abort);
            float* own = s_x + ((par * 2 + 0) * kT2 + t) * N;
            const uint32_t remote = map_to_cta(smem_u32(s_x + ((par * 2 + 1) * kT2 + t) * N), peer);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int pos = (j + t) & 7;       // rotate 16-byte chunks: conflict-free rows
              const float4 v = make_float4(sv[4 * j], sv[4 * j + 1], sv[4 * j + 2], sv[4 * j + 3]);
              *(float4*)(own + pos * 4) = v;
              st_cluster_f4(remote + pos * 16, v);
            }
            mbar_arrive(smem_u32(&bars->x_full[par]));
            mbar_arrive_cluster(map_to_cta(smem_u32(&bars->x_full[par]), peer));
          }
        }
        named_bar_sync(1, kSm2);
        return w;
      };

      // full scores -> probabilities -> P tile (and TMEM rescale when the reference max moves)
      auto softmax_tile = [&](int tile) -> bool {
        const unsigned gt = gt_base + tile, par = gt & 1, k = gt >> 1;
        bool w = mbar_wait_cluster(smem_u32(&bars->x_full[par]), k & 1, s_abort);
        const int nvalid = min(kT2, ntok - tile * kT2);
        float s[8];
        float mloc = -INFINITY;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int t = tg * 8 + i;
          const int idx = t * N + ((((h >> 2) + t) & 7) << 2) + (h & 3);
          const float v = s_x[(par * 2 + 0) * kT2 * N + idx] + s_x[(par * 2 + 1) * kT2 * N + idx];
          s[i] = (t < nvalid && w) ? v * a.scale_log2e : -INFINITY;
          mloc = fmaxf(mloc, s[i]);
        }
        float* wmax = s_wmax + par * 4 * N;
        wmax[tg * N + h] = mloc;
        named_bar_sync(1, kSm2);
        // every thread has read the peer-written copy: hand the buffer back
        if (sid == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->x_free[par]), peer));
        const float tm = fmaxf(fmaxf(wmax[h], wmax[N + h]), fmaxf(wmax[2 * N + h], wmax[3 * N + h]));
        const bool move = tm > m_ref + 8.f;        // reference moves only past a 2^8 head-room
        const float m_new = move ? tm : m_ref;
        const float corr = move ? exp2f(m_ref - m_new) : 1.f;   // 0 on the first tile of an item
        m_ref = m_new;
        const bool any_move = __any_sync(0xffffffffu, move);    // identical in all four warps
        l_part *= corr;
        // the P buffer of this parity was last read by the value MMA two tiles ago
        if (k > 0) w = mbar_wait(smem_u32(&bars->pv_done[par]), (k - 1) & 1, s_abort) && w;
        unsigned char* pb = s_p + par * (kT2 * N * 2) + (h >> 3) * 512 + tg * 128 + (h & 7) * 2;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const bf16 p = __float2bfloat16_rn(exp2f(s[i] - m_new));
          l_part += __bfloat162float(p);           // sum what the tensor core will see
          *(bf16*)(pb + i * 16) = p;
        }
        if (any_move && tile > 0) {
          // the output must be quiescent: value MMA of the previous tile
          const unsigned gp = gt - 1;
          w = mbar_wait(smem_u32(&bars->pv_done[gp & 1]), (gp >> 1) & 1, s_abort) && w;
          float* corr_s = s_corr + par * N;
          if (tg == 0) corr_s[h] = corr;
          named_bar_sync(1, kSm2);
          tc_fence_after();
          for (int blk = 0; blk < NBh; ++blk) {
            float v[32];
            tc_ld32(tmem_base + blk * N + lane_base, v);
            tc_wait_ld();
#pragma unroll
            for (int j = 0; j < N; ++j) v[j] *= corr_s[j];
            tc_st32(tmem_base + blk * N + lane_base, v);
          }
          tc_wait_st();
        }
        fence_proxy_async();
        tc_fence_before();
        mbar_arrive(smem_u32(&bars->p_ready));
        return w;
      };

      if (n_tiles > 0) ok = rope_and_send(0);
      for (int tile = 0; tile < n_tiles && ok; ++tile) {
        if (tile + 1 < n_tiles) {
          ok = rope_and_send(tile + 1);
          if (!ok) break;
        }
        ok = softmax_tile(tile);
      }

      // ---- epilogue: this block's half of the partial output, and the softmax statistics
      if (ok && n_tiles > 0) {
        const unsigned gl = gt_base + n_tiles - 1;
        ok = mbar_wait(smem_u32(&bars->pv_done[gl & 1]), (gl >> 1) & 1, s_abort);
      }
      if (ok && n_tiles > 0) {
        tc_fence_after();
        float* pa = a.part_acc + (size_t)item * a.n_h * d_c + (size_t)rank * DH + quarter * 32 + lane;
        for (int blk = 0; blk < NBh; ++blk) {
          float v[32];
          tc_ld32(tmem_base + blk * N + lane_base, v);
          tc_wait_ld();
#pragma unroll
          for (int j = 0; j < N; ++j) pa[(size_t)j * d_c + blk * 128] = v[j];
        }
      }
      named_bar_sync(1, kSm2);
      s_wmax[tg * N + h] = l_part;
      named_bar_sync(1, kSm2);
      if (ok && rank == 0 && tg == 0) {
        a.part_ml[((size_t)item * a.n_h + h) * 2 + 0] = m_ref;
        a.part_ml[((size_t)item * a.n_h + h) * 2 + 1] = s_wmax[h] + s_wmax[N + h] + s_wmax[2 * N + h] + s_wmax[3 * N + h];
      }
    }
    gt_base += (unsigned)n_tiles;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }

  // ============================================================== teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) ekv_record(a.status, ELITEKV_ERR_TIMEOUT, worker, (int)rank);
  cluster_sync_all();                   // no block leaves while its peer may still write into it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

int tc2_units(const elitekv_layer* L) {
  const int fixed = smem2_layout(L->d_c, 2 * L->r, 0).total;
  int nu = (L->smem_optin - fixed) / kUnitBytes;
  if (nu > kMaxUnits) nu = kMaxUnits;
  return nu;
}

template <int R2>
int tc2_launch(const CUtensorMap& m_lat, const CUtensorMap& m_rope, const CUtensorMap& m_q, const Tc2Args& a,
               int n_workers, int smem, cudaStream_t st) {
  EKV_CUDA_OK(cudaFuncSetAttribute(decode_tc2_kernel<R2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * n_workers);
  cfg.blockDim = dim3(kThreads2);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  EKV_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_tc2_kernel<R2>, m_lat, m_rope, m_q, a));
  return ELITEKV_OK;
}

template <int R2>
int tc2_max_clusters(int smem) {
  if (cudaFuncSetAttribute(decode_tc2_kernel<R2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2);
  cfg.blockDim = dim3(kThreads2);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, decode_tc2_kernel<R2>, &cfg) != cudaSuccess) return 0;
  return n;
}

}  // namespace

int ekv_tc2_supported(const elitekv_layer* L, const elitekv_cache* cache) {
  const int r2 = 2 * L->r;
  if (L->n_h != 32) return 0;
  if (L->d_c % 256 != 0 || L->d_c > 1536) return 0;
  if (!(r2 == 8 || r2 == 16 || r2 == 32)) return 0;
  if (tc2_units(L) < 2 * (L->d_c / 256)) return 0;
  if (cache && cache->page_table && (cache->page_size % kT2 != 0)) return 0;
  return 1;
}

// Number of pairs that can be resident at once = number of persistent workers.
int ekv_tc2_workers(const elitekv_layer* L) {
  static int cached_for = -1, cached = 0;
  const int nu = tc2_units(L);
  const int smem = smem2_layout(L->d_c, 2 * L->r, nu).total;
  const int key = smem * 64 + 2 * L->r;
  if (cached_for != key) {
    int n = 0;
    switch (2 * L->r) {
      case 8: n = tc2_max_clusters<8>(smem); break;
      case 16: n = tc2_max_clusters<16>(smem); break;
      default: n = tc2_max_clusters<32>(smem); break;
    }
    if (n <= 0) n = L->sm_count / 2 > 2 ? L->sm_count / 2 - 2 : 1;
    if (n > L->sm_count / 2) n = L->sm_count / 2;
    cached = n;
    cached_for = key;
  }
  return cached;
}

int ekv_tc2_max_items(const elitekv_layer* L, int B) { return L->sm_count / 2 + B; }

int ekv_launch_decode_tc2(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                          const void* q_rope, const void* q_abs, int B, const DecodeScratch& ws,
                          cudaStream_t st) {
  if (!ekv_tc2_supported(L, cache)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  const unsigned long long rows =
      cv.page_table ? (unsigned long long)cv.num_pages << cv.page_shift : (unsigned long long)cv.max_ctx * cv.n_seqs;
  if (rows >= (1ull << 31)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap m_lat, m_rope, m_q;
  int rc = make_map(&m_lat, cache->latent, rows, L->d_c, kT2);
  if (rc == ELITEKV_OK) rc = make_map(&m_rope, cache->rope, rows, (unsigned long long)L->n_h * 2 * L->r, 16);
  if (rc == ELITEKV_OK) rc = make_map(&m_q, q_abs, (unsigned long long)B * L->n_h, L->d_c, 32);
  if (rc != ELITEKV_OK) return rc;
  Tc2Args a;
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
  a.n_units = tc2_units(L);
  a.scale_log2e = L->scale * 1.4426950408889634f;
  const int smem = smem2_layout(L->d_c, 2 * L->r, a.n_units).total;
  switch (2 * L->r) {
    case 8: return tc2_launch<8>(m_lat, m_rope, m_q, a, ws.n_workers, smem, st);
    case 16: return tc2_launch<16>(m_lat, m_rope, m_q, a, ws.n_workers, smem, st);
    default: return tc2_launch<32>(m_lat, m_rope, m_q, a, ws.n_workers, smem, st);
  }
}
