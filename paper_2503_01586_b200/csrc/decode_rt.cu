// Resident-tile split-K decode kernel for sm_100a (tcgen05 + TMEM + TMA, 2-block clusters).
//
// Every cache byte enters shared memory exactly once: a 64-token tile of the latent plane stays
// where TMA put it from the score product to the value product.  The absorbed queries of a
// sequence (n_h x d_c bf16, 96 KB at d_c = 1536) have to sit in shared memory as well, as the
// second operand of the score product, and the two do not fit one block with any room to
// prefetch.  A cluster of two blocks therefore splits the LATENT axis: block c owns latent
// coordinates [c d_c/2, (c+1) d_c/2) -- half of the absorbed queries (resident for a whole plan
// item), half of every token row (the ring below), half of the output rows (TMEM).
//
// Per 64-token tile each block
//   1. computes its PARTIAL latent scores (score equation of Section 3.1 with B^k absorbed,
//      Section 5) over its coordinates.  The tile sits in the ring as units of two 64-coordinate
//      chunks, [2][64 tokens][64] bf16.  One tcgen05.mma (M = 128, N = 64, K = 16) takes a whole
//      unit as A (rows 0-63 = chunk 2u, rows 64-127 = chunk 2u+1) and the two matching query
//      chunks stacked as B, so the two diagonal 64 x 32 blocks of the accumulator are the
//      contributions of the two chunks and the off-diagonal blocks are never read: half the
//      MMAs of a plain M = 64 formulation at the same cost per MMA;
//   2. adds the two diagonal blocks, adds the rope dot products (FP32 FMA, straight from global
//      memory into registers) of the 32 tokens it is responsible for, sends the sum to its peer
//      through distributed shared memory and keeps it;
//   3. once the peer's sum has arrived both blocks hold the same full scores bit for bit
//      (a + b = b + a) and run the same online softmax (Section 2.1; base 2, reference maximum
//      moved only when a tile maximum exceeds it by more than 2^8);
//   4. accumulates acc_c[d_c/2 x n_h] += C[:, half_c]^T . P into its TMEM-resident output (the
//      latent is key and value source at once, Section 3.2), which frees the unit for the next
//      tile's data.
// The ring holds one tile plus spare units, so the loads of the next tile run under steps 2-4.
//
// A cluster is a persistent worker walking its items of the balanced plan (64-token tiles); per
// item each block writes its half of (acc) and block 0 writes (m, l).
//
// Roles per block (256 threads):
//   warps 0, 2   TMA producers (units dealt alternately); warp 0 also loads the query half
//   warp 1       TMEM owner and MMA issuer (warp-uniform, instructions under an elected lane,
//                as many landed units as possible per election; slot and phase counters advance
//                incrementally so that the descriptor words stay in uniform registers)
//   warp 3       hands the receive buffer back to the peer
//   warps 4-7    mixing of the partial scores, exchange, softmax, rescale, epilogue; while the
//                tensor core works on the value product of a tile and the score product of the
//                next one they compute the next tile's rope dot products (a warp reads whole rope
//                rows with 16-byte loads per lane, straight from global memory into registers)
// Every wait is bounded; on a timeout the block records ELITEKV_ERR_TIMEOUT, stops issuing work
// and leaves through the common exit (its peer then runs into its own limit).
#include "tc_ptx.cuh"

namespace {

constexpr int kT = 64;                 // tokens per tile
constexpr int kUnit = 16384;           // ring unit: [2 chunks][64 tokens][64 bf16]
constexpr int kMaxRing = 9;
constexpr int kRtThreads = 256;
constexpr int kSm = 128;               // softmax threads (warps 4-7)
constexpr int kHeads = 32;

struct RtArgs {
  const int32_t* items;
  const int32_t* worker_first;
  const int32_t* page_table;
  float* part_acc;          // [items][32][d_c]
  float* part_ml;           // [items][32][2]
  const bf16* q_rope;       // [B][32][R2]
  const bf16* rope_plane;   // [rows][32 * R2]
  int32_t* status;
  long long max_ctx;
  long long num_pages;
  int page_shift, page_mask, max_pages_per_seq;
  int d_c;
  int n_ring;               // ring units
  float scale_log2e;
};

struct __align__(8) RtBarriers {
  uint64_t full[kMaxRing], empty[kMaxRing];
  uint64_t q_full, q_free, s_full, p_ready, pv_done, recv_done;
  uint64_t x_full[2], x_free[2];
};

// shared-memory carve-up (offsets from a 1024-byte aligned base)
struct RtSmem {
  int q, ring, p, xmix, recv, wmax, corr, bars, total;
};
__host__ __device__ inline RtSmem rt_layout(int d_c, int n_ring) {
  RtSmem s;
  int o = 0;
  s.q = o;     o += (d_c / 128) * kHeads * 128;     // query half: d_c/128 chunks of [32 heads][64]
  s.ring = o;  o += n_ring * kUnit;
  s.p = o;     o += kT * kHeads * 2;                // probabilities bf16, operand layout
  s.xmix = o;  o += kT * kHeads * 4;                // rope scores, then the two halves' hand-over
  s.recv = o;  o += 2 * kT * kHeads * 4;            // the peer's partial scores, two tiles deep
  s.wmax = o;  o += 4 * 16 * 4;
  s.corr = o;  o += kHeads * 4;
  s.bars = o;  o += (int)sizeof(RtBarriers) + 64;   // + tmem base, abort flag, two verdict words
  s.total = o + 1024;
  return s;
}

__device__ __forceinline__ float4 ld_f4(const float* p) { return *(const float4*)p; }

#ifndef RT_WAIT_MODE
#define RT_WAIT_MODE 1
#endif
// Warp-level wait used by the roles that wait long (producers for a free unit, rope warps for
// the hand-over buffer, the MMA warp for P): the probe is mbarrier.try_wait, which parks the
// warp in hardware for a while instead of spinning, so a waiting warp does not take issue
// slots and shared-memory cycles from the warp of its scheduler that is doing the work.
template <bool kClusterAcquire = false>
__device__ __forceinline__ bool rt_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int why) {
#if RT_WAIT_MODE == 0
  return warp_wait(bar, parity, abort_flag, why);
#else
  for (unsigned i = 0; i < kWaitLimit; ++i) {
    if (__any_sync(0xffffffffu, kClusterAcquire ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity))) return true;
#if RT_WAIT_MODE == 2
    asm volatile("nanosleep.u32 64;" ::: "memory");
#endif
    if ((i & 255) == 255 && __any_sync(0xffffffffu, *abort_flag != 0)) return false;
  }
  if (*abort_flag == 0) *abort_flag = why;
  return false;
#endif
}

template <int R2>
__global__ void __launch_bounds__(kRtThreads, 1)
decode_rt_kernel(const __grid_constant__ CUtensorMap map_lat, const __grid_constant__ CUtensorMap map_q,
                 const RtArgs a) {
  constexpr int N = kHeads;
  constexpr int LPT = R2 / 8;           // 16-byte loads per lane per rope row (row = 32 * R2 bf16)
  extern __shared__ unsigned char smem_raw[];
  const int worker = blockIdx.x >> 1;
  const uint32_t rank = cluster_ctarank();
  const uint32_t peer = rank ^ 1u;
  const int d_c = a.d_c, DH = d_c >> 1;
  const int NU = DH >> 7;               // units per tile = 128-row output blocks of this block
  const int NR = a.n_ring;
  const RtSmem L = rt_layout(d_c, NR);

  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char* s_q = base + L.q;
  unsigned char* s_ring = base + L.ring;
  unsigned char* s_p = base + L.p;
  float* s_xmix = (float*)(base + L.xmix);      // [64 tokens][32 heads], 16-byte chunks rotated by the token
  float* s_recv = (float*)(base + L.recv);      // [2][64][32], same rotation
  float* s_wmax = (float*)(base + L.wmax);      // [4 warps][16 heads]
  float* s_corr = (float*)(base + L.corr);      // [32]
  RtBarriers* bars = (RtBarriers*)(base + L.bars);
  uint32_t* s_tmem = (uint32_t*)(bars + 1);
  volatile int* s_abort = (volatile int*)(s_tmem + 1);
  volatile int* s_verdict = s_abort + 1;        // [2]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 32) {
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_lat) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)&map_q) : "memory");
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxRing; ++i) {
      mbar_init(smem_u32(&bars->full[i]), 1);
      mbar_init(smem_u32(&bars->empty[i]), 1);
    }
    mbar_init(smem_u32(&bars->q_full), 1);
    mbar_init(smem_u32(&bars->q_free), 1);
    mbar_init(smem_u32(&bars->s_full), 1);
    mbar_init(smem_u32(&bars->p_ready), kSm / 32);
    mbar_init(smem_u32(&bars->pv_done), 1);
    mbar_init(smem_u32(&bars->recv_done), kSm / 32);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->x_full[i]), 1);       // armed per tile; completed by the peer's bulk copy
      mbar_init(smem_u32(&bars->x_free[i]), 1);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  constexpr uint32_t tmem_cols = 256;    // NU * 32 output columns (<= 192) + 64 score columns
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                    // the peer's barriers exist before any remote arrive
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const uint32_t tmem_s = tmem_base + NU * N;
  // Everything above touched only this cluster's own state; the plan, the queries and the cache
  // come from kernels earlier in the stream.
  ekv_pdl_wait();
  ekv_pdl_trigger();
  const int item_lo = a.worker_first[worker], item_hi = a.worker_first[worker + 1];

  // first cache row of a tile (tiles start on multiples of 64 tokens and pages hold a multiple
  // of 64 tokens, so a tile never straddles pages)
  auto tile_row = [&](int seq, int t_abs, bool report) -> long long {
    if (a.page_table == nullptr) return (long long)seq * a.max_ctx + t_abs;
    const int pi = t_abs >> a.page_shift;
    int page = pi < a.max_pages_per_seq ? a.page_table[(long long)seq * a.max_pages_per_seq + pi] : -1;
    if (page < 0 || page >= a.num_pages) {
      if (report) ekv_record(a.status, ELITEKV_ERR_BAD_PAGE, seq, page);
      page = 0;
    }
    return ((long long)page << a.page_shift) + (t_abs & a.page_mask);
  };
  // Items follow one another without a block-wide barrier: the roles are coupled only through
  // the mbarriers of the data they hand over (the query half through q_full / q_free, tiles
  // through the ring, scores and probabilities through s_full / p_ready), so the loads and the
  // score product of the next item run under the epilogue of the current one.
  int seq = -1;

  if (warp < 4) {
    // ============================================================ warps 0, 2: TMA producers
    if (warp == 0 || warp == 2) {
      const int prod = warp >> 1;
      const uint64_t pol_drop = make_l2_policy_evict_first(), pol_keep = make_l2_policy_evict_last();
      unsigned slot = 0, par = 0;          // ring position of the next unit and its phase parity
      for (int item = item_lo; item < item_hi; ++item) {
        seq = a.items[4 * item + 0];
        const int tok0 = a.items[4 * item + 1];
        const int n_tiles = (a.items[4 * item + 2] + kT - 1) / kT;
        if (prod == 0 && item > item_lo) {
          // the score product of the previous item's last tile has read the query half
          if (!rt_wait(smem_u32(&bars->q_free), (unsigned)(item - item_lo - 1) & 1, s_abort, 12)) break;
        }
        if (prod == 0 && elect_one()) {
          // this block's half of the sequence's absorbed queries: stays for the whole item
          const uint32_t qb = smem_u32(&bars->q_full);
          mbar_expect_tx(qb, (uint32_t)(2 * NU * N * 128));
          for (int kc = 0; kc < 2 * NU; ++kc)
            tma_load_2d_hint(smem_u32(s_q + kc * N * 128), &map_q, (int)rank * DH + kc * 64, seq * N, qb, pol_keep);
        }
        __syncwarp();
        bool ok = true;
        for (int tile = 0; tile < n_tiles && ok; ++tile) {
          const int row = (int)tile_row(seq, tok0 + tile * kT, prod == 0 && lane == 0);
          for (int u = 0; u < NU; ++u) {
            if ((u & 1) == prod) {
              ok = rt_wait(smem_u32(&bars->empty[slot]), par ^ 1, s_abort, 1);
              if (!ok) break;
              if (elect_one()) {
                const uint32_t fb = smem_u32(&bars->full[slot]);
                mbar_expect_tx(fb, (uint32_t)kUnit);
                const uint32_t dst = smem_u32(s_ring + slot * kUnit);
                tma_load_2d_hint(dst, &map_lat, (int)rank * DH + (2 * u) * 64, row, fb, pol_drop);
                tma_load_2d_hint(dst + 8192, &map_lat, (int)rank * DH + (2 * u + 1) * 64, row, fb, pol_drop);
              }
              __syncwarp();
            }
            if (++slot == (unsigned)NR) { slot = 0; par ^= 1; }
          }
        }
        if (!ok) break;
      }
    }
    // ============================================================ warp 1: MMA issuer
    else if (warp == 1) {
      constexpr uint32_t idesc_s = make_idesc(128, 2 * N, 0, 0);   // [unit rows] . [two query chunks]^T, K-major both
      constexpr uint32_t idesc_pv = make_idesc(128, N, 1, 1);      // acc = C^T . P, MN-major both
      constexpr uint32_t hi_sw = desc_hi(1024, 2);                 // 128-byte swizzle, 1024 bytes between 8-row groups
      constexpr uint32_t hi_p = desc_hi(kT * 16, 0);               // P: no swizzle, 1024 bytes between 8-head groups
      // 14-bit start-address fields of the operand descriptors: in a cluster the shared-window
      // address of a block of non-zero rank carries the rank above the offset, which must not
      // spill into the neighbouring descriptor fields
      const uint32_t ring16 = (smem_u32(s_ring) >> 4) & 0x3FFFu, q16 = (smem_u32(s_q) >> 4) & 0x3FFFu;
      const uint32_t lo_p = desc_lo(smem_u32(s_p), 128);
      const uint32_t full0 = smem_u32(&bars->full[0]), empty0 = smem_u32(&bars->empty[0]);
      unsigned slot = 0, par = 0;          // ring position of the next tile's first unit
      unsigned tiles_done = 0;
      for (int item = item_lo; item < item_hi; ++item) {
        seq = a.items[4 * item + 0];
        const int ntok = a.items[4 * item + 2];
        const int n_tiles = (ntok + kT - 1) / kT;
        bool ok = rt_wait(smem_u32(&bars->q_full), (unsigned)(item - item_lo) & 1, s_abort, 2);
        for (int tile = 0; tile < n_tiles && ok; ++tile) {
          const int nvalid = min(kT, ntok - tile * kT);
          const int ksteps = (nvalid + 15) >> 4;
          // ---- partial scores: 4 MMAs per unit (two chunks).  Units whose data has already landed
          //      are issued under one election (probing a completed phase is cheap, entering an
          //      elected block is not); only a unit that is still in flight is waited for.
          unsigned sa = slot, pa = par;
          uint32_t lb = q16 | (1u << 16);
          int u = 0;
          while (u < NU) {
            int n_ready = 0;
            {
              unsigned s2 = sa, p2 = pa;
              while (u + n_ready < NU && __any_sync(0xffffffffu, mbar_test_wait(full0 + s2 * 8, p2))) {
                ++n_ready;
                if (++s2 == (unsigned)NR) { s2 = 0; p2 ^= 1; }
              }
            }
            if (n_ready == 0) {
              ok = rt_wait(full0 + sa * 8, pa, s_abort, 3);
              if (!ok) break;
              n_ready = 1;
            }
            if (elect_one()) {
              unsigned s2 = sa;
              uint32_t lb2 = lb;
              for (int k = 0; k < n_ready; ++k) {
                const uint32_t la = (ring16 + s2 * (kUnit >> 4)) | (1u << 16);
                tc_mma_w(tmem_s, la, hi_sw, lb2, hi_sw, idesc_s, (u + k) != 0);
                tc_mma_w(tmem_s, la + 2, hi_sw, lb2 + 2, hi_sw, idesc_s, 1);   // +32 bytes along K per step
                tc_mma_w(tmem_s, la + 4, hi_sw, lb2 + 4, hi_sw, idesc_s, 1);
                tc_mma_w(tmem_s, la + 6, hi_sw, lb2 + 6, hi_sw, idesc_s, 1);
                lb2 += 512u;                                                   // next pair of query chunks
                if (++s2 == (unsigned)NR) s2 = 0;
              }
            }
            __syncwarp();
            for (int k = 0; k < n_ready; ++k) {
              lb += 512u;
              if (++sa == (unsigned)NR) { sa = 0; pa ^= 1; }
            }
            u += n_ready;
          }
          if (!ok) break;
          if (elect_one()) {
            tc_commit(smem_u32(&bars->s_full));
            if (tile == n_tiles - 1) tc_commit(smem_u32(&bars->q_free));   // the query half may be replaced
          }
          __syncwarp();
          // ---- wait for P (and the rescaled output) of this tile
          ok = rt_wait(smem_u32(&bars->p_ready), tiles_done & 1, s_abort, 4);
          if (!ok) break;
          tc_fence_after();
          // ---- value product: unit u = output block u (two 64-coordinate atoms 8 KB apart).
          //      Entering and leaving an elected block costs about as much as issuing four MMAs,
          //      so a full tile is issued under one election; every unit still gets its own commit
          //      so that the producers can refill it as early as possible.
          if (ksteps == 4) {
            if (elect_one()) {
              unsigned sb = slot;
              for (int u = 0; u < NU; ++u) {
                const uint32_t la = (ring16 + sb * (kUnit >> 4)) | (512u << 16);
                const uint32_t d = tmem_base + (uint32_t)u * N;
                tc_mma_w(d, la, hi_sw, lo_p, hi_p, idesc_pv, tile != 0);
                tc_mma_w(d, la + 128, hi_sw, lo_p + 16, hi_p, idesc_pv, 1);   // +16 tokens: 2048 bytes in A, 256 in P
                tc_mma_w(d, la + 256, hi_sw, lo_p + 32, hi_p, idesc_pv, 1);
                tc_mma_w(d, la + 384, hi_sw, lo_p + 48, hi_p, idesc_pv, 1);
                tc_commit(empty0 + sb * 8);
                if (++sb == (unsigned)NR) sb = 0;
              }
            }
            __syncwarp();
          } else {
            // ragged end of a sequence: rows past its last token inside the last 16-token step
            // become exact zeros so that zero-probability rows cannot inject NaN/Inf bit patterns
            unsigned sb = slot;
            for (int u = 0; u < NU; ++u) {
              if (ksteps * 16 > nvalid) {
                unsigned char* unit = s_ring + sb * kUnit;
                for (int e = lane; e < (ksteps * 16 - nvalid) * 16; e += 32) {
                  const int rrow = nvalid + (e >> 4), c16 = e & 15;
                  *(uint4*)(unit + (c16 >> 3) * 8192 + rrow * 128 + (c16 & 7) * 16) = make_uint4(0, 0, 0, 0);
                }
                fence_proxy_async();
                __syncwarp();
              }
              const uint32_t la = (ring16 + sb * (kUnit >> 4)) | (512u << 16);
              const uint32_t d = tmem_base + (uint32_t)u * N;
              if (elect_one()) {
                for (int k = 0; k < ksteps; ++k)
                  tc_mma_w(d, la + 128 * k, hi_sw, lo_p + 16 * k, hi_p, idesc_pv, (tile | k) != 0);
                tc_commit(empty0 + sb * 8);
              }
              __syncwarp();
              if (++sb == (unsigned)NR) sb = 0;
            }
          }
          if (elect_one()) tc_commit(smem_u32(&bars->pv_done));
          __syncwarp();
          slot = sa;
          par = pa;
          ++tiles_done;
        }
        if (!ok) break;
      }
    }
    // ============================================================ warp 3: hand-back of the receive buffer
    // Tells the peer that this block has consumed the partial scores the peer sent for a tile
    // (so the peer may reuse that receive buffer and its own send buffer), off the softmax
    // threads' critical path: a remote arrive with release semantics takes a round trip.
    else {
      unsigned gt = 0;
      for (int item = item_lo; item < item_hi; ++item) {
        const int n_tiles = (a.items[4 * item + 2] + kT - 1) / kT;
        bool ok = true;
        for (int tile = 0; tile < n_tiles && ok; ++tile, ++gt) {
          ok = rt_wait(smem_u32(&bars->recv_done), gt & 1, s_abort, 11);
          if (!ok) break;
          if (elect_one()) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->x_free[gt & 1]), peer));
          __syncwarp();
        }
        if (!ok) break;
      }
    }
  }
  else {
    // ============================================================ warps 4-7: scores -> P, rescale, epilogue
    // Thread (quarter, lane) may touch TMEM lanes 32 quarter + lane.  Quarters 0, 1 hold the
    // even-chunk diagonal block (accumulator rows = tokens 0-63, columns 0-31), quarters 2, 3 the
    // odd-chunk block (rows 64-127 = tokens 0-63 again, columns 32-63).  The two threads of a
    // token split the heads: the even-side thread finishes heads 0-15, the odd-side thread heads
    // 16-31, each handing the other 16 values to its partner through s_xmix.
    {
      const int sid = threadIdx.x - 128;
      unsigned gt_base = 0;              // tiles of this worker before the current item
      unsigned gw_turn = 0;              // group waits taken so far
      const int quarter = warp & 3;
      const int hh = quarter >> 1;                       // head half this thread finishes
      const int t = (quarter & 1) * 32 + lane;           // token row inside the tile
      const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
      const bool leader = sid == 0;
      const bool own_tok = (uint32_t)(t >> 5) == rank;   // this block added the rope part of the token
      float* xrow = s_xmix + t * N;
      for (int item = item_lo; item < item_hi; ++item) {
      seq = a.items[4 * item + 0];
      const int ntok = a.items[4 * item + 2];
      const int n_tiles = (ntok + kT - 1) / kT;
      float l_part[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) l_part[i] = 0.f;
      float m_ref = -INFINITY;                           // lane h: reference maximum of head h (all 32, in every warp)
      bool ok = true;
      // ---- rope part of the scores (FP32 FMA): the block adds it for tokens [32 rank, 32 rank + 32)
      // of every tile, a warp taking 8 of them.  A rope row is 32 heads x R2 bf16 = 4 R2 pieces of
      // 16 bytes; lane L of load i reads piece 32 i + L (one coalesced 512-byte request per
      // load), which belongs to head 8 (32 i + L) / R2.  The sums go to s_xmix[token][head], the
      // buffer the two halves of the block mix their partial scores in.
      const int tok0 = a.items[4 * item + 1];
      float qr[LPT][8];
#pragma unroll
      for (int i = 0; i < LPT; ++i) {
        const uint4 v = *(const uint4*)(a.q_rope + (size_t)seq * N * R2 + 8 * (32 * i + lane));
        const bf162* p2 = (const bf162*)&v;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float2 f = __bfloat1622float2(p2[j]);
          qr[i][2 * j] = f.x;
          qr[i][2 * j + 1] = f.y;
        }
      }
      // `g` = global tile count of the tile; the buffer was the send buffer of tile g - 1 and is free
      // once the peer has handed that tile's rows back
      auto rope_tile = [&](int tile, unsigned g) {
        const int nvalid = min(kT, ntok - tile * kT);
        const long long row0 = tile_row(seq, tok0 + tile * kT, false);
        float part[8][LPT];
#pragma unroll
        for (int tt = 0; tt < 8; ++tt) {
          const int tk = 32 * (int)rank + 8 * quarter + tt;
          uint4 v[LPT];
#pragma unroll
          for (int i = 0; i < LPT; ++i) {
            v[i] = make_uint4(0, 0, 0, 0);
            if (tk < nvalid)
              v[i] = __ldcs((const uint4*)(a.rope_plane + (size_t)(row0 + tk) * (size_t)(N * R2)) + 32 * i + lane);
          }
#pragma unroll
          for (int i = 0; i < LPT; ++i) {
            const bf162* k2 = (const bf162*)&v[i];
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float2 f = __bfloat1622float2(k2[j]);
              acc = fmaf(qr[i][2 * j], f.x, acc);
              acc = fmaf(qr[i][2 * j + 1], f.y, acc);
            }
            part[tt][i] = acc;
          }
        }
        // sum over the LPT adjacent lanes that share a head
#pragma unroll
        for (int tt = 0; tt < 8; ++tt)
#pragma unroll
          for (int i = 0; i < LPT; ++i) {
            float v = part[tt][i];
            if (LPT >= 2) v += __shfl_xor_sync(0xffffffffu, v, 1);
            if (LPT >= 4) v += __shfl_xor_sync(0xffffffffu, v, 2);
            part[tt][i] = v;
          }
        if (g > 0) (void)mbar_wait_cluster(smem_u32(&bars->x_free[(g - 1) & 1]), ((g - 1) >> 1) & 1, s_abort, 5);
        if ((lane & (LPT - 1)) == 0) {
#pragma unroll
          for (int tt = 0; tt < 8; ++tt) {
            const int tk = 32 * (int)rank + 8 * quarter + tt;
#pragma unroll
            for (int i = 0; i < LPT; ++i) {
              const int h = (8 * (32 * i + lane)) / R2;
              s_xmix[tk * N + ((((h >> 2) + tk) & 7) << 2) + (h & 3)] = part[tt][i];
            }
          }
        }
        named_bar_sync(1, kSm);              // rows are read by other warps than the ones that wrote them
      };
      rope_tile(0, gt_base);
      for (int tile = 0; tile < n_tiles; ++tile) {
        const unsigned gt = gt_base + (unsigned)tile, par = gt & 1, k2 = gt >> 1;
        const int nvalid = min(kT, ntok - tile * kT);
        // Waits inside a tile are per thread (try_wait parks the thread between probes).  A
        // thread whose wait gives up goes on to the tile's named barriers all the same; behind
        // the last of them the leader's view of the abort flag decides for the whole group.
        // ---- this thread's diagonal block row out of TMEM
        (void)mbar_wait(smem_u32(&bars->s_full), gt & 1, s_abort, 6);
        tc_fence_after();
        float mine[16], other[16];                       // heads 16 hh .. + 15, and the partner's 16
        tc_ld16(tmem_s + lane_base + (uint32_t)(hh * 32 + hh * 16), mine);
        tc_ld16(tmem_s + lane_base + (uint32_t)(hh * 32 + (1 - hh) * 16), other);
        tc_wait_ld();
        if (leader) mbar_expect_tx(smem_u32(&bars->x_full[par]), (uint32_t)(kT * N * 4));   // the peer's rows of this tile
        // ---- hand the partner its 16 heads (on top of the rope part where this block owns it)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int c = 4 * (1 - hh) + j;                // logical 16-byte chunk = heads 4c .. 4c+3
          float* px = xrow + (((c + t) & 7) << 2);
          float4 v = make_float4(other[4 * j], other[4 * j + 1], other[4 * j + 2], other[4 * j + 3]);
          if (own_tok) {
            const float4 x = ld_f4(px);
            v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
          }
          *(float4*)px = v;
        }
        named_bar_sync(1, kSm);
        // ---- this block's sum for the thread's 16 heads, kept and put back in place: the buffer
        //      then holds the block's whole [64 x 32] contribution, which one bulk copy takes to
        //      the peer
        float s[16];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int c = 4 * hh + j;
          float* px = xrow + (((c + t) & 7) << 2);
          const float4 x = ld_f4(px);
          s[4 * j] = mine[4 * j] + x.x;
          s[4 * j + 1] = mine[4 * j + 1] + x.y;
          s[4 * j + 2] = mine[4 * j + 2] + x.z;
          s[4 * j + 3] = mine[4 * j + 3] + x.w;
          *(float4*)px = make_float4(s[4 * j], s[4 * j + 1], s[4 * j + 2], s[4 * j + 3]);
        }
        fence_proxy_async();
        named_bar_sync(1, kSm);
        if (leader) {
          // the peer's receive buffer of this parity was handed back two tiles ago
          const bool free_ok = k2 == 0 || mbar_wait_cluster(smem_u32(&bars->x_free[par]), (k2 - 1) & 1, s_abort, 8);
          if (free_ok)
            bulk_copy_to_peer(map_to_cta(smem_u32(s_recv + par * kT * N), peer), smem_u32(s_xmix), (uint32_t)(kT * N * 4),
                              map_to_cta(smem_u32(&bars->x_full[par]), peer));
        }
        (void)mbar_wait(smem_u32(&bars->x_full[par]), k2 & 1, s_abort, 9);
        {
          const float* rrow = s_recv + (par * kT + t) * N;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int c = 4 * hh + j;
            const float4 x = ld_f4(rrow + (((c + t) & 7) << 2));
            s[4 * j] += x.x; s[4 * j + 1] += x.y; s[4 * j + 2] += x.z; s[4 * j + 3] += x.w;
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->recv_done));   // warp 3 hands the buffer back to the peer
        const bool live = t < nvalid;
#pragma unroll
        for (int i = 0; i < 16; ++i) s[i] = live ? s[i] * a.scale_log2e : -INFINITY;
        // ---- per-head maximum over the 64 tokens: two warps per head half
        float wm = -INFINITY;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float v = ord2f(__reduce_max_sync(0xffffffffu, f2ord(s[i])));
          if (lane == i) wm = v;
        }
        if (lane < 16) s_wmax[quarter * 16 + lane] = wm;
        if (leader) s_verdict[0] = *s_abort;             // every wait of this tile lies behind us
        named_bar_sync(1, kSm);
        if (s_verdict[0] != 0) {
          ok = false;
          break;
        }
        // lane h follows head h (all 32 heads, identically in the four warps and in both blocks)
        const int hq = (lane >> 4) * 2;                  // the two warps that hold head `lane`
        const float tm = fmaxf(s_wmax[hq * 16 + (lane & 15)], s_wmax[(hq + 1) * 16 + (lane & 15)]);
        const bool move = tm > m_ref + 8.f;              // reference moves only past a 2^8 head-room
        const float m_new = move ? tm : m_ref;
        const float corr = move ? exp2f(m_ref - m_new) : 1.f;   // 0 on the first tile of an item
        m_ref = m_new;
        const bool any_move = __any_sync(0xffffffffu, move);
        if (any_move && quarter == 0) s_corr[lane] = corr;
        // ---- probabilities, partial sums, P in the no-swizzle MN-major operand layout
#pragma unroll
        for (int g = 0; g < 2; ++g) {
          uint32_t packed[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int i0 = g * 8 + 2 * e;
            const float mh0 = __shfl_sync(0xffffffffu, m_new, 16 * hh + i0), mh1 = __shfl_sync(0xffffffffu, m_new, 16 * hh + i0 + 1);
            const float p0 = exp2f(s[i0] - mh0), p1 = exp2f(s[i0 + 1] - mh1);
            if (any_move) {
              l_part[i0] *= __shfl_sync(0xffffffffu, corr, 16 * hh + i0);
              l_part[i0 + 1] *= __shfl_sync(0xffffffffu, corr, 16 * hh + i0 + 1);
            }
            const bf162 pb = __floats2bfloat162_rn(p0, p1);
            const float2 pr = __bfloat1622float2(pb);     // sum what the tensor core will see
            l_part[i0] += pr.x;
            l_part[i0 + 1] += pr.y;
            packed[e] = *(const uint32_t*)&pb;
          }
          *(uint4*)(s_p + (2 * hh + g) * (kT * 16) + (t >> 3) * 128 + (t & 7) * 16) =
              make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
        // ---- rescale the TMEM-resident output when a reference moved (not on the first tile:
        //      its first value MMA overwrites).  s_full of this tile was committed after the
        //      value MMAs of the previous tile, so the output is quiescent here.
        if (any_move && tile > 0) {
          named_bar_sync(1, kSm);          // s_corr visible
          for (int blk = 0; blk < NU; ++blk) {
            float v[32];
            tc_ld32(tmem_base + blk * N + lane_base, v);
            tc_wait_ld();
#pragma unroll
            for (int h = 0; h < 32; ++h) v[h] *= s_corr[h];
            tc_st32(tmem_base + blk * N + lane_base, v);
          }
          tc_wait_st();
        }
        fence_proxy_async();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&bars->p_ready));
        // ---- the tensor core is busy with this tile's value product and the next tile's scores
        if (tile + 1 < n_tiles) rope_tile(tile + 1, gt + 1);
      }

      // ---- epilogue, once the last value MMAs are done (group wait: one outcome for all)
      const unsigned gl = gt_base + (unsigned)n_tiles - 1u;
      ok = mbar_wait_group(smem_u32(&bars->pv_done), gl & 1, s_abort, s_verdict, gw_turn, leader, 2, kSm, 10) && ok;
      // softmax statistics of this item ...
      if (ok) {
        float wl = 0.f;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float v = warp_sum(l_part[i]);
          if (lane == i) wl = v;
        }
        named_bar_sync(1, kSm);
        if (lane < 16) s_wmax[quarter * 16 + lane] = wl;
        named_bar_sync(1, kSm);
        if (rank == 0 && quarter == 0) {
          const int hq = (lane >> 4) * 2;
          const float lsum = s_wmax[hq * 16 + (lane & 15)] + s_wmax[(hq + 1) * 16 + (lane & 15)];
          *(float2*)(a.part_ml + ((size_t)item * N + lane) * 2) = make_float2(m_ref, lsum);
        }
      }
      // ... and this block's half of the partial output: a [128 coords x 32 heads] block leaves
      // TMEM with one thread per coordinate, so for a fixed head the lanes of a warp hold 32
      // consecutive coordinates: 128-byte stores straight from registers.  No shared memory is
      // involved, so the ring already carries the next item's tiles meanwhile.
      if (ok) {
        tc_fence_after();
        float* dst = a.part_acc + (size_t)item * N * d_c + (size_t)rank * DH + quarter * 32 + lane;
        for (int blk = 0; blk < NU; ++blk) {
          float v[32];
          tc_ld32(tmem_base + blk * N + lane_base, v);
          tc_wait_ld();
#pragma unroll
          for (int h = 0; h < 32; ++h) __stcg(dst + (size_t)h * d_c + blk * 128, v[h]);
        }
        tc_fence_before();     // the next item's first value MMA overwrites these columns (after p_ready)
      }
      gt_base += (unsigned)n_tiles;
      if (!ok) break;
      }
    }
  }

  // ============================================================== teardown
  if (*s_abort) drain_after_abort();
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) ekv_record(a.status, ELITEKV_ERR_TIMEOUT, worker | (*s_abort << 16), seq);
  cluster_sync_all();                    // no block leaves while its peer may still write into it
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

int rt_ring_units(const elitekv_layer* L) {
  const int fixed = rt_layout(L->d_c, 0).total;
  int nr = (L->smem_optin - fixed) / kUnit;
  return nr > kMaxRing ? kMaxRing : nr;
}

cudaLaunchAttribute rt_cluster_attr() {
  cudaLaunchAttribute at;
  at.id = cudaLaunchAttributeClusterDimension;
  at.val.clusterDim.x = 2;
  at.val.clusterDim.y = 1;
  at.val.clusterDim.z = 1;
  return at;
}

template <int R2>
int rt_launch(const CUtensorMap& m_lat, const CUtensorMap& m_q, const RtArgs& a,
              int n_workers, int smem, cudaStream_t st) {
  EKV_CUDA_OK(cudaFuncSetAttribute(decode_rt_kernel<R2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * n_workers);
  cfg.blockDim = dim3(kRtThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0] = rt_cluster_attr();
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  EKV_CUDA_OK(cudaLaunchKernelEx(&cfg, decode_rt_kernel<R2>, m_lat, m_q, a));
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

// Clusters of this kernel that the device can hold at once (one block per SM; pairs need two
// free SMs of one GPC).
template <int R2>
int rt_max_clusters(int smem) {
  if (cudaFuncSetAttribute(decode_rt_kernel<R2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
    return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2);
  cfg.blockDim = dim3(kRtThreads);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0] = rt_cluster_attr();
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, decode_rt_kernel<R2>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

}  // namespace

int ekv_rt_supported(const elitekv_layer* L, const elitekv_cache* cache) {
  const int r2 = 2 * L->r;
  if (L->n_h != kHeads) return 0;
  if (L->d_c % 256 != 0 || L->d_c > 1536) return 0;
  if (L->kw != L->d_c || L->voff != 0) return 0;     // separated latents: nothing is read twice, the two-pass kernel serves them
  if (!(r2 == 8 || r2 == 16 || r2 == 32)) return 0;
  if (rt_ring_units(L) < L->d_c / 256 + 1) return 0;          // one tile resident plus a spare unit
  if (cache && cache->page_table && (cache->page_size % kT != 0)) return 0;
  return 1;
}

// Persistent workers = clusters that are resident at once.
int ekv_rt_workers(const elitekv_layer* L) {
  static int cached_key = -1, cached = 0;
  const int smem = rt_layout(L->d_c, rt_ring_units(L)).total;
  const int key = (smem * 64 + 2 * L->r) * 8 + L->device;
  if (cached_key != key) {
    int n = 0;
    switch (2 * L->r) {
      case 8: n = rt_max_clusters<8>(smem); break;
      case 16: n = rt_max_clusters<16>(smem); break;
      default: n = rt_max_clusters<32>(smem); break;
    }
    if (n <= 0 || n > L->sm_count / 2) n = L->sm_count / 2 > 0 ? L->sm_count / 2 : 1;
    cached = n;
    cached_key = key;
  }
  return cached;
}

int ekv_rt_max_items(const elitekv_layer* L, int B) { return L->sm_count / 2 + B; }

int ekv_launch_decode_rt(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                         const void* q_rope, const void* q_abs, int B, const DecodeScratch& ws,
                         cudaStream_t st) {
  if (!ekv_rt_supported(L, cache) || ws.rows > 1) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if ((uintptr_t)q_rope & 15) return ELITEKV_ERR_INVALID_ARG;   // rope rows are read with 16-byte loads
  const unsigned long long rows =
      cv.page_table ? (unsigned long long)cv.num_pages << cv.page_shift : (unsigned long long)cv.max_ctx * cv.n_seqs;
  if (rows >= (1ull << 31)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap m_lat, m_q;
  int rc = make_map(&m_lat, cache->latent, rows, L->d_c, kT);
  if (rc == ELITEKV_OK) rc = make_map(&m_q, q_abs, (unsigned long long)B * L->n_h, L->d_c, kHeads);
  if (rc != ELITEKV_OK) return rc;
  RtArgs a;
  a.items = ws.items;
  a.worker_first = ws.worker_first;
  a.page_table = cv.page_table;
  a.part_acc = ws.part_acc;
  a.part_ml = ws.part_ml;
  a.q_rope = (const bf16*)q_rope;
  a.rope_plane = (const bf16*)cache->rope;
  a.status = L->d_status;
  a.max_ctx = cv.max_ctx;
  a.num_pages = cv.num_pages;
  a.page_shift = cv.page_shift;
  a.page_mask = cv.page_mask;
  a.max_pages_per_seq = cv.max_pages_per_seq;
  a.d_c = L->d_c;
  a.n_ring = rt_ring_units(L);
  a.scale_log2e = L->scale * 1.4426950408889634f;
  const int smem = rt_layout(L->d_c, a.n_ring).total;
  switch (2 * L->r) {
    case 8: return rt_launch<8>(m_lat, m_q, a, ws.n_workers, smem, st);
    case 16: return rt_launch<16>(m_lat, m_q, a, ws.n_workers, smem, st);
    default: return rt_launch<32>(m_lat, m_q, a, ws.n_workers, smem, st);
  }
}
