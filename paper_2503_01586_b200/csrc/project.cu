// Projection fused with the cache append (tcgen05 + TMEM + TMA).
//
// The cache row of a token is made from its hidden state x by two projections (Section 3.2):
// the elite key chunks k_e = x W^k_e (the columns of W^k that belong to the head's elite chunks,
// Eq. 2) and the shared latent c = x A^kv.  Both are one GEMM against the column-concatenated
// weight [W^k_e | A^kv], x [T x d] . [d x (2 r n_h + d_c)].  The append (Section 3.1: the elite
// chunks are rotated once, at the token's position) is the epilogue of that GEMM: accumulators
// leave TMEM with one thread per token, rope columns are rotated as (even, odd) pairs with the
// (cos, sin) of pos * theta_{idx[h][j]}, everything is rounded once to bf16 and written straight
// to the token's cache row (contiguous or paged).  k_e and c never touch memory.
//
// One block computes a [128 tokens x 128 output columns] tile (prefill-sized calls: 256 x 256,
// see further down): warp 0 streams the operand tiles
// ([128 x 64] of x and of the transposed weight, 128-byte swizzle) through a 4-stage ring, warp 1
// issues tcgen05.mma (M = 128, N = 128, K = 16, bf16 in, fp32 in TMEM), warps 2-5 run the epilogue.
// A tile lies either in the rope part or in the latent part (both are multiples of 128 wide).
//
// A batch of at most 128 tokens (a decode step) has one token tile, so the grid above would be
// n_out / 128 blocks reading the 2 d n_out bytes of weights between them: 16 blocks for the 7B
// shape.  Such a call runs as clusters of kSplit = 8 blocks instead, each block taking an eighth
// of the depth d.  The partial sums leave TMEM, cross distributed shared memory (block i of a
// cluster collects rows [16 i, 16 i + 16) from all eight) and are added in block order, so the
// result does not depend on scheduling; the collecting block rotates, rounds and stores.
// Every wait is bounded (timeouts are recorded and the block leaves through the common exit).
#include "tc_ptx.cuh"

namespace {

constexpr int kPM = 128, kPN = 128, kPK = 64;     // tile: tokens, output columns, depth per stage
constexpr int kPStages = 4;
constexpr int kPStageBytes = (kPM + kPN) * kPK * 2;   // 32 KB
constexpr int kPThreads = 192;
constexpr int kSplit = 8;                         // blocks per cluster of the split-depth form
constexpr int kSplitRows = kPM / kSplit;          // token rows each block of a cluster finishes
constexpr int kRecvBytes = kSplit * kSplitRows * kPN * 4;   // 64 KB: [source block][row][column] fp32

struct ProjArgs {
  const int32_t* seq_id;
  const int32_t* pos;
  long long T;
  bf16* rope;
  bf16* latent;
  CacheView cv;
  const int32_t* idx;       // [n_h * r] chunk id of every cached pair
  const float2* cs;         // [max_pos][d_h/2]
  int rope_w, d_c, half, max_pos, nk;
  int32_t* status;
};

struct __align__(8) ProjBarriers {
  uint64_t full[kPStages], empty[kPStages], done;
};

// rotation, single rounding and the 16-byte stores of 8 consecutive output columns of one token
__device__ __forceinline__ void finish_columns(const ProjArgs& a, const float* v, long long row, int p, int g0) {
  uint32_t packed[4];
  if (g0 < a.rope_w) {
    const float2* csrow = a.cs + (long long)p * a.half;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 w = __ldg(csrow + __ldg(a.idx + (g0 >> 1) + j));
      const float y0 = __fsub_rn(__fmul_rn(v[2 * j], w.x), __fmul_rn(v[2 * j + 1], w.y));
      const float y1 = __fadd_rn(__fmul_rn(v[2 * j], w.y), __fmul_rn(v[2 * j + 1], w.x));
      const bf162 y = __floats2bfloat162_rn(y0, y1);
      packed[j] = *(const uint32_t*)&y;
    }
    *(uint4*)(a.rope + row * a.rope_w + g0) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bf162 y = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      packed[j] = *(const uint32_t*)&y;
    }
    *(uint4*)(a.latent + row * a.d_c + (g0 - a.rope_w)) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
  }
}

// cache row of token t (-1 and a recorded error when its position or sequence is out of range)
__device__ __forceinline__ long long token_row(const ProjArgs& a, long long t, int* p_out) {
  const int s = a.seq_id[t];
  const int p = a.pos[t];
  *p_out = p;
  if (p < 0 || p >= a.max_pos) {
    ekv_record(a.status, ELITEKV_ERR_BAD_POSITION, s, p);
    return -1;
  }
  int code, detail;
  const long long row = ekv_token_row(a.cv, s, p, &code, &detail);
  if (row < 0) ekv_record(a.status, code, s, detail);
  return row;
}

template <bool kSplitDepth>
__global__ void __launch_bounds__(kPThreads, 1)
project_append_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                      const ProjArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  float* s_recv = (float*)(base + kPStages * kPStageBytes);      // split-depth form only
  ProjBarriers* bars = (ProjBarriers*)(base + kPStages * kPStageBytes + (kSplitDepth ? kRecvBytes : 0));
  uint32_t* s_tmem = (uint32_t*)(bars + 1);
  volatile int* s_abort = (volatile int*)(s_tmem + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kPN;                 // first output column of the tile
  const long long t0 = (long long)blockIdx.y * kPM; // first token of the tile
  // depth steps of this block: all of them, or the cluster rank's share
  const int crank = kSplitDepth ? (int)cluster_ctarank() : 0;
  const int k_lo = kSplitDepth ? (int)((long long)a.nk * crank / kSplit) : 0;
  const int k_hi = kSplitDepth ? (int)((long long)a.nk * (crank + 1) / kSplit) : a.nk;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPStages; ++i) {
      mbar_init(smem_u32(&bars->full[i]), 1);
      mbar_init(smem_u32(&bars->empty[i]), 1);
    }
    mbar_init(smem_u32(&bars->done), 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  constexpr uint32_t tmem_cols = 128;
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 0) {
    // ---- operand tiles: x rows [t0, t0+128) and weight rows [n0, n0+128), 64 of d per stage
    //      (rows past T come back as zeros: they are never stored)
    bool ok = true;
    for (int k = 0; k < k_hi - k_lo && ok; ++k) {
      const int s = k % kPStages;
      ok = warp_wait(smem_u32(&bars->empty[s]), ((k / kPStages) & 1) ^ 1, s_abort, 1);
      if (!ok) break;
      if (elect_one()) {
        const uint32_t fb = smem_u32(&bars->full[s]);
        mbar_expect_tx(fb, (uint32_t)kPStageBytes);
        tma_load_2d(smem_u32(base + s * kPStageBytes), &map_x, (k_lo + k) * kPK, (int)t0, fb);
        tma_load_2d(smem_u32(base + s * kPStageBytes + kPM * kPK * 2), &map_w, (k_lo + k) * kPK, n0, fb);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = make_idesc(kPM, kPN, 0, 0);
    constexpr uint32_t hi_sw = desc_hi(1024, 2);
    const uint32_t base16 = (smem_u32(base) >> 4) & 0x3FFFu;
    bool ok = true;
    for (int k = 0; k < k_hi - k_lo && ok; ++k) {
      const int s = k % kPStages;
      ok = warp_wait(smem_u32(&bars->full[s]), (k / kPStages) & 1, s_abort, 2);
      if (!ok) break;
      const uint32_t la = (base16 + (uint32_t)s * (kPStageBytes >> 4)) | (1u << 16);
      const uint32_t lb = la + ((kPM * kPK * 2) >> 4);
      if (elect_one()) {
        tc_mma_w(tmem_base, la, hi_sw, lb, hi_sw, idesc, k != 0);
        tc_mma_w(tmem_base, la + 2, hi_sw, lb + 2, hi_sw, idesc, 1);
        tc_mma_w(tmem_base, la + 4, hi_sw, lb + 4, hi_sw, idesc, 1);
        tc_mma_w(tmem_base, la + 6, hi_sw, lb + 6, hi_sw, idesc, 1);
        tc_commit(smem_u32(&bars->empty[s]));
      }
      __syncwarp();
    }
    if (ok && elect_one()) tc_commit(smem_u32(&bars->done));
    __syncwarp();
  } else {
    // ---- epilogue: thread = token row of the tile
    const int quarter = warp & 3;
    const int trow = quarter * 32 + lane;
    const long long t = t0 + trow;
    long long row = -1;
    int p = 0;
    if (!kSplitDepth && t < a.T) row = token_row(a, t, &p);
    // one outcome per warp: the TMEM loads below want all 32 lanes
    const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->done), 0, s_abort, 3));
    tc_fence_after();
    if (ok) {
      // split depth: this row's partial sums go to the block that finishes the row
      const uint32_t dst = kSplitDepth
          ? map_to_cta(smem_u32(s_recv + ((size_t)crank * kSplitRows + (trow % kSplitRows)) * kPN), (uint32_t)(trow / kSplitRows))
          : 0u;
      for (int cc = 0; cc < kPN / 32; ++cc) {
        float v[32];
        tc_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(cc * 32), v);
        tc_wait_ld();
        if (kSplitDepth) {
          if (t < a.T) {
#pragma unroll
            for (int q = 0; q < 8; ++q)
              st_cluster_f4(dst + (uint32_t)(cc * 32 + 4 * q) * 4u, make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]));
          }
        } else if (row >= 0) {
#pragma unroll
          for (int q = 0; q < 4; ++q) finish_columns(a, v + 8 * q, row, p, n0 + cc * 32 + 8 * q);
        }
      }
    }
  }

  if (kSplitDepth) {
    // every block of the cluster has delivered (or given up): the barrier orders the remote
    // stores above before the sums below, and nobody is written to after it
    cluster_sync_all();
    if (warp >= 2 && !*s_abort) {
      const int e = threadIdx.x - 64;                    // 128 threads: 16 rows x 8 column groups
      const int rr = e >> 3, cg = e & 7;
      const long long t = t0 + crank * kSplitRows + rr;
      if (t < a.T) {
        int p = 0;
        const long long row = token_row(a, t, &p);
        if (row >= 0) {
          float v[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) v[i] = 0.f;
          for (int src = 0; src < kSplit; ++src) {       // fixed order: the sum does not depend on timing
            const float4* pr = (const float4*)(s_recv + ((size_t)src * kSplitRows + rr) * kPN + cg * 16);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float4 x = pr[i];
              v[4 * i] += x.x; v[4 * i + 1] += x.y; v[4 * i + 2] += x.z; v[4 * i + 3] += x.w;
            }
          }
          finish_columns(a, v, row, p, n0 + cg * 16);
          finish_columns(a, v + 8, row, p, n0 + cg * 16 + 8);
        }
      }
    }
  }

  // ---- teardown
  tc_fence_before();
  __syncthreads();
  if (*s_abort) drain_after_abort();
  if (threadIdx.x == 0 && *s_abort) ekv_record(a.status, ELITEKV_ERR_TIMEOUT, (int)blockIdx.x | (*s_abort << 16), (int)blockIdx.y);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------ prefill form: 256 x 256 tiles
// A 128 x 128 tile asks L2 for 32 KB of operands per 256 tensor-core clocks; at prefill size all
// SMs together ask for more than L2 delivers, and the tensor pipe idles more than half of the
// time.  A block of the prefill form computes 256 tokens x 256 columns: the two halves of the
// token rows are two accumulators (TMEM columns 0-255 and 256-511) that share every weight tile,
// so a stage of 64 KB (256 rows of x and 256 rows of the weights, 64 of d each) feeds eight
// M128 N256 K16 MMAs = 1024 clocks: half the operand bytes per flop.
constexpr int kBM = 256, kBN = 256;
constexpr int kBStages = 3;
constexpr int kBStageBytes = (kBM + kBN) * kPK * 2;   // 64 KB
constexpr int kBThreads = 224;    // warp 0 loads x, warp 6 the weights (one issuing warp draws ~50 GB/s, two
                                  // about twice that), warp 1 issues the MMAs, warps 2-5 run the epilogue

struct __align__(8) BigBarriers {
  uint64_t full[kBStages], empty[kBStages], done;
};

__global__ void __launch_bounds__(kBThreads, 1)
project_append_big_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                          const ProjArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  BigBarriers* bars = (BigBarriers*)(base + kBStages * kBStageBytes);
  uint32_t* s_tmem = (uint32_t*)(bars + 1);
  volatile int* s_abort = (volatile int*)(s_tmem + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kBN;
  const long long t0 = (long long)blockIdx.y * kBM;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kBStages; ++i) {
      mbar_init(smem_u32(&bars->full[i]), 2);      // one arrival per loading warp
      mbar_init(smem_u32(&bars->empty[i]), 1);
    }
    mbar_init(smem_u32(&bars->done), 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  constexpr uint32_t tmem_cols = 512;      // the whole tensor memory: one block per SM (192 KB of shared memory)
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  if (warp == 0 || warp == 6) {
    // ---- warp 0: one 256-row box of x per stage (rows past the end: zeros); warp 6: one of the weights
    const bool wload = warp == 6;
    bool ok = true;
    for (int k = 0; k < a.nk && ok; ++k) {
      const int s = k % kBStages;
      ok = warp_wait(smem_u32(&bars->empty[s]), ((k / kBStages) & 1) ^ 1, s_abort, wload ? 4 : 1);
      if (!ok) break;
      if (elect_one()) {
        const uint32_t fb = smem_u32(&bars->full[s]);
        mbar_expect_tx(fb, (uint32_t)(kBStageBytes / 2));
        if (wload) tma_load_2d(smem_u32(base + s * kBStageBytes + kBM * kPK * 2), &map_w, k * kPK, n0, fb);
        else tma_load_2d(smem_u32(base + s * kBStageBytes), &map_x, k * kPK, (int)t0, fb);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = make_idesc(128, kBN, 0, 0);
    constexpr uint32_t hi_sw = desc_hi(1024, 2);
    const uint32_t base16 = (smem_u32(base) >> 4) & 0x3FFFu;
    bool ok = true;
    for (int k = 0; k < a.nk && ok; ++k) {
      const int s = k % kBStages;
      ok = warp_wait(smem_u32(&bars->full[s]), (k / kBStages) & 1, s_abort, 2);
      if (!ok) break;
      const uint32_t la0 = (base16 + (uint32_t)s * (kBStageBytes >> 4)) | (1u << 16);   // token rows 0-127
      const uint32_t la1 = la0 + ((128 * kPK * 2) >> 4);                                // token rows 128-255
      const uint32_t lb = la0 + ((kBM * kPK * 2) >> 4);
      if (elect_one()) {
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {          // +32 bytes along d per step
          tc_mma_w(tmem_base, la0 + 2 * ks, hi_sw, lb + 2 * ks, hi_sw, idesc, (k | ks) != 0);
          tc_mma_w(tmem_base + kBN, la1 + 2 * ks, hi_sw, lb + 2 * ks, hi_sw, idesc, (k | ks) != 0);
        }
        tc_commit(smem_u32(&bars->empty[s]));
      }
      __syncwarp();
    }
    if (ok && elect_one()) tc_commit(smem_u32(&bars->done));
    __syncwarp();
  } else {
    // ---- epilogue: a thread owns token rows trow and trow + 128 of the tile
    const int quarter = warp & 3;
    const int trow = quarter * 32 + lane;
    long long row[2];
    int p[2] = {0, 0};
#pragma unroll
    for (int hf = 0; hf < 2; ++hf) {
      const long long t = t0 + hf * 128 + trow;
      row[hf] = t < a.T ? token_row(a, t, &p[hf]) : -1;
    }
    const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->done), 0, s_abort, 3));
    tc_fence_after();
    if (ok) {
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {
        for (int cc = 0; cc < kBN / 32; ++cc) {
          float v[32];
          tc_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(hf * kBN + cc * 32), v);
          tc_wait_ld();
          if (row[hf] < 0) continue;
#pragma unroll
          for (int q = 0; q < 4; ++q) finish_columns(a, v + 8 * q, row[hf], p[hf], n0 + cc * 32 + 8 * q);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*s_abort) drain_after_abort();
  if (threadIdx.x == 0 && *s_abort) ekv_record(a.status, ELITEKV_ERR_TIMEOUT, (int)blockIdx.x | (*s_abort << 16), (int)blockIdx.y);
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

}  // namespace

int ekv_launch_project_append(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                              const void* x, const int32_t* seq_id, const int32_t* pos, long long T,
                              cudaStream_t st) {
  const int rope_w = L->n_h * 2 * L->r;
  const int n_out = rope_w + L->d_c;
  if (L->d % kPK != 0 || rope_w % kPN != 0 || L->d_c % kPN != 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if (T >= (1ll << 31)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  // prefill-sized calls whose output width is whole 256-column tiles: the 256 x 256 form
  if (T >= 1024 && n_out % kBN == 0) {
    const int smem_big = kBStages * kBStageBytes + (int)sizeof(BigBarriers) + 64 + 1024;
    if (smem_big <= L->smem_optin) {
      CUtensorMap b_x, b_w;
      int rcb = make_map(&b_x, x, (unsigned long long)T, (unsigned long long)L->d, kBM);
      if (rcb == ELITEKV_OK) rcb = make_map(&b_w, L->d_WcatT, (unsigned long long)n_out, (unsigned long long)L->d, kBN);
      if (rcb != ELITEKV_OK) return rcb;
      ProjArgs b;
      b.seq_id = seq_id; b.pos = pos; b.T = T;
      b.rope = (bf16*)cache->rope; b.latent = (bf16*)cache->latent; b.cv = cv;
      b.idx = L->d_idx; b.cs = L->d_cs; b.rope_w = rope_w; b.d_c = L->d_c;
      b.half = L->d_h / 2; b.max_pos = L->max_pos; b.nk = L->d / kPK; b.status = L->d_status;
      EKV_CUDA_OK(cudaFuncSetAttribute(project_append_big_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_big));
      dim3 grid((unsigned)(n_out / kBN), (unsigned)((T + kBM - 1) / kBM));
      project_append_big_kernel<<<grid, kBThreads, smem_big, st>>>(b_x, b_w, b);
      EKV_CUDA_OK(cudaGetLastError());
      return ELITEKV_OK;
    }
  }
  // at most one token tile and enough depth for every block of a cluster: the split-depth form
  const bool split = T <= kPM && L->d / kPK >= kSplit;
  const int smem = kPStages * kPStageBytes + (split ? kRecvBytes : 0) + (int)sizeof(ProjBarriers) + 64 + 1024;
  if (smem > L->smem_optin) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  CUtensorMap m_x, m_w;
  int rc = make_map(&m_x, x, (unsigned long long)T, (unsigned long long)L->d, kPM);
  if (rc == ELITEKV_OK) rc = make_map(&m_w, L->d_WcatT, (unsigned long long)n_out, (unsigned long long)L->d, kPN);
  if (rc != ELITEKV_OK) return rc;
  ProjArgs a;
  a.seq_id = seq_id;
  a.pos = pos;
  a.T = T;
  a.rope = (bf16*)cache->rope;
  a.latent = (bf16*)cache->latent;
  a.cv = cv;
  a.idx = L->d_idx;
  a.cs = L->d_cs;
  a.rope_w = rope_w;
  a.d_c = L->d_c;
  a.half = L->d_h / 2;
  a.max_pos = L->max_pos;
  a.nk = L->d / kPK;
  a.status = L->d_status;
  if (split) {
    EKV_CUDA_OK(cudaFuncSetAttribute(project_append_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_out / kPN), 1, kSplit);
    cfg.blockDim = dim3(kPThreads);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = kSplit;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    EKV_CUDA_OK(cudaLaunchKernelEx(&cfg, project_append_kernel<true>, m_x, m_w, a));
  } else {
    EKV_CUDA_OK(cudaFuncSetAttribute(project_append_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    dim3 grid((unsigned)(n_out / kPN), (unsigned)((T + kPM - 1) / kPM));
    project_append_kernel<false><<<grid, kPThreads, smem, st>>>(m_x, m_w, a);
  }
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
