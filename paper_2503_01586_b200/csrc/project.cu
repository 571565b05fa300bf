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
// One block computes a [128 tokens x 128 output columns] tile: warp 0 streams the operand tiles
// ([128 x 64] of x and of the transposed weight, 128-byte swizzle) through a 4-stage ring, warp 1
// issues tcgen05.mma (M = 128, N = 128, K = 16, bf16 in, fp32 in TMEM), warps 2-5 run the epilogue.
// A tile lies either in the rope part or in the latent part (both are multiples of 128 wide).
// Every wait is bounded (timeouts are recorded and the block leaves through the common exit).
#include "tc_ptx.cuh"

namespace {

constexpr int kPM = 128, kPN = 128, kPK = 64;     // tile: tokens, output columns, depth per stage
constexpr int kPStages = 4;
constexpr int kPStageBytes = (kPM + kPN) * kPK * 2;   // 32 KB
constexpr int kPThreads = 192;

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

__global__ void __launch_bounds__(kPThreads, 1)
project_append_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                      const ProjArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* base = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  ProjBarriers* bars = (ProjBarriers*)(base + kPStages * kPStageBytes);
  uint32_t* s_tmem = (uint32_t*)(bars + 1);
  volatile int* s_abort = (volatile int*)(s_tmem + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * kPN;                 // first output column of the tile
  const long long t0 = (long long)blockIdx.y * kPM; // first token of the tile

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
    for (int k = 0; k < a.nk && ok; ++k) {
      const int s = k % kPStages;
      ok = warp_wait(smem_u32(&bars->empty[s]), ((k / kPStages) & 1) ^ 1, s_abort, 1);
      if (!ok) break;
      if (elect_one()) {
        const uint32_t fb = smem_u32(&bars->full[s]);
        mbar_expect_tx(fb, (uint32_t)kPStageBytes);
        tma_load_2d(smem_u32(base + s * kPStageBytes), &map_x, k * kPK, (int)t0, fb);
        tma_load_2d(smem_u32(base + s * kPStageBytes + kPM * kPK * 2), &map_w, k * kPK, n0, fb);
      }
      __syncwarp();
    }
  } else if (warp == 1) {
    constexpr uint32_t idesc = make_idesc(kPM, kPN, 0, 0);
    constexpr uint32_t hi_sw = desc_hi(1024, 2);
    const uint32_t base16 = (smem_u32(base) >> 4) & 0x3FFFu;
    bool ok = true;
    for (int k = 0; k < a.nk && ok; ++k) {
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
    const long long t = t0 + quarter * 32 + lane;
    long long row = -1;
    int p = 0;
    if (t < a.T) {
      const int s = a.seq_id[t];
      p = a.pos[t];
      if (p < 0 || p >= a.max_pos) {
        ekv_record(a.status, ELITEKV_ERR_BAD_POSITION, s, p);
      } else {
        int code, detail;
        row = ekv_token_row(a.cv, s, p, &code, &detail);
        if (row < 0) ekv_record(a.status, code, s, detail);
      }
    }
    // one outcome per warp: the TMEM loads below want all 32 lanes
    const bool ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->done), 0, s_abort, 3));
    tc_fence_after();
    if (ok) {
      const bool rope_tile = n0 < a.rope_w;
      const float2* csrow = a.cs + (long long)p * a.half;
      for (int cc = 0; cc < kPN / 32; ++cc) {
        float v[32];
        tc_ld32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(cc * 32), v);
        tc_wait_ld();
        if (row < 0) continue;
        const int g0 = n0 + cc * 32;
        uint32_t packed[16];
        if (rope_tile) {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 w = __ldg(csrow + __ldg(a.idx + (g0 >> 1) + j));
            const float y0 = __fsub_rn(__fmul_rn(v[2 * j], w.x), __fmul_rn(v[2 * j + 1], w.y));
            const float y1 = __fadd_rn(__fmul_rn(v[2 * j], w.y), __fmul_rn(v[2 * j + 1], w.x));
            const bf162 y = __floats2bfloat162_rn(y0, y1);
            packed[j] = *(const uint32_t*)&y;
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const bf162 y = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
            packed[j] = *(const uint32_t*)&y;
          }
        }
        uint4* dst = rope_tile ? (uint4*)(a.rope + row * a.rope_w + g0)
                               : (uint4*)(a.latent + row * a.d_c + (g0 - a.rope_w));
#pragma unroll
        for (int q = 0; q < 4; ++q) dst[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
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

}  // namespace

int ekv_launch_project_append(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                              const void* x, const int32_t* seq_id, const int32_t* pos, long long T,
                              cudaStream_t st) {
  const int rope_w = L->n_h * 2 * L->r;
  const int n_out = rope_w + L->d_c;
  if (L->d % kPK != 0 || rope_w % kPN != 0 || L->d_c % kPN != 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if (T >= (1ll << 31)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  const int smem = kPStages * kPStageBytes + (int)sizeof(ProjBarriers) + 64 + 1024;
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
  EKV_CUDA_OK(cudaFuncSetAttribute(project_append_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  dim3 grid((unsigned)(n_out / kPN), (unsigned)((T + kPM - 1) / kPM));
  project_append_kernel<<<grid, kPThreads, smem, st>>>(m_x, m_w, a);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
