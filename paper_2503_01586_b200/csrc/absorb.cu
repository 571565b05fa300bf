// Query preparation: RoPE on the elite chunks of q and absorption of B^k into the query
// (score equation of Section 3.1; Section 5 on folding B^k into the neighbouring product).
//
//   q_rope[b,h,2j:2j+2] = q[b,h,chunk idx[h][j]] . R(q_pos[b] * theta_idx[h][j])
//   q_abs [b,h,k]       = sum_i q_nope[b,h,i] * W_uk[k][h*dn + i]
//
// Grid (n_h, ceil(d_c/128)): a block owns one head and 128 latent coordinates.  Its 256 threads
// are 64 coordinate pairs x 4 groups over the head's un-rotated dims; every thread keeps one fp32
// accumulator pair per sequence of the current chunk of 16 sequences, so each weight element is
// read once per chunk, and the four groups are added through shared memory.  The weights come
// regrouped as [n_h][dn][d_c] (d_c contiguous); the block's [dn x 128] slab is brought into
// shared memory by one bulk copy per weight row, all issued at once by one warp, so the whole
// slab costs one trip to memory (the kernel is bound by latency, not by its 11 MB of traffic)
// and overlaps the gather of the queries.
#include "tc_ptx.cuh"

namespace {

constexpr int kAbsorbBatch = 16;
constexpr int kAbsorbThreads = 256;
constexpr int kAbsorbGroups = 4;
constexpr int kAbsorbCoords = 128;

__global__ void __launch_bounds__(kAbsorbThreads)
absorb_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ q_pos, int B,
              const bf16* __restrict__ WukT, const int32_t* __restrict__ qdims,
              const int32_t* __restrict__ idx, const float2* __restrict__ cs, bf16* __restrict__ q_rope,
              bf16* __restrict__ q_abs, int n_h, int d_h, int r, int d_c, int max_pos,
              int32_t* status) {
  extern __shared__ __align__(16) float smem_f[];
  ekv_pdl_trigger();      // nothing later in the stream is held up by this kernel's start
  const int h = blockIdx.x;
  const int dn = d_h - 2 * r;
  float* q_nope = smem_f;                                   // [dn][16] (sequence fastest)
  float* red = smem_f + (size_t)(dn > 0 ? dn : 1) * kAbsorbBatch;   // [3][16][128]
  bf16* s_w = (bf16*)(red + (size_t)(kAbsorbGroups - 1) * kAbsorbBatch * kAbsorbCoords);   // [dn][128]
  __shared__ __align__(8) uint64_t w_bar;
  __shared__ int s_abort;
  const bool rope_block = blockIdx.y == gridDim.y - 1;      // last grid row: query RoPE only
  const int k0 = blockIdx.y * kAbsorbCoords;
  const int kw = min(kAbsorbCoords, d_c - k0);       // coordinates of this slab (a multiple of 8)
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&w_bar), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();
  if (threadIdx.x < 32 && dn > 0 && !rope_block) {
    if (threadIdx.x == 0) mbar_expect_tx(smem_u32(&w_bar), (uint32_t)(dn * kw * 2));
    __syncwarp();
    const bf16* src = WukT + (size_t)h * dn * d_c + k0;
    for (int i = threadIdx.x; i < dn; i += 32)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(s_w + (size_t)i * kAbsorbCoords)), "l"(src + (size_t)i * d_c), "r"(kw * 2),
                     "r"(smem_u32(&w_bar)) : "memory");
  }
  bool w_ready = dn == 0;
  const int pair = threadIdx.x & 63, grp = threadIdx.x >> 6;
  const int k = blockIdx.y * kAbsorbCoords + 2 * pair;
  const int32_t* dims = qdims + (size_t)h * d_h;

  // rope part: one extra block per head does it (three dependent loads: kept off the path of
  // the blocks that do the absorption)
  if (rope_block) {
    for (int e = threadIdx.x; e < B * r; e += blockDim.x) {
      const int b = e / r, j = e % r;
      int p = q_pos[b];
      if (p < 0 || p >= max_pos) {
        ekv_record(status, ELITEKV_ERR_BAD_POSITION, b, p);
        p = 0;
      }
      const float2 w = cs[(size_t)p * (d_h / 2) + idx[h * r + j]];
      const bf16* qq = q + ((size_t)b * n_h + h) * d_h;
      const float x0 = __bfloat162float(qq[dims[2 * j]]), x1 = __bfloat162float(qq[dims[2 * j + 1]]);
      const float y0 = __fsub_rn(__fmul_rn(x0, w.x), __fmul_rn(x1, w.y));
      const float y1 = __fadd_rn(__fmul_rn(x0, w.y), __fmul_rn(x1, w.x));
      bf162* dst = (bf162*)(q_rope + ((size_t)b * n_h + h) * 2 * r + 2 * j);
      *dst = __floats2bfloat162_rn(y0, y1);
    }
      return;
  }

  const int per_grp = (dn + kAbsorbGroups - 1) / kAbsorbGroups;
  const int i_lo = min(dn, grp * per_grp), i_hi = min(dn, i_lo + per_grp);
  for (int b0 = 0; b0 < B; b0 += kAbsorbBatch) {
    const int nb = min(kAbsorbBatch, B - b0);
    __syncthreads();
    for (int e = threadIdx.x; e < kAbsorbBatch * dn; e += blockDim.x) {
      const int i = e / kAbsorbBatch, bb = e % kAbsorbBatch;
      q_nope[e] = bb < nb ? __bfloat162float(q[((size_t)(b0 + bb) * n_h + h) * d_h + dims[2 * r + i]]) : 0.f;
    }
    __syncthreads();
    float a0[kAbsorbBatch], a1[kAbsorbBatch];
#pragma unroll
    for (int bb = 0; bb < kAbsorbBatch; ++bb) a0[bb] = a1[bb] = 0.f;
    if (!w_ready) {
      // the weight slab has landed (bounded wait; a timeout is recorded and the block leaves)
      volatile int* abort_flag = &s_abort;
      w_ready = mbar_wait(smem_u32(&w_bar), 0, abort_flag, 1);
      if (!w_ready) {
        if (threadIdx.x == 0) ekv_record(status, ELITEKV_ERR_TIMEOUT, h, blockIdx.y);
        return;
      }
    }
    if (k < d_c) {
      const bf16* wp = s_w + 2 * pair;
      for (int i0 = i_lo; i0 < i_hi; i0 += 8) {
        float2 w[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)
          w[j] = i0 + j < i_hi ? __bfloat1622float2(*(const bf162*)(wp + (size_t)(i0 + j) * kAbsorbCoords))
                               : make_float2(0.f, 0.f);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (i0 + j < i_hi) {
            const float4* xr = (const float4*)(q_nope + (size_t)(i0 + j) * kAbsorbBatch);
#pragma unroll
            for (int v = 0; v < kAbsorbBatch / 4; ++v) {
              const float4 x = xr[v];
              a0[4 * v + 0] = fmaf(x.x, w[j].x, a0[4 * v + 0]); a1[4 * v + 0] = fmaf(x.x, w[j].y, a1[4 * v + 0]);
              a0[4 * v + 1] = fmaf(x.y, w[j].x, a0[4 * v + 1]); a1[4 * v + 1] = fmaf(x.y, w[j].y, a1[4 * v + 1]);
              a0[4 * v + 2] = fmaf(x.z, w[j].x, a0[4 * v + 2]); a1[4 * v + 2] = fmaf(x.z, w[j].y, a1[4 * v + 2]);
              a0[4 * v + 3] = fmaf(x.w, w[j].x, a0[4 * v + 3]); a1[4 * v + 3] = fmaf(x.w, w[j].y, a1[4 * v + 3]);
            }
          }
        }
      }
    }
    if (grp > 0) {
#pragma unroll
      for (int bb = 0; bb < kAbsorbBatch; ++bb)
        *(float2*)(red + ((size_t)(grp - 1) * kAbsorbBatch + bb) * kAbsorbCoords + 2 * pair) =
            make_float2(a0[bb], a1[bb]);
    }
    __syncthreads();
    if (grp == 0 && k < d_c) {
#pragma unroll
      for (int bb = 0; bb < kAbsorbBatch; ++bb) {
        if (bb < nb) {
          float s0 = a0[bb], s1 = a1[bb];
#pragma unroll
          for (int g = 0; g < kAbsorbGroups - 1; ++g) {
            const float2 t = *(const float2*)(red + ((size_t)g * kAbsorbBatch + bb) * kAbsorbCoords + 2 * pair);
            s0 += t.x;
            s1 += t.y;
          }
          *(bf162*)(q_abs + ((size_t)(b0 + bb) * n_h + h) * d_c + k) = __floats2bfloat162_rn(s0, s1);
        }
      }
    }
  }
}

}  // namespace

int ekv_launch_absorb(const elitekv_layer* L, const void* q, const int32_t* q_pos, int B,
                      void* q_rope, void* q_abs, cudaStream_t st) {
  if (B == 0) return ELITEKV_OK;
  dim3 grid(L->n_h, (L->d_c + kAbsorbCoords - 1) / kAbsorbCoords + 1);   // + one row of rope blocks
  size_t smem = sizeof(float) * (kAbsorbBatch * (size_t)(L->dn > 0 ? L->dn : 1) +
                                 (size_t)(kAbsorbGroups - 1) * kAbsorbBatch * kAbsorbCoords) +
                sizeof(bf16) * (size_t)L->dn * kAbsorbCoords;
  if ((int)smem > L->smem_optin || L->d_c % 8 != 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  EKV_CUDA_OK(cudaFuncSetAttribute(absorb_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  absorb_kernel<<<grid, kAbsorbThreads, smem, st>>>(
      (const bf16*)q, q_pos, B, L->d_WukT, L->d_qdims, L->d_idx, L->d_cs, (bf16*)q_rope,
      (bf16*)q_abs, L->n_h, L->d_h, L->r, L->d_c, L->max_pos, L->d_status);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
