// Query preparation: RoPE on the elite chunks of q and absorption of B^k into the query
// (score equation of Section 3.1; Section 5 on folding B^k into the neighbouring product).
//
//   q_rope[b,h,2j:2j+2] = q[b,h,chunk idx[h][j]] . R(q_pos[b] * theta_idx[h][j])
//   q_abs [b,h,k]       = sum_i q_nope[b,h,i] * W_uk[k][h*dn + i]
//
// Grid (n_h, ceil(d_c/256)): a block owns one head and 256 latent coordinates; each thread
// owns two adjacent coordinates and keeps one fp32 accumulator pair per sequence of the
// current batch chunk, so every weight element is read once per chunk of 16 sequences.  The
// weights come regrouped as [n_h][dn][d_c] (d_c contiguous), which makes the reads coalesced.
#include "common.cuh"

namespace {

constexpr int kAbsorbBatch = 16;
constexpr int kAbsorbThreads = 128;

__global__ void __launch_bounds__(kAbsorbThreads)
absorb_kernel(const bf16* __restrict__ q, const int32_t* __restrict__ q_pos, int B,
              const bf16* __restrict__ WukT, const int32_t* __restrict__ qdims,
              const int32_t* __restrict__ idx, const float2* __restrict__ cs, bf16* __restrict__ q_rope,
              bf16* __restrict__ q_abs, int n_h, int d_h, int r, int d_c, int max_pos,
              int32_t* status) {
  extern __shared__ float q_nope[];   // [kAbsorbBatch][dn]
  const int h = blockIdx.x;
  const int dn = d_h - 2 * r;
  const int k = (blockIdx.y * kAbsorbThreads + threadIdx.x) * 2;
  const int32_t* dims = qdims + (size_t)h * d_h;

  // rope part: one block per head does it
  if (blockIdx.y == 0) {
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
  }

  for (int b0 = 0; b0 < B; b0 += kAbsorbBatch) {
    const int nb = min(kAbsorbBatch, B - b0);
    __syncthreads();
    for (int e = threadIdx.x; e < nb * dn; e += blockDim.x) {
      const int bb = e / dn, i = e % dn;
      q_nope[bb * dn + i] = __bfloat162float(q[((size_t)(b0 + bb) * n_h + h) * d_h + dims[2 * r + i]]);
    }
    __syncthreads();
    if (k < d_c) {
      float a0[kAbsorbBatch], a1[kAbsorbBatch];
#pragma unroll
      for (int bb = 0; bb < kAbsorbBatch; ++bb) a0[bb] = a1[bb] = 0.f;
      const bf16* wp = WukT + (size_t)h * dn * d_c + k;
#pragma unroll 4
      for (int i = 0; i < dn; ++i) {
        const float2 w = __bfloat1622float2(*(const bf162*)(wp + (size_t)i * d_c));
#pragma unroll
        for (int bb = 0; bb < kAbsorbBatch; ++bb) {
          const float x = q_nope[bb * dn + i];   // rows beyond nb hold stale values; results unused
          a0[bb] = fmaf(x, w.x, a0[bb]);
          a1[bb] = fmaf(x, w.y, a1[bb]);
        }
      }
#pragma unroll
      for (int bb = 0; bb < kAbsorbBatch; ++bb)
        if (bb < nb)
          *(bf162*)(q_abs + ((size_t)(b0 + bb) * n_h + h) * d_c + k) = __floats2bfloat162_rn(a0[bb], a1[bb]);
    }
  }
}

}  // namespace

int ekv_launch_absorb(const elitekv_layer* L, const void* q, const int32_t* q_pos, int B,
                      void* q_rope, void* q_abs, cudaStream_t st) {
  if (B == 0) return ELITEKV_OK;
  dim3 grid(L->n_h, (L->d_c + 2 * kAbsorbThreads - 1) / (2 * kAbsorbThreads));
  size_t smem = sizeof(float) * kAbsorbBatch * (size_t)(L->dn > 0 ? L->dn : 1);
  absorb_kernel<<<grid, kAbsorbThreads, smem, st>>>(
      (const bf16*)q, q_pos, B, L->d_WukT, L->d_qdims, L->d_idx, L->d_cs, (bf16*)q_rope,
      (bf16*)q_abs, L->n_h, L->d_h, L->r, L->d_c, L->max_pos, L->d_status);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
