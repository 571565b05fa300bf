// Split combine + value up-projection.
//
// Each plan item left (m_s, l_s, acc_s[d_c]) per head, with m in base-2 log units.  For
// sequence b and head h (items s of b):
//   M = max_s m_s,  L = sum_s l_s 2^(m_s - M),  o_lat = sum_s acc_s 2^(m_s - M) / L
//   o[b,h,:] = o_lat . W_uv[:, h*d_h:(h+1)*d_h]        (B^v folded outwards, Section 5;
//                                                      V = c W_uv of Section 3.2)
// Grid (n_h, ceil(B/8)): a block owns one head and up to 8 sequences, so W_uv's head slice is
// read once per 8 sequences.  Threads are (output dim pair) x (k group); the latent axis is
// walked in chunks of 128 that are merged into shared memory first.
#include "common.cuh"

namespace {

constexpr int kCombBatch = 8;
constexpr int kCombThreads = 256;
constexpr int kCombChunk = 128;

__global__ void __launch_bounds__(kCombThreads)
combine_upproj_kernel(const float* __restrict__ part_acc, const float* __restrict__ part_ml,
                      const int32_t* __restrict__ seq_first, const bf16* __restrict__ Wuv,
                      bf16* __restrict__ out, int B, int n_h, int d_h, int d_c) {
  __shared__ float s_olat[kCombBatch][kCombChunk];
  __shared__ float s_M[kCombBatch], s_invL[kCombBatch];
  __shared__ int s_first[kCombBatch + 1];
  extern __shared__ float s_red[];     // [kgroups][kCombBatch][d_h]
  const int h = blockIdx.x;
  const int b0 = blockIdx.y * kCombBatch;
  const int nb = min(kCombBatch, B - b0);
  const int npair = d_h >> 1;
  const int kgroups = max(1, kCombThreads / npair);
  const int pair = threadIdx.x % npair;
  const int kg = threadIdx.x / npair;
  const bool worker = kg < kgroups;

  if (threadIdx.x <= nb) s_first[threadIdx.x] = seq_first[b0 + threadIdx.x];
  __syncthreads();
  // softmax statistics of each sequence: one warp per sequence
  {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int bb = warp; bb < nb; bb += kCombThreads / 32) {
      const int i0 = s_first[bb], i1 = s_first[bb + 1];
      float M = -INFINITY;
      for (int i = i0 + lane; i < i1; i += 32) M = fmaxf(M, part_ml[((size_t)i * n_h + h) * 2]);
      M = warp_max(M);
      float Lsum = 0.f;
      for (int i = i0 + lane; i < i1; i += 32) {
        const float* ml = part_ml + ((size_t)i * n_h + h) * 2;
        Lsum += ml[1] * exp2f(ml[0] - M);
      }
      Lsum = warp_sum(Lsum);
      if (lane == 0) {
        s_M[bb] = M;
        s_invL[bb] = (i1 > i0 && Lsum > 0.f) ? 1.f / Lsum : 0.f;
      }
    }
  }
  __syncthreads();

  float acc0[kCombBatch], acc1[kCombBatch];
#pragma unroll
  for (int bb = 0; bb < kCombBatch; ++bb) acc0[bb] = acc1[bb] = 0.f;

  for (int k0 = 0; k0 < d_c; k0 += kCombChunk) {
    const int kc = min(kCombChunk, d_c - k0);
    // merge the items of each sequence for this slice of the latent axis
    for (int e = threadIdx.x; e < kCombBatch * kCombChunk; e += kCombThreads) {
      const int bb = e / kCombChunk, k = e % kCombChunk;
      float v = 0.f;
      if (bb < nb && k < kc) {
        const float M = s_M[bb];
        for (int i = s_first[bb]; i < s_first[bb + 1]; ++i) {
          const float w = exp2f(part_ml[((size_t)i * n_h + h) * 2] - M);
          v = fmaf(w, part_acc[((size_t)i * n_h + h) * d_c + k0 + k], v);
        }
        v *= s_invL[bb];
      }
      s_olat[bb][k] = v;
    }
    __syncthreads();
    if (worker) {
      for (int k = kg; k < kc; k += kgroups) {
        const float2 w = __bfloat1622float2(
            *(const bf162*)(Wuv + (size_t)(k0 + k) * n_h * d_h + (size_t)h * d_h + 2 * pair));
#pragma unroll
        for (int bb = 0; bb < kCombBatch; ++bb) {
          const float x = s_olat[bb][k];
          acc0[bb] = fmaf(x, w.x, acc0[bb]);
          acc1[bb] = fmaf(x, w.y, acc1[bb]);
        }
      }
    }
    __syncthreads();
  }

  // reduce over k groups
  if (worker) {
#pragma unroll
    for (int bb = 0; bb < kCombBatch; ++bb) {
      s_red[((size_t)kg * kCombBatch + bb) * d_h + 2 * pair] = acc0[bb];
      s_red[((size_t)kg * kCombBatch + bb) * d_h + 2 * pair + 1] = acc1[bb];
    }
  }
  __syncthreads();
  for (int e = threadIdx.x; e < nb * d_h; e += kCombThreads) {
    const int bb = e / d_h, d = e % d_h;
    float v = 0.f;
    for (int g = 0; g < kgroups; ++g) v += s_red[((size_t)g * kCombBatch + bb) * d_h + d];
    out[((size_t)(b0 + bb) * n_h + h) * d_h + d] = __float2bfloat16_rn(v);
  }
}

}  // namespace

int ekv_launch_combine(const elitekv_layer* L, int B, const DecodeScratch& ws, void* out,
                       cudaStream_t st) {
  const int npair = L->d_h / 2;
  if (npair > kCombThreads) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  const int kgroups = kCombThreads / npair > 0 ? kCombThreads / npair : 1;
  const size_t smem = sizeof(float) * (size_t)kgroups * kCombBatch * L->d_h;
  dim3 grid(L->n_h, (B + kCombBatch - 1) / kCombBatch);
  EKV_CUDA_OK(cudaFuncSetAttribute(combine_upproj_kernel,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  combine_upproj_kernel<<<grid, kCombThreads, smem, st>>>(ws.part_acc, ws.part_ml, ws.seq_first,
                                                          L->d_Wuv, (bf16*)out, B, L->n_h, L->d_h,
                                                          L->d_c);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
