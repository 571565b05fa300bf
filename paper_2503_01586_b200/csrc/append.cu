// Fused RoPE + cache append (Section 3.1: the rotated elite chunks of the new token enter the
// cache once; Section 3.2: the shared latent row is stored beside them).
//
// One thread block per token (grid-stride).  The latent row is moved with 16-byte accesses,
// the rope row as bf16 pairs: thread p owns chunk (h, j) = (p / r, p % r), reads the pair,
// looks up (cos, sin) of pos*theta_{idx[h][j]} and writes the rotated pair.  Every product and
// sum is rounded separately in fp32 (no fused multiply-add) so that the stored bits are a pure
// function of the table.
#include "common.cuh"

namespace {

__global__ void __launch_bounds__(256)
append_kernel(const bf162* __restrict__ k_e, const uint4* __restrict__ c,
              const int32_t* __restrict__ seq_id, const int32_t* __restrict__ pos,
              long long T, bf162* __restrict__ rope, uint4* __restrict__ latent, CacheView cv,
              const int32_t* __restrict__ idx, const float2* __restrict__ cs, int n_h, int r,
              int d_c, int half, int max_pos, int32_t* status) {
  const int n_pairs = n_h * r;
  const int n_vec = d_c >> 3;
  for (long long t = blockIdx.x; t < T; t += gridDim.x) {
    const int s = seq_id[t], p = pos[t];
    if (p < 0 || p >= max_pos) {
      if (threadIdx.x == 0) ekv_record(status, ELITEKV_ERR_BAD_POSITION, s, p);
      continue;
    }
    int code, detail;
    const long long row = ekv_token_row(cv, s, p, &code, &detail);
    if (row < 0) {
      if (threadIdx.x == 0) ekv_record(status, code, s, detail);
      continue;
    }
    const uint4* csrc = c + t * n_vec;
    uint4* cdst = latent + row * n_vec;
    for (int v = threadIdx.x; v < n_vec; v += blockDim.x) cdst[v] = __ldg(csrc + v);
    const bf162* ksrc = k_e + t * n_pairs;
    bf162* kdst = rope + row * n_pairs;
    const float2* csrow = cs + (long long)p * half;
    for (int q = threadIdx.x; q < n_pairs; q += blockDim.x) {
      const float2 w = __ldg(csrow + __ldg(idx + q));
      const float2 x = __bfloat1622float2(ksrc[q]);
      const float y0 = __fsub_rn(__fmul_rn(x.x, w.x), __fmul_rn(x.y, w.y));
      const float y1 = __fadd_rn(__fmul_rn(x.x, w.y), __fmul_rn(x.y, w.x));
      kdst[q] = __floats2bfloat162_rn(y0, y1);
    }
  }
}

}  // namespace

int ekv_launch_append(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                      const void* k_e, const void* c, const int32_t* seq_id, const int32_t* pos,
                      long long T, cudaStream_t st) {
  if (T == 0) return ELITEKV_OK;
  long long blocks = T < (long long)L->sm_count * 16 ? T : (long long)L->sm_count * 16;
  append_kernel<<<(unsigned)blocks, 256, 0, st>>>(
      (const bf162*)k_e, (const uint4*)c, seq_id, pos, T, (bf162*)cache->rope,
      (uint4*)cache->latent, cv, L->d_idx, L->d_cs, L->n_h, L->r, L->d_c, L->d_h / 2, L->max_pos,
      L->d_status);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
