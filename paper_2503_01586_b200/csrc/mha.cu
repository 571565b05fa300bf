// Comparator: decode attention over an UNCOMPRESSED cache of rotated keys and values
// (Sections 2.1 and 2.2), used to measure what the compressed cache saves.  Pure streaming:
// 4 n_h d_h bytes per token, one multiply-add per byte, so CUDA-core FMA is enough.
//
// Grid (splits, ceil(n_h/8), B), one warp per head.  d_h/8 lanes share a token (16-byte loads
// of K and V), so a warp walks 32/(d_h/8) tokens at once and every lane group keeps its own
// online-softmax state; groups are merged with shuffles at the end.  A second kernel merges
// the splits.
#include "common.cuh"

namespace {

constexpr int kMhaHeads = 8;
constexpr int kMhaMaxSplits = 64;

template <int LPT>   // lanes per token = d_h / 8
__global__ void __launch_bounds__(kMhaHeads * 32)
mha_split_kernel(const bf16* __restrict__ q_hat, const bf16* __restrict__ K, const bf16* __restrict__ V,
                 const int32_t* __restrict__ seq_lens, int n_h, long long max_ctx,
                 float scale_log2e, float* __restrict__ part /* [B][n_h][S][d_h+2] */) {
  constexpr int D_H = LPT * 8;
  constexpr int TPW = 32 / LPT;
  const int S = gridDim.x, split = blockIdx.x, b = blockIdx.z;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int h = blockIdx.y * kMhaHeads + warp;
  if (h >= n_h) return;
  const int n = min((long long)max(seq_lens[b], 0), max_ctx);
  const int tiles = (n + 63) >> 6;
  const int t_begin = min(n, (int)((long long)tiles * split / S) * 64);
  const int t_end = min(n, (int)((long long)tiles * (split + 1) / S) * 64);
  const int grp = lane / LPT, sub = lane % LPT;

  float qf[8];
  {
    const uint4 v = *(const uint4*)(q_hat + ((size_t)b * n_h + h) * D_H + sub * 8);
    const bf162* p2 = (const bf162*)&v;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(p2[e]);
      qf[2 * e] = f.x * scale_log2e;
      qf[2 * e + 1] = f.y * scale_log2e;
    }
  }
  float m = -INFINITY, l = 0.f, acc[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) acc[e] = 0.f;

  const size_t tok_stride = (size_t)n_h * D_H;
  const bf16* Kb = K + ((size_t)b * max_ctx) * tok_stride + (size_t)h * D_H + sub * 8;
  const bf16* Vb = V + ((size_t)b * max_ctx) * tok_stride + (size_t)h * D_H + sub * 8;
  constexpr int UNROLL = 4;
  for (int t0 = t_begin; t0 < t_end; t0 += TPW * UNROLL) {
    uint4 kv[UNROLL], vv[UNROLL];
    bool ok[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const int t = t0 + u * TPW + grp;
      ok[u] = t < t_end;
      if (ok[u]) {
        kv[u] = __ldg((const uint4*)(Kb + (size_t)t * tok_stride));
        vv[u] = __ldg((const uint4*)(Vb + (size_t)t * tok_stride));
      } else {
        kv[u] = make_uint4(0, 0, 0, 0);
        vv[u] = make_uint4(0, 0, 0, 0);
      }
    }
#pragma unroll
    for (int u = 0; u < UNROLL; ++u) {
      const bf162* k2 = (const bf162*)&kv[u];
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 f = __bfloat1622float2(k2[e]);
        s = fmaf(qf[2 * e], f.x, s);
        s = fmaf(qf[2 * e + 1], f.y, s);
      }
#pragma unroll
      for (int o = LPT / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      if (ok[u]) {
        const float m_new = fmaxf(m, s);
        const float corr = exp2f(m - m_new);
        const float p = exp2f(s - m_new);
        l = l * corr + p;
        m = m_new;
        const bf162* v2 = (const bf162*)&vv[u];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(v2[e]);
          acc[2 * e] = fmaf(p, f.x, acc[2 * e] * corr);
          acc[2 * e + 1] = fmaf(p, f.y, acc[2 * e + 1] * corr);
        }
      }
    }
  }
  // merge the lane groups of the warp
#pragma unroll
  for (int o = LPT; o < 32; o <<= 1) {
    const float m_o = __shfl_xor_sync(0xffffffffu, m, o);
    const float l_o = __shfl_xor_sync(0xffffffffu, l, o);
    const float m_new = fmaxf(m, m_o);
    const float w_self = m == -INFINITY ? 0.f : exp2f(m - m_new);
    const float w_o = m_o == -INFINITY ? 0.f : exp2f(m_o - m_new);
    l = l * w_self + l_o * w_o;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float a_o = __shfl_xor_sync(0xffffffffu, acc[e], o);
      acc[e] = acc[e] * w_self + a_o * w_o;
    }
    m = m_new;
  }
  if (grp == 0) {
    float* pp = part + (((size_t)b * n_h + h) * S + split) * (D_H + 2);
#pragma unroll
    for (int e = 0; e < 8; ++e) pp[sub * 8 + e] = acc[e];
    if (sub == 0) {
      pp[D_H] = m;
      pp[D_H + 1] = l;
    }
  }
}

__global__ void mha_combine_kernel(const float* __restrict__ part, int S, int d_h,
                                   bf16* __restrict__ out) {
  const size_t bh = blockIdx.x;
  const float* pp = part + bh * S * (d_h + 2);
  float M = -INFINITY;
  for (int s = 0; s < S; ++s) M = fmaxf(M, pp[(size_t)s * (d_h + 2) + d_h]);
  for (int d = threadIdx.x; d < d_h; d += blockDim.x) {
    float L = 0.f, v = 0.f;
    for (int s = 0; s < S; ++s) {
      const float ms = pp[(size_t)s * (d_h + 2) + d_h];
      const float w = ms == -INFINITY ? 0.f : exp2f(ms - M);
      L = fmaf(pp[(size_t)s * (d_h + 2) + d_h + 1], w, L);
      v = fmaf(pp[(size_t)s * (d_h + 2) + d], w, v);
    }
    out[bh * d_h + d] = __float2bfloat16_rn(L > 0.f ? v / L : 0.f);
  }
}

int mha_splits(int B, int n_h, int sm_count) {
  const int groups = (n_h + kMhaHeads - 1) / kMhaHeads;
  int S = (8 * sm_count + B * groups - 1) / (B * groups);
  if (S < 1) S = 1;
  if (S > kMhaMaxSplits) S = kMhaMaxSplits;
  return S;
}

int sm_count_current(int* out) {
  int dev;
  EKV_CUDA_OK(cudaGetDevice(&dev));
  EKV_CUDA_OK(cudaDeviceGetAttribute(out, cudaDevAttrMultiProcessorCount, dev));
  return ELITEKV_OK;
}

}  // namespace

extern "C" int elitekv_mha_workspace_size(int32_t B, int32_t n_h, int32_t d_h, size_t* bytes) {
  if (!bytes || B <= 0 || n_h <= 0 || d_h <= 0) return ELITEKV_ERR_INVALID_ARG;
  *bytes = sizeof(float) * (size_t)B * n_h * kMhaMaxSplits * (d_h + 2);
  return ELITEKV_OK;
}

extern "C" int elitekv_mha_decode(const void* q_hat, const void* K_hat, const void* V,
                                  const int32_t* seq_lens, int32_t B, int32_t n_h, int32_t d_h,
                                  int64_t max_ctx, float scale, void* workspace,
                                  size_t workspace_bytes, void* out, elitekv_stream_t stream) {
  if (!q_hat || !K_hat || !V || !seq_lens || !workspace || !out || B <= 0 || n_h <= 0 || max_ctx <= 0)
    return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)q_hat | (uintptr_t)K_hat | (uintptr_t)V | (uintptr_t)workspace) & 15)
    return ELITEKV_ERR_INVALID_ARG;
  size_t need;
  if (elitekv_mha_workspace_size(B, n_h, d_h, &need) != ELITEKV_OK) return ELITEKV_ERR_INVALID_ARG;
  if (workspace_bytes < need) return ELITEKV_ERR_WORKSPACE_TOO_SMALL;
  int sms;
  if (sm_count_current(&sms) != ELITEKV_OK) return ELITEKV_ERR_CUDA;
  const int S = mha_splits(B, n_h, sms);
  const float sc = (scale > 0.f ? scale : (float)(1.0 / sqrt((double)d_h))) * 1.4426950408889634f;
  cudaStream_t st = (cudaStream_t)stream;
  dim3 grid(S, (n_h + kMhaHeads - 1) / kMhaHeads, B);
  float* part = (float*)workspace;
#define EKV_MHA_CASE(LPT_)                                                                    \
  case LPT_ * 8:                                                                              \
    mha_split_kernel<LPT_><<<grid, kMhaHeads * 32, 0, st>>>((const bf16*)q_hat, (const bf16*)K_hat, \
        (const bf16*)V, seq_lens, n_h, max_ctx, sc, part);                                    \
    break;
  switch (d_h) {
    EKV_MHA_CASE(1)
    EKV_MHA_CASE(2)
    EKV_MHA_CASE(4)
    EKV_MHA_CASE(8)
    EKV_MHA_CASE(16)
    EKV_MHA_CASE(32)
    default: return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  }
#undef EKV_MHA_CASE
  EKV_CUDA_OK(cudaGetLastError());
  mha_combine_kernel<<<B * n_h, 128, 0, st>>>(part, S, d_h, (bf16*)out);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
