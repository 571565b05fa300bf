// Fused RoPE + cache append (Section 3.1: the rotated elite chunks of the new token enter the
// cache once; Section 3.2: the shared latent row is stored beside them).
//
// One thread block per token (grid-stride, two tokens in flight per block).  Both rows move with
// 16-byte accesses: a work item is either 8 latent elements or 4 rope pairs.  For the pairs the
// thread reads the 4 un-rotated pairs and their 4 chunk ids, looks up (cos, sin) of
// pos*theta_{idx[h][j]} and writes the 4 rotated pairs in one store.  Every product and sum is
// rounded separately in fp32 (no fused multiply-add) so that the stored bits are a pure function
// of the table.  Layers whose rope row is not a multiple of 4 pairs take the pair-by-pair path.
#include "common.cuh"

namespace {

struct AppendArgs {
  const bf162* k_e;
  const uint4* c;
  const int32_t* seq_id;
  const int32_t* pos;
  long long T;
  bf162* rope;
  uint4* latent;
  CacheView cv;
  const int32_t* idx;
  const float2* cs;
  int n_h, r, d_c, half, max_pos;
  int32_t* status;
};

// cache row of token t, or -1 (fault recorded by thread 0)
__device__ __forceinline__ long long append_row(const AppendArgs& a, long long t, int* p_out) {
  const int s = a.seq_id[t], p = a.pos[t];
  *p_out = p;
  if (p < 0 || p >= a.max_pos) {
    if (threadIdx.x == 0) ekv_record(a.status, ELITEKV_ERR_BAD_POSITION, s, p);
    return -1;
  }
  int code, detail;
  const long long row = ekv_token_row(a.cv, s, p, &code, &detail);
  if (row < 0 && threadIdx.x == 0) ekv_record(a.status, code, s, detail);
  return row;
}

__device__ __forceinline__ uint32_t rotate_pair(uint32_t raw, float2 w) {
  const float2 x = __bfloat1622float2(*(const bf162*)&raw);
  const float y0 = __fsub_rn(__fmul_rn(x.x, w.x), __fmul_rn(x.y, w.y));
  const float y1 = __fadd_rn(__fmul_rn(x.x, w.y), __fmul_rn(x.y, w.x));
  const bf162 y = __floats2bfloat162_rn(y0, y1);
  return *(const uint32_t*)&y;
}

constexpr int kTok = 2;      // tokens a block works on at once (independent 16-byte loads per thread;
                             // four were measured slower: the registers cost more occupancy than the
                             // extra loads in flight bring)

template <bool kVec>
__global__ void __launch_bounds__(256)
append_kernel(const AppendArgs a) {
  const int n_pairs = a.n_h * a.r;
  const int n_vec = a.d_c >> 3;
  const int n_rv = kVec ? n_pairs >> 2 : 0;
  const int n_items = n_vec + n_rv;
  for (long long t0 = blockIdx.x; t0 < a.T; t0 += (long long)kTok * gridDim.x) {
    long long tk[kTok], row[kTok];
    int p[kTok];
#pragma unroll
    for (int e = 0; e < kTok; ++e) {
      tk[e] = t0 + (long long)e * gridDim.x;
      p[e] = 0;
      row[e] = tk[e] < a.T ? append_row(a, tk[e], &p[e]) : -1;
    }
    for (int v = threadIdx.x; v < n_items; v += blockDim.x) {
      // loads of all tokens first, then the arithmetic and the stores
      uint4 x[kTok];
      int4 id[kTok];
      const bool lat = v < n_vec;
#pragma unroll
      for (int e = 0; e < kTok; ++e) {
        if (row[e] < 0) continue;
        if (lat) {
          x[e] = __ldcs(a.c + tk[e] * n_vec + v);
        } else {
          x[e] = __ldcs((const uint4*)(a.k_e + tk[e] * n_pairs) + (v - n_vec));
          id[e] = __ldg((const int4*)a.idx + (v - n_vec));
        }
      }
#pragma unroll
      for (int e = 0; e < kTok; ++e) {
        if (row[e] < 0) continue;
        if (lat) {
          a.latent[row[e] * n_vec + v] = x[e];
        } else {
          const float2* csrow = a.cs + (long long)p[e] * a.half;
          uint4 y;
          y.x = rotate_pair(x[e].x, __ldg(csrow + id[e].x));
          y.y = rotate_pair(x[e].y, __ldg(csrow + id[e].y));
          y.z = rotate_pair(x[e].z, __ldg(csrow + id[e].z));
          y.w = rotate_pair(x[e].w, __ldg(csrow + id[e].w));
          ((uint4*)(a.rope + row[e] * n_pairs))[v - n_vec] = y;
        }
      }
    }
    if (!kVec) {
#pragma unroll
      for (int e = 0; e < kTok; ++e) {
        if (row[e] < 0) continue;
        const bf162* ksrc = a.k_e + tk[e] * n_pairs;
        bf162* kdst = a.rope + row[e] * n_pairs;
        const float2* csrow = a.cs + (long long)p[e] * a.half;
        for (int q = threadIdx.x; q < n_pairs; q += blockDim.x) {
          const uint32_t y = rotate_pair(*(const uint32_t*)(ksrc + q), __ldg(csrow + __ldg(a.idx + q)));
          kdst[q] = *(const bf162*)&y;
        }
      }
    }
  }
}

}  // namespace

int ekv_launch_append(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                      const void* k_e, const void* c, const int32_t* seq_id, const int32_t* pos,
                      long long T, cudaStream_t st) {
  if (T == 0) return ELITEKV_OK;
  AppendArgs a;
  a.k_e = (const bf162*)k_e;
  a.c = (const uint4*)c;
  a.seq_id = seq_id;
  a.pos = pos;
  a.T = T;
  a.rope = (bf162*)cache->rope;
  a.latent = (uint4*)cache->latent;
  a.cv = cv;
  a.idx = L->d_idx;
  a.cs = L->d_cs;
  a.n_h = L->n_h;
  a.r = L->r;
  a.d_c = L->d_c;
  a.half = L->d_h / 2;
  a.max_pos = L->max_pos;
  a.status = L->d_status;
  const long long groups = (T + kTok - 1) / kTok;
  long long blocks = groups < (long long)L->sm_count * 8 ? groups : (long long)L->sm_count * 8;
  // 16-byte rope accesses need rows of whole 4-pair groups (the buffers themselves are 16-byte
  // aligned: checked at the entry point)
  if ((L->n_h * L->r) % 4 == 0 && L->r > 0)
    append_kernel<true><<<(unsigned)blocks, 256, 0, st>>>(a);
  else
    append_kernel<false><<<(unsigned)blocks, 256, 0, st>>>(a);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
