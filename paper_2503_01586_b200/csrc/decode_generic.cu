// Generic split-K decode kernel on CUDA cores: works for every shape the layer object accepts
// (any n_h, r <= d_h/2, d_c a multiple of 8 up to 3072) and serves the shapes the tensor-core
// kernel does not cover.
//
// A block takes one plan item (a token range of one sequence) and a group of 8 heads, one warp
// per head.  Token sub-tiles are staged in shared memory with cp.async (two stages); the warp
// keeps the head's absorbed query and its running output (sum_t p_t c_t, fp32) in registers,
// lane l owning the latent coordinates {(ch*32 + l)*8 .. +8}.  Per token:
//   s = q_rope . k_rope[t,h] + q_abs . c[t]          (score equation of Section 3.1 with B^k
//                                                    folded into the query, Section 5)
//   online softmax in base 2, acc += p * c[t]        (Section 2.1; c is both K and V source,
//                                                    Section 3.2)
// Four tokens are processed together to give the warp independent dependency chains.
// The block writes (m, l, acc) of its item; the combine kernel merges items and applies W_uv.
#include "common.cuh"

namespace {

constexpr int kHeadsPerBlock = 8;
constexpr int kThreads = kHeadsPerBlock * 32;
constexpr int kTokBatch = 4;

struct GenericArgs {
  const bf16* rope;
  const bf16* latent;
  CacheView cv;
  const bf16* q_rope;     // [B][n_h][2r]
  const bf16* q_abs;      // [B][n_h][kw]
  const int32_t* items;   // [max_items][4]
  float* part_acc;
  float* part_ml;
  int32_t* status;
  int n_h, r2, d_c, sub_tokens;
  int kw, voff, vw;       // latent columns of the scores [0, kw) and of the outputs [voff, voff + vw)
  float scale_log2e;
};

template <int NCH>
__global__ void __launch_bounds__(kThreads)
decode_generic_kernel(const GenericArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int item = blockIdx.x;
  const int seq = a.items[4 * item + 0];
  if (seq < 0) return;
  const int tok0 = a.items[4 * item + 1];
  const int ntok = a.items[4 * item + 2];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int hg0 = blockIdx.y * kHeadsPerBlock;
  const int hcount = min(kHeadsPerBlock, a.n_h - hg0);
  const int h = hg0 + warp;
  const bool active = warp < hcount;
  const int d_c = a.d_c, r2 = a.r2, T = a.sub_tokens;
  const int rope_w = hcount * r2;                       // rope elements per token for this group
  const int rope_w_pad = (kHeadsPerBlock * r2 + 7) & ~7;
  // smem: [2][T][d_c] latent, then [2][T][rope_w_pad] rope
  bf16* s_lat = (bf16*)smem_raw;
  bf16* s_rope = s_lat + (size_t)2 * T * d_c;
  __shared__ long long s_rows[2][64];

  // query registers
  bf162 qa[NCH][4];
  float qr[4];
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch) {
    const int d = (ch * 32 + lane) * 8;
    uint4 v = make_uint4(0, 0, 0, 0);
    // columns the scores do not read (the value latent of S-LRD) get a zero query
    if (active && d < a.kw) v = *(const uint4*)(a.q_abs + ((size_t)seq * a.n_h + h) * a.kw + d);
    qa[ch][0] = *(bf162*)&v.x; qa[ch][1] = *(bf162*)&v.y; qa[ch][2] = *(bf162*)&v.z; qa[ch][3] = *(bf162*)&v.w;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int e = lane + 32 * k;
    qr[k] = (active && e < r2) ? __bfloat162float(a.q_rope[((size_t)seq * a.n_h + h) * r2 + e]) : 0.f;
  }

  float acc[NCH][8];
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[ch][e] = 0.f;
  float m_run = -INFINITY, l_run = 0.f;

  const int n_sub = (ntok + T - 1) / T;
  const bool rope_vec = ((r2 & 7) == 0) && (((hg0 * r2) & 7) == 0) && (((a.n_h * r2) & 7) == 0);
  const int lat_vecs = d_c >> 3;

  auto stage_load = [&](int sub, int buf) {
    const int t_base = tok0 + sub * T;
    const int nt = min(T, ntok - sub * T);
    // resolve rows (first T threads)
    if (threadIdx.x < T) {
      long long row = -1;
      if (threadIdx.x < nt) {
        int code, detail;
        row = ekv_token_row(a.cv, seq, t_base + threadIdx.x, &code, &detail);
        if (row < 0) ekv_record(a.status, code, seq, detail);
      }
      s_rows[buf][threadIdx.x] = row;
    }
    __syncthreads();
    bf16* dl = s_lat + (size_t)buf * T * d_c;
    bf16* dr = s_rope + (size_t)buf * T * rope_w_pad;
    for (int e = threadIdx.x; e < T * lat_vecs; e += kThreads) {
      const int tt = e / lat_vecs, v = e - tt * lat_vecs;
      const long long row = s_rows[buf][tt];
      bf16* dst = dl + (size_t)tt * d_c + v * 8;
      if (row >= 0) cp_async16(dst, a.latent + row * d_c + v * 8);
      else *(uint4*)dst = make_uint4(0, 0, 0, 0);
    }
    if (rope_vec) {
      const int rv = rope_w >> 3;
      for (int e = threadIdx.x; e < T * rv; e += kThreads) {
        const int tt = e / rv, v = e - tt * rv;
        const long long row = s_rows[buf][tt];
        bf16* dst = dr + (size_t)tt * rope_w_pad + v * 8;
        if (row >= 0) cp_async16(dst, a.rope + row * ((long long)a.n_h * r2) + hg0 * r2 + v * 8);
        else *(uint4*)dst = make_uint4(0, 0, 0, 0);
      }
    } else {
      for (int e = threadIdx.x; e < T * rope_w; e += kThreads) {
        const int tt = e / rope_w, v = e - tt * rope_w;
        const long long row = s_rows[buf][tt];
        dr[(size_t)tt * rope_w_pad + v] =
            row >= 0 ? a.rope[row * ((long long)a.n_h * r2) + hg0 * r2 + v] : __float2bfloat16(0.f);
      }
    }
    cp_async_commit();
  };

  stage_load(0, 0);
  for (int sub = 0; sub < n_sub; ++sub) {
    const int buf = sub & 1;
    if (sub + 1 < n_sub) {
      stage_load(sub + 1, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const int nt = min(T, ntok - sub * T);
    if (active) {
      const bf16* tl = s_lat + (size_t)buf * T * d_c;
      const bf16* tr = s_rope + (size_t)buf * T * rope_w_pad + warp * r2;
      for (int tt0 = 0; tt0 < nt; tt0 += kTokBatch) {
        float s[kTokBatch];
#pragma unroll
        for (int u = 0; u < kTokBatch; ++u) {
          const int tt = tt0 + u;          // rows >= nt were zero-filled or are stale but finite? -> masked below
          float sum = 0.f;
          if (tt < nt) {
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {
              const int d = (ch * 32 + lane) * 8;
              if (d < d_c) {
                const uint4 v = *(const uint4*)(tl + (size_t)tt * d_c + d);
                const bf162* cv = (const bf162*)&v;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float2 x = __bfloat1622float2(cv[e]);
                  const float2 w = __bfloat1622float2(qa[ch][e]);
                  sum = fmaf(x.x, w.x, sum);
                  sum = fmaf(x.y, w.y, sum);
                }
              }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int e = lane + 32 * k;
              if (e < r2) sum = fmaf(qr[k], __bfloat162float(tr[(size_t)tt * rope_w_pad + e]), sum);
            }
          }
          s[u] = sum;
        }
#pragma unroll
        for (int u = 0; u < kTokBatch; ++u) {
          s[u] = warp_sum(s[u]) * a.scale_log2e;
          if (tt0 + u >= nt) s[u] = -INFINITY;
        }
        float m_new = m_run;
#pragma unroll
        for (int u = 0; u < kTokBatch; ++u) m_new = fmaxf(m_new, s[u]);
        const float corr = exp2f(m_run - m_new);     // 0 on the first batch (m_run = -inf)
        float p[kTokBatch];
        float psum = 0.f;
#pragma unroll
        for (int u = 0; u < kTokBatch; ++u) {
          p[u] = exp2f(s[u] - m_new);
          psum += p[u];
        }
        l_run = l_run * corr + psum;
        m_run = m_new;
#pragma unroll
        for (int ch = 0; ch < NCH; ++ch) {
          const int d = (ch * 32 + lane) * 8;
          if (d < d_c) {
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[ch][e] *= corr;
#pragma unroll
            for (int u = 0; u < kTokBatch; ++u) {
              if (tt0 + u < nt) {
                const uint4 v = *(const uint4*)(tl + (size_t)(tt0 + u) * d_c + d);
                const bf162* cv = (const bf162*)&v;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float2 x = __bfloat1622float2(cv[e]);
                  acc[ch][2 * e] = fmaf(p[u], x.x, acc[ch][2 * e]);
                  acc[ch][2 * e + 1] = fmaf(p[u], x.y, acc[ch][2 * e + 1]);
                }
              }
            }
          }
        }
      }
    }
    __syncthreads();
  }

  if (active) {
    float* pa = a.part_acc + ((size_t)item * a.n_h + h) * a.vw;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int d = (ch * 32 + lane) * 8 - a.voff;      // only the columns the outputs read leave the block
      if (d >= 0 && d < a.vw) {
        *(float4*)(pa + d) = make_float4(acc[ch][0], acc[ch][1], acc[ch][2], acc[ch][3]);
        *(float4*)(pa + d + 4) = make_float4(acc[ch][4], acc[ch][5], acc[ch][6], acc[ch][7]);
      }
    }
    if (lane == 0) {
      a.part_ml[((size_t)item * a.n_h + h) * 2 + 0] = m_run;
      a.part_ml[((size_t)item * a.n_h + h) * 2 + 1] = l_run;
    }
  }
}

int pick_sub_tokens(const elitekv_layer* L) {
  const int rope_w_pad = (kHeadsPerBlock * 2 * L->r + 7) & ~7;
  const size_t per_tok = 2 * (size_t)(L->d_c + rope_w_pad) * sizeof(bf16);   // two stages
  const size_t budget = 96 * 1024;
  int T = 64;
  while (T > kTokBatch && per_tok * T > budget) T >>= 1;
  return T;
}

template <int NCH>
int launch_nch(const elitekv_layer* L, const GenericArgs& a, dim3 grid, size_t smem, cudaStream_t st) {
  EKV_CUDA_OK(cudaFuncSetAttribute(decode_generic_kernel<NCH>,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  decode_generic_kernel<NCH><<<grid, kThreads, smem, st>>>(a);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

}  // namespace

int ekv_generic_supported(const elitekv_layer* L) {
  return L->d_c <= 3072 && 2 * L->r <= 128;
}

int ekv_generic_max_items(const elitekv_layer* L, int B) {
  const int groups = (L->n_h + kHeadsPerBlock - 1) / kHeadsPerBlock;
  int items = (4 * L->sm_count + groups - 1) / groups;   // about four blocks per SM in flight
  if (items < 1) items = 1;
  return items + B;
}

int ekv_launch_decode_generic(const elitekv_layer* L, const elitekv_cache* cache,
                              const CacheView& cv, const void* q_rope, const void* q_abs, int B,
                              const DecodeScratch& ws, cudaStream_t st) {
  if (!ekv_generic_supported(L)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if (ws.rows > 1) return ELITEKV_ERR_UNSUPPORTED_SHAPE;      // one query row per sequence here
  GenericArgs a;
  a.rope = (const bf16*)cache->rope;
  a.latent = (const bf16*)cache->latent;
  a.cv = cv;
  a.q_rope = (const bf16*)q_rope;
  a.q_abs = (const bf16*)q_abs;
  a.items = ws.items;
  a.part_acc = ws.part_acc;
  a.part_ml = ws.part_ml;
  a.status = L->d_status;
  a.n_h = L->n_h;
  a.r2 = 2 * L->r;
  a.d_c = L->d_c;
  a.kw = L->kw;
  a.voff = L->voff;
  a.vw = L->vw;
  a.sub_tokens = pick_sub_tokens(L);
  a.scale_log2e = L->scale * 1.4426950408889634f;
  const int rope_w_pad = (kHeadsPerBlock * a.r2 + 7) & ~7;
  const size_t smem = 2 * (size_t)a.sub_tokens * (L->d_c + rope_w_pad) * sizeof(bf16);
  dim3 grid(ws.max_items, (L->n_h + kHeadsPerBlock - 1) / kHeadsPerBlock);
  const int nch = (L->d_c + 255) / 256;
  if (nch <= 1) return launch_nch<1>(L, a, grid, smem, st);
  if (nch <= 2) return launch_nch<2>(L, a, grid, smem, st);
  if (nch <= 3) return launch_nch<3>(L, a, grid, smem, st);
  if (nch <= 4) return launch_nch<4>(L, a, grid, smem, st);
  if (nch <= 6) return launch_nch<6>(L, a, grid, smem, st);
  if (nch <= 8) return launch_nch<8>(L, a, grid, smem, st);
  return launch_nch<12>(L, a, grid, smem, st);
}
