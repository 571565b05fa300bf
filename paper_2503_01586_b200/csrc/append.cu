// Fused RoPE + cache append (Section 3.1: the rotated elite chunks of the new token enter the
// cache once; Section 3.2: the shared latent row is stored beside them).
//
// One thread block per token (grid-stride, two tokens in flight per block).  Both rows move with
// 16-byte accesses: a work item is either 8 latent elements or 4 rope pairs.  For the pairs the
// thread reads the 4 un-rotated pairs and their 4 chunk ids, looks up (cos, sin) of
// pos*theta_{idx[h][j]} and writes the 4 rotated pairs in one store.  Every product and sum is
// rounded separately in fp32 (no fused multiply-add) so that the stored bits are a pure function
// of the table.  Layers whose rope row is not a multiple of 4 pairs take the pair-by-pair path.
//
// Prefill-sized calls (thousands of tokens) run the staged form instead: a block moves groups of
// tokens through a three-stage shared-memory ring with bulk asynchronous copies, one per row
// (un-rotated rope row and latent row in, cache rows out), so that two groups of loads are in
// flight behind the group being rotated and stored and no row passes through registers except
// the rope pairs while they are rotated in place.  Same arithmetic, same bits.
#include "tc_ptx.cuh"

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

// ------------------------------------------------------------------ staged form (prefill)
constexpr int kStages = 3;
constexpr int kStageBudget = 32 * 1024;   // bytes of token rows per stage
constexpr int kMaxGroup = 16;             // tokens per stage at most
constexpr int kStagedThreads = 128;

struct __align__(8) StagedBars {
  uint64_t full[kStages];
};

__device__ __forceinline__ void bulk_load_row(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store_row(void* dst, uint32_t src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
}

// Tokens per group G; group g of the call = tokens [g G, g G + G).  Block b takes groups b,
// b + gridDim.x, ...  In iteration `it` lane l < G of warp 0 issues the loads of its token of the
// block's it-th group, and the whole block rotates and stores the group loaded kStages - 1
// iterations earlier.  A stage is loaded again one iteration after its stores were issued; the
// issuing lane first waits until those stores have read the stage.
__global__ void __launch_bounds__(kStagedThreads)
append_staged_kernel(const AppendArgs a, int G) {
  extern __shared__ __align__(128) unsigned char smem_stage[];
  __shared__ StagedBars bars;
  __shared__ long long s_row[kStages][kMaxGroup];
  __shared__ int s_pos[kStages][kMaxGroup];
  __shared__ int s_abort_word;
  volatile int* s_abort = &s_abort_word;
  const int n_pairs = a.n_h * a.r;
  const uint32_t rope_bytes = (uint32_t)n_pairs * 4u, lat_bytes = (uint32_t)a.d_c * 2u;
  const uint32_t tok_bytes = rope_bytes + lat_bytes;          // a token's slot in a stage: rope row, then latent row
  const uint32_t stage_bytes = tok_bytes * (uint32_t)G;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) mbar_init(smem_u32(&bars.full[i]), (uint32_t)G);
    s_abort_word = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();
  const long long n_groups = (a.T + G - 1) / G;
  const long long mine = blockIdx.x < n_groups ? (n_groups - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  for (long long it = 0; it < mine + kStages - 1; ++it) {
    // ---- loads of the block's it-th group (warp 0, one lane per token)
    if (warp == 0 && lane < G && it < mine && !*s_abort) {
      const int st = (int)(it % kStages);
      bulk_wait_group_read<0>();        // this lane's stores out of the stage (previous iteration) have read it
      const long long t = (blockIdx.x + it * gridDim.x) * G + lane;
      long long row = -1;
      int p = 0;
      if (t < a.T) {                    // every lane owns a token here, so every lane records its own fault
        const int sq = a.seq_id[t];
        p = a.pos[t];
        if (p < 0 || p >= a.max_pos) {
          ekv_record(a.status, ELITEKV_ERR_BAD_POSITION, sq, p);
        } else {
          int code, detail;
          row = ekv_token_row(a.cv, sq, p, &code, &detail);
          if (row < 0) ekv_record(a.status, code, sq, detail);
        }
      }
      s_row[st][lane] = row;
      s_pos[st][lane] = p;
      const uint32_t fb = smem_u32(&bars.full[st]);
      if (row >= 0) {
        const uint32_t dst = smem_u32(smem_stage) + (uint32_t)st * stage_bytes + (uint32_t)lane * tok_bytes;
        mbar_expect_tx(fb, tok_bytes);
        if (rope_bytes) bulk_load_row(dst, a.k_e + t * n_pairs, rope_bytes, fb);
        bulk_load_row(dst + rope_bytes, a.c + t * (a.d_c >> 3), lat_bytes, fb);
      } else {
        mbar_arrive(fb);
      }
    }
    // ---- the group loaded kStages - 1 iterations ago: rotate in place, store
    const long long gp = it - (kStages - 1);
    if (gp >= 0) {
      const int st = (int)(gp % kStages);
      const bool ok = mbar_wait(smem_u32(&bars.full[st]), (uint32_t)((gp / kStages) & 1), s_abort, 1);
      unsigned char* stage = smem_stage + (size_t)st * stage_bytes;
      if (ok) {
        // work item = 4 pairs (16 bytes) of one token; four items per thread and pass, every
        // look-up of a pass issued before the first rotation
        const int n_rv = n_pairs >> 2, n_items = G * n_rv;
        for (int e0 = threadIdx.x; e0 < n_items; e0 += 4 * kStagedThreads) {
          uint4* pr[4];
          uint4 x[4];
          float2 w[4][4];
          bool on[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int e = e0 + u * kStagedThreads;
            on[u] = e < n_items;
            const int tt = on[u] ? e / n_rv : 0, v = on[u] ? e - tt * n_rv : 0;
            on[u] = on[u] && s_row[st][tt] >= 0;
            pr[u] = (uint4*)(stage + (size_t)tt * tok_bytes) + v;
            if (on[u]) {
              const int4 id = __ldg((const int4*)a.idx + v);
              const float2* csrow = a.cs + (long long)s_pos[st][tt] * a.half;
              w[u][0] = __ldg(csrow + id.x); w[u][1] = __ldg(csrow + id.y);
              w[u][2] = __ldg(csrow + id.z); w[u][3] = __ldg(csrow + id.w);
              x[u] = *pr[u];
            }
          }
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            if (!on[u]) continue;
            uint4 y;
            y.x = rotate_pair(x[u].x, w[u][0]); y.y = rotate_pair(x[u].y, w[u][1]);
            y.z = rotate_pair(x[u].z, w[u][2]); y.w = rotate_pair(x[u].w, w[u][3]);
            *pr[u] = y;
          }
        }
        fence_proxy_async();       // the rotated pairs, written by ordinary stores, are read by the bulk stores below
      }
      __syncthreads();
      if (ok && warp == 0 && lane < G) {
        const long long row = s_row[st][lane];
        if (row >= 0) {
          const uint32_t src = smem_u32(stage) + (uint32_t)lane * tok_bytes;
          if (rope_bytes) bulk_store_row(a.rope + row * n_pairs, src, rope_bytes);
          bulk_store_row(a.latent + row * (a.d_c >> 3), src + rope_bytes, lat_bytes);
        }
        bulk_commit_group();
      }
    } else {
      __syncthreads();
    }
  }
  if (warp == 0 && lane < G) bulk_wait_group_all();       // the cache rows are written before the block leaves
  __syncthreads();
  if (*s_abort) {
    drain_after_abort();
    if (threadIdx.x == 0) ekv_record(a.status, ELITEKV_ERR_TIMEOUT, (int)blockIdx.x, 0);
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
  // prefill-sized calls: the staged form (rows are whole 16-byte units, and the buffers are
  // 16-byte aligned: checked at the entry point)
  const long long tok_bytes = (long long)L->n_h * L->r * 4 + (long long)L->d_c * 2;
  if (T >= 2048 && (L->n_h * L->r) % 4 == 0 && tok_bytes <= kStageBudget) {
    int G = (int)(kStageBudget / tok_bytes);
    if (G > kMaxGroup) G = kMaxGroup;
    const size_t smem = (size_t)kStages * G * tok_bytes;
    const long long n_groups = (T + G - 1) / G;
    const long long want = (long long)L->sm_count * 2;       // two blocks of ~100 KB per SM
    EKV_CUDA_OK(cudaFuncSetAttribute(append_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    append_staged_kernel<<<(unsigned)(n_groups < want ? n_groups : want), kStagedThreads, smem, st>>>(a, G);
    EKV_CUDA_OK(cudaGetLastError());
    return ELITEKV_OK;
  }
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
