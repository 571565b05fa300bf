// Split combine + value up-projection.
//
// Each plan item left (m_s, l_s, acc_s[d_c]) per head, with m in base-2 log units.  For
// sequence b and head h (items s of b):
//   M = max_s m_s,  L = sum_s l_s 2^(m_s - M),  o_lat = sum_s acc_s 2^(m_s - M) / L
//   o[b,h,:] = o_lat . W_uv[:, h*d_h:(h+1)*d_h]        (B^v folded outwards, Section 5;
//                                                      V = c W_uv of Section 3.2)
//
// Fast kernel (d_h = 128, d_c % 128 == 0): grid (n_h, d_c/128).  A block owns one head and one
// 128-wide slice of the latent axis: it stages W_uv's [128 x 128] sub-block in shared memory
// once, then for every group of 16 sequences merges the items' partial outputs of its slice
// (16-byte loads, weights 2^(m_s-M)/L) and multiplies.  The d_c/128 slice results of a head are
// written to scratch; the block that finishes last for that (head, sequence group) adds them in
// a fixed order and writes bf16, so the result does not depend on scheduling.
//
// Generic kernel: any even d_h <= 512, any d_c; block per (head, 8 sequences).
//
// With several query rows per sequence the kernels see rows x heads "heads" (n_h below); entry
// i * heads + h multiplies with head h's columns of W_uv (n_phys = heads).
//
// With separated latents (S-LRD) the partial outputs span the value latent only; `d_c` below is
// then d_cv and W_uv is B^v_S.
#include "common.cuh"

namespace {

__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------ fast path
constexpr int kFB = 16;          // sequences per group
constexpr int kFK = 128;         // latent slice
constexpr int kFD = 128;         // head dim
constexpr int kFThreads = 256;
constexpr int kFI = 16;          // items per sequence whose merge weights are staged in shared memory
constexpr int kFStage = 448;     // items per sequence group whose (m, l) are staged in shared memory

__global__ void __launch_bounds__(kFThreads)
combine_fast_kernel(const float* part_acc, const float* part_ml,   // written by the split-K kernel while this
                                                                   // kernel may already be resident: read
                                                                   // with plain L2 loads, never ld.global.nc
                    const int32_t* seq_first, const bf16* __restrict__ Wuv,
                    float* __restrict__ slice_out /* [n_slices][B][n_h][128] */,
                    int32_t* __restrict__ counters /* [n_h][n_groups], zeroed by the plan kernel */,
                    bf16* __restrict__ out, int B, int n_h /* query rows x heads */, int n_phys /* heads */,
                    int d_c) {
  __shared__ __align__(16) bf16 s_w[kFK][kFD + 8];      // W_uv slice; rows padded by 16 bytes so that the
                                                        // fragment loads of the product spread over the banks
  __shared__ __align__(16) float s_x[kFB][kFK + 8];     // merged latent outputs (padded rows: bank spread)
  __shared__ float s_M[kFB], s_invL[kFB];
  __shared__ float s_wt[kFB][kFI];
  __shared__ float2 s_ml[kFStage];
  __shared__ int s_first[kFB + 1];
  __shared__ int s_last;
  const int h = blockIdx.x, slice = blockIdx.y, n_slices = gridDim.y;
  const int k0 = slice * kFK;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // W_uv[k0 + k][h*128 + d] -> shared, 16-byte asynchronous copies that land while the softmax
  // statistics of the first group are worked out
  for (int e = tid; e < kFK * (kFD / 8); e += kFThreads) {
    const int k = e / (kFD / 8), v = e % (kFD / 8);
    cp_async16(&s_w[k][v * 8], Wuv + (size_t)(k0 + k) * n_phys * kFD + (size_t)(h % n_phys) * kFD + v * 8);
  }
  cp_async_commit();
  const int n_groups = (B + kFB - 1) / kFB;
  // The plan (seq_first) was written before the split-K kernel started computing (that kernel
  // waited for it before it let this one be launched), so the first group's item ranges are
  // fetched while the split-K kernel is still running.
  if (tid <= min(kFB, B)) s_first[tid] = __ldcg(seq_first + tid);
  ekv_pdl_wait();         // everything below reads the split-K kernel's output

  for (int g = 0; g < n_groups; ++g) {
    const int b0 = g * kFB, nb = min(kFB, B - b0);
    __syncthreads();
    if (g > 0 && tid <= nb) s_first[tid] = __ldcg(seq_first + b0 + tid);
    __syncthreads();
    // (m, l) of the group's items for this head: one trip to global memory, then shared
    const int gi0 = s_first[0], gin = s_first[nb] - gi0;
    for (int e = tid; e < min(gin, kFStage); e += kFThreads)
      s_ml[e] = __ldcg((const float2*)(part_ml + ((size_t)(gi0 + e) * n_h + h) * 2));
    __syncthreads();
    auto item_ml = [&](int i) -> float2 {
      return i - gi0 < kFStage ? s_ml[i - gi0] : __ldcg((const float2*)(part_ml + ((size_t)i * n_h + h) * 2));
    };
    // softmax statistics per sequence: one warp each
    for (int bb = warp; bb < nb; bb += kFThreads / 32) {
      const int i0 = s_first[bb], i1 = s_first[bb + 1];
      float M = -INFINITY;
      for (int i = i0 + lane; i < i1; i += 32) M = fmaxf(M, item_ml(i).x);
      M = warp_max(M);
      float Ls = 0.f;
      for (int i = i0 + lane; i < i1; i += 32) {
        const float2 ml = item_ml(i);
        Ls += ml.y * exp2f(ml.x - M);
      }
      Ls = warp_sum(Ls);
      if (lane == 0) {
        s_M[bb] = M;
        s_invL[bb] = (i1 > i0 && Ls > 0.f) ? 1.f / Ls : 0.f;
      }
    }
    __syncthreads();
    // normalised merge weights 2^(m_s - M) / L of the first kFI items of every sequence
    for (int e = tid; e < kFB * kFI; e += kFThreads) {
      const int bb = e / kFI, j = e % kFI;
      float wv = 0.f;
      if (bb < nb) {
        const int i = s_first[bb] + j;
        if (i < s_first[bb + 1]) wv = exp2f(item_ml(i).x - s_M[bb]) * s_invL[bb];
      }
      s_wt[bb][j] = wv;
    }
    __syncthreads();
    // merge the items of each sequence on this latent slice (independent 16-byte loads)
    for (int e = tid; e < kFB * (kFK / 4); e += kFThreads) {
      const int bb = e / (kFK / 4), v = e % (kFK / 4);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      if (bb < nb) {
        const int i0 = s_first[bb], ni = s_first[bb + 1] - i0;
        const float* src = part_acc + ((size_t)i0 * n_h + h) * d_c + k0 + v * 4;
        const size_t stride = (size_t)n_h * d_c;
        const int nfast = min(ni, kFI);
        // eight independent 16-byte loads in flight per thread
        for (int j0 = 0; j0 < nfast; j0 += 8) {
          float4 p[8];
#pragma unroll
          for (int j = 0; j < 8; ++j)
            p[j] = j0 + j < nfast ? __ldcg((const float4*)(src + (size_t)(j0 + j) * stride)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float w = j0 + j < nfast ? s_wt[bb][j0 + j] : 0.f;
            acc.x = fmaf(w, p[j].x, acc.x); acc.y = fmaf(w, p[j].y, acc.y);
            acc.z = fmaf(w, p[j].z, acc.z); acc.w = fmaf(w, p[j].w, acc.w);
          }
        }
        for (int j = kFI; j < ni; ++j) {     // rare: a sequence cut into more than kFI items
          const float w = exp2f(item_ml(i0 + j).x - s_M[bb]) * s_invL[bb];
          const float4 p = __ldcg((const float4*)(src + (size_t)j * stride));
          acc.x = fmaf(w, p.x, acc.x); acc.y = fmaf(w, p.y, acc.y);
          acc.z = fmaf(w, p.z, acc.z); acc.w = fmaf(w, p.w, acc.w);
        }
      }
      *(float4*)&s_x[bb][v * 4] = acc;
    }
    cp_async_wait<0>();      // the W_uv slice (first group only; later a no-op)
    __syncthreads();
    // [16 x 128] . [128 x 128] on mma.sync (m16n8k16, bf16 in, fp32 accumulate): one warp per 16
    // output dims.  The fp32 rows of x are fed as a bf16 head plus a bf16 remainder (two MMAs),
    // so nothing but the last ~2^-17 of x is lost; W_uv is bf16 as stored.
    {
      const int g = lane >> 2, t = lane & 3, n0 = warp * 16;
      float acc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll 2
      for (int kk = 0; kk < kFK; kk += 16) {
        uint32_t ahi[4], alo[4];
#pragma unroll
        for (int f = 0; f < 4; ++f) {
          const float2 x = *(const float2*)&s_x[g + (f & 1) * 8][kk + 2 * t + (f >> 1) * 8];
          const bf162 hi = __floats2bfloat162_rn(x.x, x.y);
          const float2 hf = __bfloat1622float2(hi);
          const bf162 lo = __floats2bfloat162_rn(x.x - hf.x, x.y - hf.y);
          ahi[f] = *(const uint32_t*)&hi;
          alo[f] = *(const uint32_t*)&lo;
        }
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const unsigned short* wp = (const unsigned short*)&s_w[kk + 2 * t][n0 + nt * 8 + g];
          const uint32_t b0r = (uint32_t)wp[0] | ((uint32_t)wp[kFD + 8] << 16);
          const uint32_t b1r = (uint32_t)wp[8 * (kFD + 8)] | ((uint32_t)wp[9 * (kFD + 8)] << 16);
          mma_bf16_16816(acc[nt], ahi, b0r, b1r);
          mma_bf16_16816(acc[nt], alo, b0r, b1r);
        }
      }
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int d = n0 + nt * 8 + 2 * t;
        if (g < nb)
          *(float2*)(slice_out + (((size_t)slice * B + b0 + g) * n_h + h) * kFD + d) = make_float2(acc[nt][0], acc[nt][1]);
        if (g + 8 < nb)
          *(float2*)(slice_out + (((size_t)slice * B + b0 + g + 8) * n_h + h) * kFD + d) = make_float2(acc[nt][2], acc[nt][3]);
      }
    }
    // last block of this (head, group) adds the slices in order
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&counters[h * n_groups + g], 1) == n_slices - 1;
    __syncthreads();
    if (s_last) {
      __threadfence();
      for (int e = tid; e < nb * (kFD / 2); e += kFThreads) {
        const int bb = e / (kFD / 2), p2 = e % (kFD / 2);
        float2 v = make_float2(0.f, 0.f);
        for (int s = 0; s < n_slices; ++s) {
          const float2 t = __ldcg((const float2*)(slice_out + (((size_t)s * B + b0 + bb) * n_h + h) * kFD + 2 * p2));
          v.x += t.x;
          v.y += t.y;
        }
        *(bf162*)(out + ((size_t)(b0 + bb) * n_h + h) * kFD + 2 * p2) = __floats2bfloat162_rn(v.x, v.y);
      }
    }
  }
}

// ------------------------------------------------------------------ generic path
constexpr int kCombBatch = 8;
constexpr int kCombThreads = 256;
constexpr int kCombChunk = 128;

__global__ void __launch_bounds__(kCombThreads)
combine_upproj_kernel(const float* __restrict__ part_acc, const float* __restrict__ part_ml,
                      const int32_t* __restrict__ seq_first, const bf16* __restrict__ Wuv,
                      bf16* __restrict__ out, int B, int n_h /* query rows x heads */, int n_phys /* heads */,
                      int d_h, int d_c) {
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
            *(const bf162*)(Wuv + (size_t)(k0 + k) * n_phys * d_h + (size_t)(h % n_phys) * d_h + 2 * pair));
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

int ekv_combine_fast_ok(const elitekv_layer* L) { return L->d_h == kFD && L->vw % kFK == 0; }

size_t ekv_combine_scratch_bytes(const elitekv_layer* L, int B) {
  if (!ekv_combine_fast_ok(L)) return 0;
  return sizeof(float) * (size_t)(L->vw / kFK) * B * L->n_h * kFD;
}

int ekv_combine_counters(const elitekv_layer* L, int B) {
  return ekv_combine_fast_ok(L) ? L->n_h * ((B + kFB - 1) / kFB) : 0;
}

int ekv_launch_combine(const elitekv_layer* L, int B, const DecodeScratch& ws, void* out,
                       cudaStream_t st) {
  // several query rows per sequence: row i, head h is "head" i * n_h + h of the partial results
  // and of the output; it uses head h's slice of W_uv
  const int nv = (ws.rows > 0 ? ws.rows : 1) * L->n_h;
  if (ekv_combine_fast_ok(L)) {
    dim3 grid(nv, L->vw / kFK);
    EKV_CUDA_OK(ekv_launch_pdl(combine_fast_kernel, grid, dim3(kFThreads), 0, st, (const float*)ws.part_acc,
                               (const float*)ws.part_ml, (const int32_t*)ws.seq_first, (const bf16*)L->d_Wuv,
                               ws.slice_out, ws.counters, (bf16*)out, B, nv, L->n_h, L->vw));
    EKV_CUDA_OK(cudaGetLastError());
    return ELITEKV_OK;
  }
  const int npair = L->d_h / 2;
  if (npair > kCombThreads) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  const int kgroups = kCombThreads / npair > 0 ? kCombThreads / npair : 1;
  const size_t smem = sizeof(float) * (size_t)kgroups * kCombBatch * L->d_h;
  dim3 grid(nv, (B + kCombBatch - 1) / kCombBatch);
  EKV_CUDA_OK(cudaFuncSetAttribute(combine_upproj_kernel,
                                   cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  combine_upproj_kernel<<<grid, kCombThreads, smem, st>>>(ws.part_acc, ws.part_ml, ws.seq_first,
                                                          L->d_Wuv, (bf16*)out, B, nv, L->n_h, L->d_h,
                                                          L->vw);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}
