// Layer object: validation, RoPE (cos, sin) table, index tables, weight regrouping, status word.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include <stdio.h>

#include "common.cuh"

namespace {

// W_uk [d_c][n_h*dn]  ->  WukT [n_h][dn][d_c]   (d_c becomes the contiguous axis so that the
// absorption kernel reads it coalesced with one thread per latent coordinate).
__global__ void regroup_wuk_kernel(const bf16* __restrict__ W, bf16* __restrict__ Wt, int d_c,
                                   int ncols) {
  __shared__ bf16 tile[32][33];
  const int col0 = blockIdx.x * 32, row0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    int rr = row0 + i, cc = col0 + threadIdx.x;
    tile[i][threadIdx.x] = (rr < d_c && cc < ncols) ? W[(size_t)rr * ncols + cc] : __float2bfloat16(0.f);
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += blockDim.y) {
    int cc = col0 + i, rr = row0 + threadIdx.x;   // cc = h*dn + j
    if (rr < d_c && cc < ncols) Wt[(size_t)cc * d_c + rr] = tile[threadIdx.x][i];
  }
}

}  // namespace

extern "C" int elitekv_layer_create(const elitekv_params* p, elitekv_layer** out) {
  if (!p || !out) return ELITEKV_ERR_INVALID_ARG;
  if (p->n_h <= 0 || p->d_h <= 0 || (p->d_h & 1) || p->r < 0 || 2 * p->r > p->d_h || p->d_c <= 0)
    return ELITEKV_ERR_INVALID_ARG;
  if (p->r > 0 && !p->elite_idx) return ELITEKV_ERR_INVALID_ARG;
  if (!p->W_uv || (p->d_h - 2 * p->r > 0 && !p->W_uk)) return ELITEKV_ERR_INVALID_ARG;
  if (p->max_pos <= 0 || !(p->rope_base > 0.f)) return ELITEKV_ERR_INVALID_ARG;
  if (p->pair_mode != 0 && p->pair_mode != 1) return ELITEKV_ERR_INVALID_ARG;
  if (p->decode_kernel < 0 || p->decode_kernel > 3) return ELITEKV_ERR_INVALID_ARG;
  if (p->d_c % 8 != 0 || p->d_h > 512) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if (p->d_ck < 0 || p->d_ck >= p->d_c) return ELITEKV_ERR_INVALID_ARG;
  if (p->d_ck % 8 != 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if (((uintptr_t)p->W_uv & 15) || ((uintptr_t)p->W_uk & 15)) return ELITEKV_ERR_INVALID_ARG;
  if (p->d < 0 || (p->d > 0 && (!p->W_down || (p->r > 0 && !p->W_ke)))) return ELITEKV_ERR_INVALID_ARG;
  const int n_h = p->n_h, d_h = p->d_h, r = p->r, half = d_h / 2;

  // index sets: in range, distinct per head; dims of the query each cache slot pairs with
  std::vector<int32_t> qdims((size_t)n_h * d_h);
  for (int h = 0; h < n_h; ++h) {
    std::vector<char> used(d_h, 0);
    for (int j = 0; j < r; ++j) {
      int i = p->elite_idx[h * r + j];
      if (i < 0 || i >= half) return ELITEKV_ERR_INVALID_ARG;
      int a = p->pair_mode == 0 ? 2 * i : i;
      int b = p->pair_mode == 0 ? 2 * i + 1 : i + half;
      if (used[a] || used[b]) return ELITEKV_ERR_INVALID_ARG;
      used[a] = used[b] = 1;
      qdims[(size_t)h * d_h + 2 * j] = a;
      qdims[(size_t)h * d_h + 2 * j + 1] = b;
    }
    int w = 2 * r;
    for (int d = 0; d < d_h; ++d)
      if (!used[d]) qdims[(size_t)h * d_h + w++] = d;
  }

  elitekv_layer* L = (elitekv_layer*)calloc(1, sizeof(elitekv_layer));
  if (!L) return ELITEKV_ERR_CUDA;
  L->n_h = n_h; L->d_h = d_h; L->r = r; L->d_c = p->d_c; L->dn = d_h - 2 * r;
  L->kw = p->d_ck > 0 ? p->d_ck : p->d_c;
  L->voff = p->d_ck > 0 ? p->d_ck : 0;
  L->vw = p->d_c - L->voff;
  L->rope_base = p->rope_base;
  L->scale = p->softmax_scale > 0.f ? p->softmax_scale : (float)(1.0 / sqrt((double)d_h));
  L->pair_mode = p->pair_mode; L->max_pos = p->max_pos; L->decode_kernel = p->decode_kernel;

  L->last_detail = (int32_t*)calloc(3, sizeof(int32_t));
  int rc = ELITEKV_ERR_CUDA;
  do {
    if (!L->last_detail) break;
    if (cudaGetDevice(&L->device) != cudaSuccess) break;
    if (cudaDeviceGetAttribute(&L->sm_count, cudaDevAttrMultiProcessorCount, L->device) != cudaSuccess) break;
    if (cudaDeviceGetAttribute(&L->smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, L->device) != cudaSuccess) break;
    if (cudaMalloc(&L->d_status, 4 * sizeof(int32_t)) != cudaSuccess) break;
    if (cudaMemset(L->d_status, 0, 4 * sizeof(int32_t)) != cudaSuccess) break;
    if (cudaMalloc(&L->d_qdims, qdims.size() * sizeof(int32_t)) != cudaSuccess) break;
    if (cudaMemcpy(L->d_qdims, qdims.data(), qdims.size() * sizeof(int32_t), cudaMemcpyHostToDevice) != cudaSuccess) break;
    if (cudaMalloc(&L->d_idx, sizeof(int32_t) * (size_t)(n_h * r > 0 ? n_h * r : 1)) != cudaSuccess) break;
    if (r > 0 && cudaMemcpy(L->d_idx, p->elite_idx, sizeof(int32_t) * (size_t)n_h * r, cudaMemcpyHostToDevice) != cudaSuccess) break;

    if (p->cos_sin) {
      L->d_cs = (const float2*)p->cos_sin;
    } else {
      // theta_i = base^(-2i/d_h); (cos, sin)(pos*theta_i) in double, rounded once to float
      size_t n = (size_t)p->max_pos * half;
      std::vector<float2> tab(n);
      std::vector<double> theta(half);
      for (int i = 0; i < half; ++i) theta[i] = pow((double)p->rope_base, -2.0 * i / (double)d_h);
      for (int pos = 0; pos < p->max_pos; ++pos)
        for (int i = 0; i < half; ++i) {
          double a = (double)pos * theta[i];
          tab[(size_t)pos * half + i] = make_float2((float)cos(a), (float)sin(a));
        }
      if (cudaMalloc(&L->d_cs_owned, n * sizeof(float2)) != cudaSuccess) break;
      if (cudaMemcpy(L->d_cs_owned, tab.data(), n * sizeof(float2), cudaMemcpyHostToDevice) != cudaSuccess) break;
      L->d_cs = L->d_cs_owned;
    }

    size_t wuv_elems = (size_t)L->vw * n_h * d_h;
    if (cudaMalloc(&L->d_Wuv, wuv_elems * sizeof(bf16)) != cudaSuccess) break;
    if (cudaMemcpy(L->d_Wuv, p->W_uv, wuv_elems * sizeof(bf16), cudaMemcpyDeviceToDevice) != cudaSuccess) break;
    if (L->dn > 0) {
      size_t wuk_elems = (size_t)L->kw * n_h * L->dn;
      if (cudaMalloc(&L->d_WukT, wuk_elems * sizeof(bf16)) != cudaSuccess) break;
      dim3 grid((n_h * L->dn + 31) / 32, (L->kw + 31) / 32), block(32, 8);
      regroup_wuk_kernel<<<grid, block>>>((const bf16*)p->W_uk, L->d_WukT, L->kw, n_h * L->dn);
      if (cudaGetLastError() != cudaSuccess) break;
    }
    if (p->d > 0) {
      // [W^k_e | A^kv] with the output column as the row, so that a tile of it is a K-major operand
      const int rope_w = n_h * 2 * r;
      const size_t n_out = (size_t)rope_w + p->d_c;
      L->d = p->d;
      if (cudaMalloc(&L->d_WcatT, n_out * p->d * sizeof(bf16)) != cudaSuccess) break;
      dim3 block(32, 8);
      if (rope_w > 0) {
        dim3 grid((rope_w + 31) / 32, (p->d + 31) / 32);
        regroup_wuk_kernel<<<grid, block>>>((const bf16*)p->W_ke, L->d_WcatT, p->d, rope_w);
      }
      dim3 grid2((p->d_c + 31) / 32, (p->d + 31) / 32);
      regroup_wuk_kernel<<<grid2, block>>>((const bf16*)p->W_down, L->d_WcatT + (size_t)rope_w * p->d, p->d, p->d_c);
      if (cudaGetLastError() != cudaSuccess) break;
    }
    if (cudaStreamCreateWithFlags(&L->side, cudaStreamNonBlocking) != cudaSuccess) break;
    if (cudaEventCreateWithFlags(&L->ev_fork, cudaEventDisableTiming) != cudaSuccess) break;
    if (cudaEventCreateWithFlags(&L->ev_join, cudaEventDisableTiming) != cudaSuccess) break;
    if (cudaDeviceSynchronize() != cudaSuccess) break;
    rc = ELITEKV_OK;
  } while (0);

  if (rc != ELITEKV_OK) {
    elitekv_layer_destroy(L);
    return rc;
  }
  *out = L;
  return ELITEKV_OK;
}

extern "C" int elitekv_layer_destroy(elitekv_layer* L) {
  if (!L) return ELITEKV_ERR_INVALID_ARG;
  cudaFree(L->d_status);
  cudaFree(L->d_qdims);
  cudaFree(L->d_idx);
  cudaFree(L->d_cs_owned);
  cudaFree(L->d_WukT);
  cudaFree(L->d_Wuv);
  cudaFree(L->d_WcatT);
  if (L->side) cudaStreamDestroy(L->side);
  if (L->ev_fork) cudaEventDestroy(L->ev_fork);
  if (L->ev_join) cudaEventDestroy(L->ev_join);
  if (L->prof) {
    for (int i = 0; i < 2 * kProfileSlots; ++i)
      if (L->prof->ev[i]) cudaEventDestroy(L->prof->ev[i]);
    free(L->prof);
  }
  free(L->last_detail);
  free(L);
  return ELITEKV_OK;
}

extern "C" int elitekv_check_status(const elitekv_layer* L, elitekv_stream_t stream) {
  if (!L) return ELITEKV_ERR_INVALID_ARG;
  int32_t h[4] = {0, 0, 0, 0};
  cudaStream_t st = (cudaStream_t)stream;
  EKV_CUDA_OK(cudaMemcpyAsync(h, L->d_status, sizeof(h), cudaMemcpyDeviceToHost, st));
  EKV_CUDA_OK(cudaMemsetAsync(L->d_status, 0, sizeof(h), st));
  EKV_CUDA_OK(cudaStreamSynchronize(st));
  L->last_detail[0] = h[1];
  L->last_detail[1] = h[2];
  L->last_detail[2] = h[3];
  return h[0];
}

extern "C" int elitekv_last_status_detail(const elitekv_layer* L, int32_t detail[3]) {
  if (!L || !detail) return ELITEKV_ERR_INVALID_ARG;
  for (int i = 0; i < 3; ++i) detail[i] = L->last_detail[i];
  return ELITEKV_OK;
}

extern "C" const char* elitekv_strerror(int status) {
  switch (status) {
    case ELITEKV_OK: return "ok";
    case ELITEKV_ERR_INVALID_ARG: return "invalid argument";
    case ELITEKV_ERR_UNSUPPORTED_SHAPE: return "shape not supported by the selected kernel";
    case ELITEKV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small or misaligned";
    case ELITEKV_ERR_CUDA: return "CUDA runtime error";
    case ELITEKV_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case ELITEKV_ERR_BAD_PAGE: return "page id outside the pool";
    case ELITEKV_ERR_BAD_POSITION: return "position or sequence outside the cache";
    case ELITEKV_ERR_STATIC_SCRATCH_EXCEEDED:
      return "scratch need exceeds the built-in array of elitekv_decode_static";
    default: return "unknown status";
  }
}

extern "C" int elitekv_profile_enable(elitekv_layer* L, int32_t on) {
  if (!L) return ELITEKV_ERR_INVALID_ARG;
  if (on && !L->prof) {
    EkvProfile* p = (EkvProfile*)calloc(1, sizeof(EkvProfile));
    if (!p) return ELITEKV_ERR_CUDA;
    for (int i = 0; i < 2 * kProfileSlots; ++i)
      if (cudaEventCreate(&p->ev[i]) != cudaSuccess) {
        for (int j = 0; j < i; ++j) cudaEventDestroy(p->ev[j]);
        free(p);
        return ELITEKV_ERR_CUDA;
      }
    L->prof = p;
  }
  if (L->prof) {
    L->prof->enabled = on ? 1 : 0;
    L->prof->count = 0;
  }
  return ELITEKV_OK;
}

extern "C" int elitekv_profile_collect(elitekv_layer* L, float* total_ms, int32_t* launches) {
  if (!L || !total_ms || !launches) return ELITEKV_ERR_INVALID_ARG;
  *total_ms = 0.f;
  *launches = 0;
  if (!L->prof) return ELITEKV_OK;
  EkvProfile* p = L->prof;
  for (int i = 0; i < p->count; ++i) {
    float ms = 0.f;
    EKV_CUDA_OK(cudaEventSynchronize(p->ev[2 * i + 1]));
    EKV_CUDA_OK(cudaEventElapsedTime(&ms, p->ev[2 * i], p->ev[2 * i + 1]));
    *total_ms += ms;
  }
  *launches = p->count;
  p->count = 0;
  return ELITEKV_OK;
}

int ekv_make_view(const elitekv_cache* c, CacheView* v) {
  if (!c || !c->rope || !c->latent || c->n_seqs <= 0) return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)c->rope & 15) || ((uintptr_t)c->latent & 15)) return ELITEKV_ERR_INVALID_ARG;
  memset(v, 0, sizeof(*v));
  v->n_seqs = c->n_seqs;
  if (c->page_table) {
    int ps = c->page_size;
    if (ps <= 0 || (ps & (ps - 1)) || c->max_pages_per_seq <= 0 || c->num_pages <= 0)
      return ELITEKV_ERR_INVALID_ARG;
    int sh = 0;
    while ((1 << sh) < ps) ++sh;
    v->page_table = c->page_table;
    v->page_shift = sh;
    v->page_mask = ps - 1;
    v->max_pages_per_seq = c->max_pages_per_seq;
    v->num_pages = c->num_pages;
    v->max_ctx = (long long)c->max_pages_per_seq * ps;
  } else {
    if (c->max_ctx <= 0) return ELITEKV_ERR_INVALID_ARG;
    v->max_ctx = c->max_ctx;
  }
  return ELITEKV_OK;
}
