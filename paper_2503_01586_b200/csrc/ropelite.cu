// RoPElite search scoring (Algorithm 1, Section 3.1), all heads of all layers in one launch.
//
// For one head the search compares the attention scores s = q K^T (pre-softmax, Section 2.1) with
// RoPE on every chunk against the scores with RoPE on the elite chunks e plus one candidate j
// only, over every decoding step of a calibration sequence (query position m, key position
// n <= m, token t at position t), and picks the candidate with the smallest L1 distance.
//
// Chunk i contributes to the score of the pair (m, n)
//     rotated:  a_i cos(phi) - b_i sin(phi),   plain:  a_i,
//     a_i = q_{m,2i} k_{n,2i} + q_{m,2i+1} k_{n,2i+1},  b_i = q_{m,2i+1} k_{n,2i} - q_{m,2i} k_{n,2i+1},
//     phi = (m - n) theta_i                                                   (Eq. 1a / 1b)
// so with D_i = a_i (cos(phi) - 1) - b_i sin(phi) the difference between the fully rotated score
// and the trial score is  R - D_j,  R = sum of D_i over the chunks not in e.  One pass over the
// pairs therefore yields the distances of ALL candidates of a round:  dist[j] = sum |R - D_j|.
// This is FP32 arithmetic on CUDA cores (there is no contraction deeper than 2 here).
//
// distance kernel: grid (row tiles of 16 query positions, heads), 128 threads.  Warp w owns query
// rows m0 + 4 w .. m0 + 4 w + 3, its lanes own keys; key tiles of 64 are staged in shared memory as fp32 pairs
// [chunk][key] together with the slice of the (cos - 1, sin) table the tile's relative positions
// need, [chunk][m - n].  A thread keeps the 64 D_i of its pair and 64 running sums in registers.
// Block results go to a [head][row tile][chunk] array; the select kernel adds them in a fixed
// order (the result does not depend on scheduling), masks the chunks already chosen and takes
// the first minimum.
#include "common.cuh"

namespace {

constexpr int kRlRows = 16;       // query rows per block (four per warp)
constexpr int kRlWarps = 4;
constexpr int kRlRowsPerWarp = kRlRows / kRlWarps;
constexpr int kRlKeys = 64;       // keys per stage
constexpr int kRlThreads = 128;
constexpr int kRlSpan = kRlKeys + kRlRows - 1;     // relative positions a stage can meet
constexpr int kRlSpanPad = kRlSpan + 1;

// (cos(d theta_i) - 1, sin(d theta_i)) for d in [0, n), laid out [chunk][d]; double precision,
// rounded once
__global__ void ropelite_table_kernel(float2* __restrict__ tab, int n, int half, int d_h, double base) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (long long)n * half) return;
  const int i = (int)(e / n), d = (int)(e % n);
  const double theta = pow(base, -2.0 * (double)i / (double)d_h);
  const double ang = (double)d * theta;
  tab[e] = make_float2((float)(cos(ang) - 1.0), (float)sin(ang));
}

template <int HALF>
__global__ void __launch_bounds__(kRlThreads)
ropelite_distance_kernel(const bf16* __restrict__ Q, const bf16* __restrict__ K, int n,
                         const float2* __restrict__ tab, const unsigned long long* __restrict__ masks,
                         float* __restrict__ partial /* [heads][row tiles][HALF] */) {
  constexpr int d_h = 2 * HALF;
  extern __shared__ __align__(16) float2 smem_rl[];
  // keys stay packed as they come (a bf16 pair per chunk: one 4-byte load per pair and chunk, widened in registers)
  float2 (*s_t)[kRlSpanPad] = (float2 (*)[kRlSpanPad])smem_rl;                        // [HALF][relative position]
  float2 (*s_q)[HALF] = (float2 (*)[HALF])(smem_rl + HALF * kRlSpanPad);             // [rows][HALF]
  float (*s_red)[HALF] = (float (*)[HALF])(smem_rl + HALF * (kRlSpanPad + kRlRows)); // [warps][HALF]
  uint32_t (*s_k)[kRlKeys] = (uint32_t (*)[kRlKeys])(&s_red[kRlWarps][0]);           // [HALF][keys]
  const int n_tiles = gridDim.x;
  const int mt = n_tiles - 1 - (int)blockIdx.x;          // long rows first
  const int head = blockIdx.y;
  const int m0 = mt * kRlRows;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const unsigned long long mask = masks ? masks[head] : 0ull;
  const bf16* Qh = Q + (size_t)head * n * d_h;
  const bf16* Kh = K + (size_t)head * n * d_h;

  for (int e = threadIdx.x; e < kRlRows * HALF; e += kRlThreads) {
    const int rr = e / HALF, i = e % HALF;
    float2 v = make_float2(0.f, 0.f);
    if (m0 + rr < n) v = __bfloat1622float2(*(const bf162*)(Qh + (size_t)(m0 + rr) * d_h + 2 * i));
    s_q[rr][i] = v;
  }
  float acc[HALF];
#pragma unroll
  for (int j = 0; j < HALF; ++j) acc[j] = 0.f;

  const int m_last = min(m0 + kRlRows - 1, n - 1);
  for (int n0 = 0; n0 <= m_last; n0 += kRlKeys) {
    __syncthreads();
    // keys of the stage: consecutive threads take consecutive keys (conflict-free stores)
    for (int e = threadIdx.x; e < kRlKeys * (HALF / 4); e += kRlThreads) {
      const int nn = e % kRlKeys, g4 = e / kRlKeys;         // 4 chunks = 8 elements = 16 bytes
      uint4 raw = make_uint4(0, 0, 0, 0);
      if (n0 + nn < n) raw = *(const uint4*)(Kh + (size_t)(n0 + nn) * d_h + g4 * 8);
      s_k[g4 * 4 + 0][nn] = raw.x; s_k[g4 * 4 + 1][nn] = raw.y;
      s_k[g4 * 4 + 2][nn] = raw.z; s_k[g4 * 4 + 3][nn] = raw.w;
    }
    // table slice: relative positions d_min .. d_min + span - 1 (negative ones belong to masked pairs)
    const int d_min = m0 - n0 - (kRlKeys - 1);
    for (int e = threadIdx.x; e < HALF * kRlSpan; e += kRlThreads) {
      const int i = e / kRlSpan, dd = e % kRlSpan;
      const int d = d_min + dd;
      s_t[i][dd] = (d >= 0 && d < n) ? tab[(size_t)i * n + d] : make_float2(0.f, 0.f);
    }
    __syncthreads();
#pragma unroll 1
    for (int e = 0; e < kRlRowsPerWarp * (kRlKeys / 32); ++e) {
      const int rr = warp * kRlRowsPerWarp + e / (kRlKeys / 32);     // row inside the block
      const int m = m0 + rr;
      const int nn = lane + 32 * (e % (kRlKeys / 32));
      const int key = n0 + nn;
      if (!(key <= m && m < n)) continue;                  // causal pairs only
      const int dd = rr + (kRlKeys - 1) - nn;              // (m - key) - d_min
      float d[HALF];
      float R = 0.f;
#pragma unroll
      for (int i = 0; i < HALF; ++i) {
        const float2 q = s_q[rr][i], t = s_t[i][dd];
        const uint32_t kp = s_k[i][nn];
        const float2 k = make_float2(__uint_as_float(kp << 16), __uint_as_float(kp & 0xffff0000u));   // bf16 pair -> fp32
        const float a = fmaf(q.x, k.x, q.y * k.y);
        const float b = fmaf(q.y, k.x, -(q.x * k.y));
        d[i] = fmaf(a, t.x, -(b * t.y));
        if (!((mask >> i) & 1ull)) R += d[i];
      }
#pragma unroll
      for (int j = 0; j < HALF; ++j) acc[j] += fabsf(R - d[j]);
    }
  }
  // block result: lanes, then warps, in a fixed order
#pragma unroll
  for (int j = 0; j < HALF; ++j) {
    const float v = warp_sum(acc[j]);
    if (lane == 0) s_red[warp][j] = v;
  }
  __syncthreads();
  for (int j = threadIdx.x; j < HALF; j += kRlThreads) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kRlWarps; ++w) v += s_red[w][j];
    partial[((size_t)head * n_tiles + mt) * HALF + j] = v;
  }
}

// One block per head: adds the row tiles' results in order, writes the round's distances
// (+inf for chunks already chosen) and, when `elite_idx` is given, appends the first minimum to
// the head's list and to its mask.
__global__ void ropelite_select_kernel(const float* __restrict__ partial, int n_tiles, int half,
                                       unsigned long long* __restrict__ masks, float* __restrict__ dist_out,
                                       int32_t* __restrict__ elite_idx, int r, int round) {
  __shared__ float s_d[64];
  const int head = blockIdx.x, j = threadIdx.x;
  const unsigned long long mask = masks ? masks[head] : 0ull;
  float v = INFINITY;
  if (j < half && !((mask >> j) & 1ull)) {
    v = 0.f;
    for (int t = 0; t < n_tiles; ++t) v += partial[((size_t)head * n_tiles + t) * half + j];
  }
  if (j < half && dist_out) dist_out[(size_t)head * half + j] = v;
  s_d[j] = j < half ? v : INFINITY;
  __syncthreads();
  if (j == 0 && elite_idx) {
    int best = 0;
    for (int c = 1; c < half; ++c)
      if (s_d[c] < s_d[best]) best = c;
    elite_idx[(size_t)head * r + round] = best;
    masks[head] = mask | (1ull << best);
  }
}

struct RlCarve {
  size_t off_tab, off_partial, off_masks, total;
};
inline size_t rl_align(size_t x) { return (x + 255) & ~(size_t)255; }
RlCarve rl_carve(int heads, int n, int half) {
  RlCarve c;
  size_t o = 0;
  const int n_tiles = (n + kRlRows - 1) / kRlRows;
  c.off_tab = o;     o = rl_align(o + sizeof(float2) * (size_t)half * n);
  c.off_partial = o; o = rl_align(o + sizeof(float) * (size_t)heads * n_tiles * half);
  c.off_masks = o;   o = rl_align(o + sizeof(unsigned long long) * (size_t)heads);
  c.total = o;
  return c;
}

int rl_check(int heads, int n, int d_h) {
  if (heads <= 0 || n <= 0) return ELITEKV_ERR_INVALID_ARG;
  if (d_h != 64 && d_h != 128) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  if ((long long)n > (1 << 20) || heads > 65535) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  return ELITEKV_OK;
}

int rl_launch_distance(const void* Q, const void* K, int heads, int n, int d_h, const float2* tab,
                       const unsigned long long* masks, float* partial, cudaStream_t st) {
  dim3 grid((unsigned)((n + kRlRows - 1) / kRlRows), (unsigned)heads);
  const int half = d_h / 2;
  const int smem = half * (kRlSpanPad + kRlRows) * (int)sizeof(float2) + kRlWarps * half * (int)sizeof(float) +
                   half * kRlKeys * (int)sizeof(uint32_t);
  if (d_h == 128) {
    EKV_CUDA_OK(cudaFuncSetAttribute(ropelite_distance_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    ropelite_distance_kernel<64><<<grid, kRlThreads, smem, st>>>((const bf16*)Q, (const bf16*)K, n, tab, masks, partial);
  } else {
    EKV_CUDA_OK(cudaFuncSetAttribute(ropelite_distance_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    ropelite_distance_kernel<32><<<grid, kRlThreads, smem, st>>>((const bf16*)Q, (const bf16*)K, n, tab, masks, partial);
  }
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

int rl_launch_table(float2* tab, int n, int d_h, float base, cudaStream_t st) {
  const long long total = (long long)n * (d_h / 2);
  ropelite_table_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(tab, n, d_h / 2, d_h, (double)base);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

}  // namespace

extern "C" int elitekv_ropelite_workspace_size(int32_t n_heads, int32_t n, int32_t d_h, size_t* bytes) {
  if (!bytes) return ELITEKV_ERR_INVALID_ARG;
  const int rc = rl_check(n_heads, n, d_h);
  if (rc != ELITEKV_OK) return rc;
  *bytes = rl_carve(n_heads, n, d_h / 2).total;
  return ELITEKV_OK;
}

extern "C" int elitekv_ropelite_distances(const void* Q, const void* K, int32_t n_heads, int32_t n, int32_t d_h,
                                          float rope_base, const uint64_t* elite_mask, void* workspace,
                                          size_t workspace_bytes, float* dist, elitekv_stream_t stream) {
  if (!Q || !K || !workspace || !dist) return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)Q & 15) || ((uintptr_t)K & 15)) return ELITEKV_ERR_INVALID_ARG;
  int rc = rl_check(n_heads, n, d_h);
  if (rc != ELITEKV_OK) return rc;
  const int half = d_h / 2;
  const RlCarve c = rl_carve(n_heads, n, half);
  if (((uintptr_t)workspace & 255) || workspace_bytes < c.total) return ELITEKV_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* base = (unsigned char*)workspace;
  float2* tab = (float2*)(base + c.off_tab);
  float* partial = (float*)(base + c.off_partial);
  cudaStream_t st = (cudaStream_t)stream;
  rc = rl_launch_table(tab, n, d_h, rope_base, st);
  if (rc != ELITEKV_OK) return rc;
  rc = rl_launch_distance(Q, K, n_heads, n, d_h, tab, (const unsigned long long*)elite_mask, partial, st);
  if (rc != ELITEKV_OK) return rc;
  ropelite_select_kernel<<<n_heads, 64, 0, st>>>(partial, (n + kRlRows - 1) / kRlRows, half,
                                                 (unsigned long long*)elite_mask, dist, nullptr, 0, 0);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

extern "C" int elitekv_ropelite_search(const void* Q, const void* K, int32_t n_heads, int32_t n, int32_t d_h,
                                       float rope_base, int32_t r, void* workspace, size_t workspace_bytes,
                                       int32_t* elite_idx, float* dist_trace, elitekv_stream_t stream) {
  if (!Q || !K || !workspace || !elite_idx) return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)Q & 15) || ((uintptr_t)K & 15)) return ELITEKV_ERR_INVALID_ARG;
  int rc = rl_check(n_heads, n, d_h);
  if (rc != ELITEKV_OK) return rc;
  const int half = d_h / 2;
  if (r < 0 || r > half) return ELITEKV_ERR_INVALID_ARG;
  const RlCarve c = rl_carve(n_heads, n, half);
  if (((uintptr_t)workspace & 255) || workspace_bytes < c.total) return ELITEKV_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* base = (unsigned char*)workspace;
  float2* tab = (float2*)(base + c.off_tab);
  float* partial = (float*)(base + c.off_partial);
  unsigned long long* masks = (unsigned long long*)(base + c.off_masks);
  cudaStream_t st = (cudaStream_t)stream;
  rc = rl_launch_table(tab, n, d_h, rope_base, st);
  if (rc != ELITEKV_OK) return rc;
  EKV_CUDA_OK(cudaMemsetAsync(masks, 0, sizeof(unsigned long long) * (size_t)n_heads, st));
  const int n_tiles = (n + kRlRows - 1) / kRlRows;
  for (int round = 0; round < r; ++round) {
    rc = rl_launch_distance(Q, K, n_heads, n, d_h, tab, masks, partial, st);
    if (rc != ELITEKV_OK) return rc;
    ropelite_select_kernel<<<n_heads, 64, 0, st>>>(partial, n_tiles, half, masks,
                                                   dist_trace ? dist_trace + (size_t)round * n_heads * half : nullptr,
                                                   elite_idx, r, round);
    EKV_CUDA_OK(cudaGetLastError());
  }
  return ELITEKV_OK;
}
