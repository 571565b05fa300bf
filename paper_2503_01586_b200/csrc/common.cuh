// Shared declarations of the EliteKV CUDA library (sm_100a).  Host-side layer object, status
// word helpers and small device utilities.  Nothing here is used by the CPU oracle.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/elitekv.h"

typedef __nv_bfloat16 bf16;
typedef __nv_bfloat162 bf162;

// The work plan cuts sequences in units of this many tokens (also the page size the
// tensor-core kernel expects).
#define ELITEKV_TILE_TOKENS 64

struct elitekv_layer {
  int n_h, d_h, r, d_c, dn;        // dn = d_h - 2r (un-rotated key dims per head); d_c = width of a latent row
  int kw, voff, vw;                // latent columns the scores read: [0, kw); the outputs: [voff, voff + vw).
                                   // Joint latent: kw = vw = d_c, voff = 0.  Separated: kw = d_ck, voff = d_ck, vw = d_cv.
  float rope_base;
  float scale;                     // softmax scale actually used
  int pair_mode;
  int max_pos;
  int decode_kernel;
  int device;
  int sm_count;
  int smem_optin;                  // max dynamic shared memory per block
  int32_t* d_idx;                  // [n_h][r] elite chunk ids
  int32_t* d_qdims;                // [n_h][d_h]: 2r dims of the elite chunks in cache order,
                                   // then the dn remaining dims ascending
  const float2* d_cs;              // [max_pos][d_h/2] (cos, sin)
  float2* d_cs_owned;              // same pointer when the library built the table
  bf16* d_WukT;                    // [n_h][dn][kw]: W_uk regrouped per head, latent axis contiguous
  bf16* d_Wuv;                     // [vw][n_h*d_h] private copy
  int32_t* d_status;               // [4] device status word: code, detail0, detail1, count
  struct EkvProfile* prof;         // optional event pairs around the split-K kernel
  int32_t* last_detail;            // host [3]: detail words + count read by the last check_status
  int d;                           // model width (0: no projection weights)
  bf16* d_WcatT;                   // [n_h*2r + d_c][d]: [W^k_e | A^kv] transposed (rows = output columns)
  cudaStream_t side;               // second stream of elitekv_decode_step (append + plan beside the absorb)
  cudaEvent_t ev_fork, ev_join;    // its fork from / join into the caller's stream
};

constexpr int kProfileSlots = 512;
struct EkvProfile {
  int enabled;
  int count;
  cudaEvent_t ev[2 * kProfileSlots];
};

#define EKV_CUDA_OK(expr)                                   \
  do {                                                      \
    cudaError_t _e = (expr);                                \
    if (_e != cudaSuccess) return ELITEKV_ERR_CUDA;         \
  } while (0)

// Records the first device-side fault; later ones only bump the counter.
__device__ __forceinline__ void ekv_record(int32_t* status, int code, int d0, int d1) {
  if (atomicCAS(&status[0], 0, code) == 0) {
    status[1] = d0;
    status[2] = d1;
  }
  atomicAdd(&status[3], 1);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gmem_src) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

// Programmatic dependent launch: the kernels of one decode step are launched with the
// programmatic-serialisation attribute, so that the next kernel's blocks are scheduled (and run
// whatever precedes their ekv_pdl_wait) while the previous kernel drains.  ekv_pdl_wait returns
// once every kernel earlier in the stream has completed and its writes are visible; a kernel
// launched without the attribute, or after one that never calls ekv_pdl_trigger, behaves as usual.
__device__ __forceinline__ void ekv_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void ekv_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t ekv_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// Where a (sequence, position) lives in the cache planes.
struct CacheView {
  const int32_t* page_table;
  int page_shift, page_mask, max_pages_per_seq;
  long long num_pages, max_ctx;
  int n_seqs;
};

// Row index (in tokens) of (seq, pos), or -1 with (code, detail) left for the caller to record.
__device__ __forceinline__ long long ekv_token_row(const CacheView& cv, int seq, int pos,
                                                   int* code, int* detail) {
  *code = ELITEKV_ERR_BAD_POSITION;
  *detail = pos;
  if (seq < 0 || seq >= cv.n_seqs || pos < 0) return -1;
  if (cv.page_table == nullptr) {
    if (pos >= cv.max_ctx) return -1;
    return (long long)seq * cv.max_ctx + pos;
  }
  int pi = pos >> cv.page_shift;
  if (pi >= cv.max_pages_per_seq) return -1;
  int page = cv.page_table[(long long)seq * cv.max_pages_per_seq + pi];
  if (page < 0 || page >= cv.num_pages) {
    *code = ELITEKV_ERR_BAD_PAGE;
    *detail = page;
    return -1;
  }
  return ((long long)page << cv.page_shift) + (pos & cv.page_mask);
}

// Host-side helpers shared by the entry points.
int ekv_make_view(const elitekv_cache* cache, CacheView* out);

// Kernel launchers (one per .cu file).
int ekv_launch_append(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                      const void* k_e, const void* c, const int32_t* seq_id, const int32_t* pos,
                      long long T, cudaStream_t st);
int ekv_launch_project_append(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                              const void* x, const int32_t* seq_id, const int32_t* pos, long long T,
                              cudaStream_t st);
int ekv_launch_absorb(const elitekv_layer* L, const void* q, const int32_t* q_pos, int B,
                      void* q_rope, void* q_abs, cudaStream_t st);
// max_len: tokens one sequence can hold in the cache; longer (or negative) lengths are recorded
// in `status` (may be null) as BAD_POSITION and clamped.
int ekv_launch_plan(const int32_t* seq_lens, int B, int tile_tokens, int max_items, int32_t* items,
                    int32_t* seq_first_item, int32_t* zero_ints, int n_zero, long long max_len,
                    int32_t* status, cudaStream_t st);

int ekv_launch_plan_balanced(const int32_t* seq_lens, int B, int tile_tokens, int n_workers,
                             int max_items, int32_t* items, int32_t* seq_first_item,
                             int32_t* worker_first, int32_t* zero_ints, int n_zero, long long max_len,
                             int32_t* status, int overhead_tiles, cudaStream_t st);

struct DecodeScratch {
  int max_items;          // capacity of the plan
  int32_t* items;         // [max_items][4]
  int32_t* seq_first;     // [B+1]
  float* part_acc;        // [max_items][n_h][vw]
  float* part_ml;         // [max_items][n_h][2]  (running max in log2 units, running sum)
  float* slice_out;       // combine: per latent slice partial outputs [vw/128][B][n_h][128]
  int32_t* counters;      // combine: arrival counters, zeroed by the plan kernel
  int n_counters;
  int32_t* worker_first;  // balanced plan: [n_workers+1] first item of each worker
  int n_workers;
  int rows;               // query rows per sequence (1: decode).  With rows > 1 every "n_h" in the shapes
                          // above reads rows * n_h: row i, head h is entry i * n_h + h
  const int32_t* seq_lens;   // rows > 1: the lengths, for the causal limit of each row
};

int ekv_combine_fast_ok(const elitekv_layer* L);
size_t ekv_combine_scratch_bytes(const elitekv_layer* L, int B);
int ekv_combine_counters(const elitekv_layer* L, int B);

int ekv_generic_supported(const elitekv_layer* L);
int ekv_generic_max_items(const elitekv_layer* L, int B);
int ekv_launch_decode_generic(const elitekv_layer* L, const elitekv_cache* cache,
                              const CacheView& cv, const void* q_rope, const void* q_abs, int B,
                              const DecodeScratch& ws, cudaStream_t st);
int ekv_tc_supported(const elitekv_layer* L, const elitekv_cache* cache);   // cache may be null
int ekv_tc_max_items(const elitekv_layer* L, int B, int rows);
int ekv_tc_workers(const elitekv_layer* L, int rows);
int ekv_launch_decode_tc(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                         const void* q_rope, const void* q_abs, int B, const DecodeScratch& ws,
                         cudaStream_t st);
int ekv_rt_supported(const elitekv_layer* L, const elitekv_cache* cache);   // cache may be null
int ekv_rt_workers(const elitekv_layer* L);
int ekv_rt_max_items(const elitekv_layer* L, int B);
int ekv_launch_decode_rt(const elitekv_layer* L, const elitekv_cache* cache, const CacheView& cv,
                         const void* q_rope, const void* q_abs, int B, const DecodeScratch& ws,
                         cudaStream_t st);
int ekv_launch_combine(const elitekv_layer* L, int B, const DecodeScratch& ws, void* out,
                       cudaStream_t st);
