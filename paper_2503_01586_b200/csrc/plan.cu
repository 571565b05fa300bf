// Work plan for the split-K decode kernels: cuts every sequence's token range into pieces of
// near-equal size so that ragged batches keep all SMs busy.  Integer arithmetic only, on
// device-resident lengths, so a decode step never synchronises with the host.  (The paper
// leaves scheduling open; this is the library's load balancer.)
//
// With tiles_b = ceil(len_b / tile), total = sum tiles_b and budget = max_items - B:
//   target   = max(1, ceil(total / budget))            tiles per item
//   pieces_b = ceil(tiles_b / target)                  (sum <= budget + B = max_items)
//   piece j of sequence b covers tiles [tiles_b*j/pieces_b, tiles_b*(j+1)/pieces_b)
#include "common.cuh"

namespace {

constexpr int kPlanThreads = 256;
constexpr int kPlanStage = 4096;       // items whose worker ids are staged in shared memory

// exclusive scan over the block (warp shuffles + one shared array of warp totals)
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += x;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  int before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kPlanThreads / 32; ++w) {
    const int t = warp_tot[w];
    if (w < warp) before += t;
    all += t;
  }
  __syncthreads();
  *total = all;
  return before + incl - v;
}

// Length of sequence b as the kernels may use it: a length beyond what the cache can hold per
// sequence (or a negative one) is recorded as BAD_POSITION and clamped, so that no kernel
// downstream walks into another sequence's rows.  Only `report` threads record.
__device__ __forceinline__ int checked_len(const int32_t* seq_lens, int b, long long max_len, int32_t* status,
                                           bool report) {
  int n = seq_lens[b];
  if (n < 0 || n > max_len) {
    if (report && status) ekv_record(status, ELITEKV_ERR_BAD_POSITION, b, n);
    n = n < 0 ? 0 : (int)max_len;
  }
  return n;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t* __restrict__ seq_lens, int B, int tile, int max_items,
            int32_t* __restrict__ items, int32_t* __restrict__ seq_first,
            int32_t* __restrict__ zero_ints, int n_zero, long long max_len, int32_t* status) {
  __shared__ int warp_tot[kPlanThreads / 32];
  __shared__ long long s_total;
  const int t = threadIdx.x;
  for (int i = t; i < n_zero; i += blockDim.x) zero_ints[i] = 0;
  if (t == 0) s_total = 0;
  __syncthreads();
  long long local = 0;
  for (int b = t; b < B; b += blockDim.x) {
    int n = checked_len(seq_lens, b, max_len, status, true);
    local += n > 0 ? (n + tile - 1) / tile : 0;
  }
  if (local) atomicAdd((unsigned long long*)&s_total, (unsigned long long)local);
  __syncthreads();
  const long long total = s_total;
  const long long budget = max_items - B > 0 ? max_items - B : 1;
  long long target = (total + budget - 1) / budget;
  if (target < 1) target = 1;

  int carry = 0;
  for (int b0 = 0; b0 < B; b0 += blockDim.x) {
    const int b = b0 + t;
    int n = 0, tiles = 0, pieces = 0;
    if (b < B) {
      n = checked_len(seq_lens, b, max_len, status, false);
      tiles = n > 0 ? (n + tile - 1) / tile : 0;
      pieces = (int)((tiles + target - 1) / target);
    }
    int chunk_total;
    const int first = carry + block_exclusive_scan(pieces, warp_tot, &chunk_total);
    if (b < B) {
      seq_first[b] = first;
      for (int j = 0; j < pieces; ++j) {
        const int ta = (int)((long long)tiles * j / pieces);
        const int tb = (int)((long long)tiles * (j + 1) / pieces);
        const int tok0 = ta * tile;
        const int tok1 = min(tb * tile, n);
        const int it = first + j;
        if (it < max_items) *(int4*)(items + 4 * it) = make_int4(b, tok0, tok1 - tok0, 0);
      }
    }
    carry += chunk_total;
  }
  if (t == 0) seq_first[B] = carry;
  for (int it = carry + t; it < max_items; it += blockDim.x) *(int4*)(items + 4 * it) = make_int4(-1, 0, 0, 0);
}

// Balanced plan for kernels whose blocks walk several items: worker w of `n_workers` owns the
// global tile range [w*total/n, (w+1)*total/n), n = min(n_workers, total) (integer division: the
// ranges differ by at most one tile and none is empty); an item is the
// intersection of one worker's range with one sequence.  Items come out in global order, so they
// are grouped by sequence (seq_first) and by worker (worker_first).  items[i] = (sequence, first
// token, token count, worker).
// Starting an item costs a worker about as much as `overhead` tiles (new queries, a partial
// result to write out), and a worker whose range contains the start of a sequence has one item
// more than the others.  The tile list therefore carries `overhead` empty tiles in front of every
// sequence: they take room in a worker's quota and hold no tokens.
__global__ void __launch_bounds__(kPlanThreads)
plan_balanced_kernel(const int32_t* __restrict__ seq_lens, int B, int tile, int n_workers,
                     int max_items, int32_t* __restrict__ items, int32_t* __restrict__ seq_first,
                     int32_t* __restrict__ worker_first, int32_t* __restrict__ zero_ints, int n_zero,
                     long long max_len, int32_t* status, int overhead) {
  __shared__ int warp_tot[kPlanThreads / 32];
  __shared__ long long s_total;
  __shared__ short s_wk[kPlanStage];       // worker of each item (n_workers < 32768)
  const int t = threadIdx.x;
  ekv_pdl_wait();         // earlier kernels may still read the arrays written here
  ekv_pdl_trigger();
  for (int i = t; i < n_zero; i += blockDim.x) zero_ints[i] = 0;
  if (t == 0) s_total = 0;
  __syncthreads();
  long long local = 0;
  for (int b = t; b < B; b += blockDim.x) {
    int n = checked_len(seq_lens, b, max_len, status, true);
    local += n > 0 ? (n + tile - 1) / tile + overhead : 0;
  }
  if (local) atomicAdd((unsigned long long*)&s_total, (unsigned long long)local);
  __syncthreads();
  const long long total = s_total > 0 ? s_total : 1;
  // first position of worker w's range, and the worker that owns position g
  // (with fewer positions than workers only the first `total` workers get a range, of one each)
  const long long nw = total < n_workers ? total : n_workers;
  auto bound = [&](long long w) -> long long { return w * total / nw; };
  auto owner = [&](long long g) -> int { return (int)(((g + 1) * nw - 1) / total); };
  int carry_tiles = 0, carry_items = 0;
  {
    for (int b0 = 0; b0 < B; b0 += blockDim.x) {
      const int b = b0 + t;
      int n = 0, tiles = 0;
      if (b < B) {
        n = checked_len(seq_lens, b, max_len, status, false);
        tiles = n > 0 ? (n + tile - 1) / tile + overhead : 0;     // with the empty tiles in front
      }
      int chunk_tiles;
      const int g0 = carry_tiles + block_exclusive_scan(tiles, warp_tot, &chunk_tiles);
      int pieces = 0, w0 = 0;
      if (tiles > 0) {
        w0 = owner(g0 + overhead);                                // workers that hold real tiles
        const int w1 = owner(g0 + tiles - 1);
        pieces = w1 - w0 + 1;
      }
      int chunk_items;
      const int first = carry_items + block_exclusive_scan(pieces, warp_tot, &chunk_items);
      if (b < B) {
        seq_first[b] = first;
        for (int j = 0; j < pieces; ++j) {
          const long long ga = max((long long)g0 + overhead, bound(w0 + j));
          const long long gb = min((long long)g0 + tiles, bound(w0 + j + 1));
          const int tok0 = (int)(ga - g0 - overhead) * tile;
          const int tok1 = min((int)(gb - g0 - overhead) * tile, n);
          const int it = first + j;
          if (it < max_items) *(int4*)(items + 4 * it) = make_int4(b, tok0, tok1 - tok0, w0 + j);
          if (it < kPlanStage) s_wk[it] = (short)(w0 + j);
        }
      }
      carry_tiles += chunk_tiles;
      carry_items += chunk_items;
    }
  }
  if (t == 0) seq_first[B] = carry_items;
  for (int it = carry_items + t; it < max_items; it += blockDim.x) *(int4*)(items + 4 * it) = make_int4(-1, 0, 0, 0);
  // worker_first[w] = number of items of workers below w (items are ordered by worker; a worker
  // without items gets an empty range).  The worker ids of up to kPlanStage items are kept in
  // shared memory while they are written, so that this is a binary search per worker instead of
  // a second trip to global memory.
  __syncthreads();
  const int n_items = min(carry_items, max_items);
  if (n_items <= kPlanStage) {
    for (int w = t; w <= n_workers; w += blockDim.x) {
      int lo = 0, hi = n_items;              // first item whose worker is >= w
      while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s_wk[mid] < w) lo = mid + 1; else hi = mid;
      }
      worker_first[w] = lo;
    }
  } else {
    for (int w = t; w <= n_workers; w += blockDim.x) worker_first[w] = n_items;
    __syncthreads();
    for (int it = t; it < n_items; it += blockDim.x) {
      const int wk = items[4 * it + 3];
      if (it == 0 || items[4 * (it - 1) + 3] != wk) worker_first[wk] = it;
    }
    __syncthreads();
    if (t == 0)       // unset entries still hold the item count; an entry may not exceed its successor
      for (int w = n_workers - 1; w >= 0; --w)
        if (worker_first[w] > worker_first[w + 1]) worker_first[w] = worker_first[w + 1];
  }
}

}  // namespace

int ekv_launch_plan_balanced(const int32_t* seq_lens, int B, int tile_tokens, int n_workers,
                             int max_items, int32_t* items, int32_t* seq_first_item,
                             int32_t* worker_first, int32_t* zero_ints, int n_zero, long long max_len,
                             int32_t* status, int overhead_tiles, cudaStream_t st) {
  EKV_CUDA_OK(ekv_launch_pdl(plan_balanced_kernel, dim3(1), dim3(kPlanThreads), 0, st, seq_lens, B, tile_tokens,
                             n_workers, max_items, items, seq_first_item, worker_first, zero_ints, n_zero,
                             max_len, status, overhead_tiles));
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

int ekv_launch_plan(const int32_t* seq_lens, int B, int tile_tokens, int max_items, int32_t* items,
                    int32_t* seq_first_item, int32_t* zero_ints, int n_zero, long long max_len,
                    int32_t* status, cudaStream_t st) {
  plan_kernel<<<1, kPlanThreads, 0, st>>>(seq_lens, B, tile_tokens, max_items, items, seq_first_item,
                                          zero_ints, n_zero, max_len, status);
  EKV_CUDA_OK(cudaGetLastError());
  return ELITEKV_OK;
}

extern "C" int elitekv_plan(const int32_t* seq_lens, int32_t B, int32_t tile_tokens,
                            int32_t max_items, int32_t* items, int32_t* seq_first_item,
                            elitekv_stream_t stream) {
  if (!seq_lens || !items || !seq_first_item || B <= 0 || tile_tokens <= 0 || max_items <= B)
    return ELITEKV_ERR_INVALID_ARG;
  if ((uintptr_t)items & 15) return ELITEKV_ERR_INVALID_ARG;
  return ekv_launch_plan(seq_lens, B, tile_tokens, max_items, items, seq_first_item, nullptr, 0,
                         0x7fffffffLL, nullptr, (cudaStream_t)stream);
}

extern "C" int elitekv_plan_workers(const int32_t* seq_lens, int32_t B, int32_t tile_tokens,
                                    int32_t n_workers, int32_t item_overhead_tiles, int32_t max_items,
                                    int32_t* items, int32_t* seq_first_item, int32_t* worker_first,
                                    elitekv_stream_t stream) {
  if (!seq_lens || !items || !seq_first_item || !worker_first || B <= 0 || tile_tokens <= 0 ||
      n_workers <= 0 || max_items < B + n_workers || item_overhead_tiles < 0 || item_overhead_tiles > 64)
    return ELITEKV_ERR_INVALID_ARG;
  if ((uintptr_t)items & 15) return ELITEKV_ERR_INVALID_ARG;
  return ekv_launch_plan_balanced(seq_lens, B, tile_tokens, n_workers, max_items, items, seq_first_item,
                                  worker_first, nullptr, 0, 0x7fffffffLL, nullptr, item_overhead_tiles, (cudaStream_t)stream);
}
