// C entry points: argument checks, workspace carving, kernel selection.
#include "common.cuh"

namespace {

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// Which split-K kernel serves a layer (and cache): 1 = generic CUDA-core kernel, 2 = two-pass
// tcgen05 kernel, 3 = resident-tile tcgen05 kernel on block pairs, -1 = none.  `cache` may be
// null (shape-only question).
int select_kernel(const elitekv_layer* L, const elitekv_cache* cache) {
  const bool tc = ekv_tc_supported(L, cache) != 0;
  const bool rt = ekv_rt_supported(L, cache) != 0;
  if (L->decode_kernel == 3) return rt ? 3 : -1;
  if (L->decode_kernel == 2) return tc ? 2 : -1;
  if (L->decode_kernel == 1) return ekv_generic_supported(L) ? 1 : -1;
  // Choice by shape when both tensor-core kernels cover the layer (measured on B200): the
  // resident-tile kernel has the lower fixed cost and wins on batches of up to a few hundred
  // thousand cached tokens at d_c = 1536 (80 us against 90 us at 16 x 4096); its per-tile chain
  // (exchange between the two blocks of a pair, softmax, value product) makes it the slower one
  // on long streams (0.73 against 0.82 of the copy bandwidth on the 4.6 GB ragged batch) and
  // at narrow latents (d_c = 768).  Lengths live on the device, so the capacity of the cache
  // stands in for them.
  if (rt && tc) {
    long long capacity = 0;
    if (cache) capacity = cache->page_table ? (long long)cache->num_pages * cache->page_size
                                            : (long long)cache->max_ctx * cache->n_seqs;
    const bool small = cache == nullptr || capacity <= 200000;
    return (small && L->d_c >= 1024) ? 3 : 2;
  }
  if (rt) return 3;
  if (tc) return 2;
  return ekv_generic_supported(L) ? 1 : -1;
}

int max_items_for(const elitekv_layer* L, int B, int kernel, int rows = 1) {
  if (kernel == 3) return ekv_rt_max_items(L, B);
  return kernel == 2 ? ekv_tc_max_items(L, B, rows) : ekv_generic_max_items(L, B);
}

// Tokens per plan tile and persistent workers (0: the plain plan) of each kernel.
int plan_tile_for(int kernel) { return kernel == 2 ? 128 : ELITEKV_TILE_TOKENS; }
// Tiles' worth of time that starting an item costs a worker (measured on B200: about one
// 64-token tile for the resident-tile kernel).
int item_overhead_for(int kernel) { return kernel == 3 ? 1 : 0; }
int workers_for(const elitekv_layer* L, int kernel, int rows = 1) {
  return kernel == 3 ? ekv_rt_workers(L) : kernel == 2 ? ekv_tc_workers(L, rows) : 0;
}

// The workspace is sized for whichever kernel may be picked once the cache layout is known.
int max_items_any(const elitekv_layer* L, int B) {
  int m = 0;
  const int want = L->decode_kernel;
  if (ekv_generic_supported(L) && (want == 0 || want == 1)) m = ekv_generic_max_items(L, B);
  if (ekv_tc_supported(L, nullptr) && (want == 0 || want == 2)) {
    const int t = ekv_tc_max_items(L, B, 1);
    if (t > m) m = t;
  }
  if (ekv_rt_supported(L, nullptr) && (want == 0 || want == 3)) {
    const int t = ekv_rt_max_items(L, B);
    if (t > m) m = t;
  }
  return m;
}

struct Carve {
  size_t off_items, off_first, off_ml, off_acc, off_slice, off_cnt, off_wfirst, total;
};

// `rows` query rows per sequence: the partial results, the combine's scratch and its counters
// hold rows x n_h entries where decoding holds n_h.
Carve carve(const elitekv_layer* L, int B, int max_items, int rows = 1) {
  Carve c;
  size_t o = 0;
  c.off_items = o; o = align256(o + sizeof(int32_t) * 4 * (size_t)max_items);
  c.off_first = o; o = align256(o + sizeof(int32_t) * ((size_t)B + 1));
  c.off_ml = o;    o = align256(o + sizeof(float) * 2 * (size_t)max_items * L->n_h * rows);
  c.off_acc = o;   o = align256(o + sizeof(float) * (size_t)max_items * L->n_h * rows * L->vw);
  c.off_slice = o; o = align256(o + ekv_combine_scratch_bytes(L, B) * rows);
  c.off_cnt = o;   o = align256(o + sizeof(int32_t) * (size_t)ekv_combine_counters(L, B) * rows);
  c.off_wfirst = o; o = align256(o + sizeof(int32_t) * ((size_t)L->sm_count + 2));
  c.total = o;
  return c;
}

}  // namespace

extern "C" int elitekv_append(const elitekv_layer* L, const elitekv_cache* cache, const void* k_e,
                              const void* c, const int32_t* seq_id, const int32_t* pos, int64_t T,
                              elitekv_stream_t stream) {
  if (!L || !cache || T < 0) return ELITEKV_ERR_INVALID_ARG;
  if (T == 0) return ELITEKV_OK;
  if (!c || !seq_id || !pos || (L->r > 0 && !k_e)) return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)k_e & 15) || ((uintptr_t)c & 15)) return ELITEKV_ERR_INVALID_ARG;
  CacheView cv;
  int rc = ekv_make_view(cache, &cv);
  if (rc != ELITEKV_OK) return rc;
  rc = ekv_launch_append(L, cache, cv, k_e, c, seq_id, pos, T, (cudaStream_t)stream);
  return rc;
}

extern "C" int elitekv_project_append(const elitekv_layer* L, const elitekv_cache* cache, const void* x,
                                      const int32_t* seq_id, const int32_t* pos, int64_t T,
                                      elitekv_stream_t stream) {
  if (!L || !cache || T < 0) return ELITEKV_ERR_INVALID_ARG;
  if (T == 0) return ELITEKV_OK;
  if (!x || !seq_id || !pos || ((uintptr_t)x & 15)) return ELITEKV_ERR_INVALID_ARG;
  if (L->d <= 0 || !L->d_WcatT) return ELITEKV_ERR_INVALID_ARG;     // layer created without W_ke / W_down
  CacheView cv;
  int rc = ekv_make_view(cache, &cv);
  if (rc != ELITEKV_OK) return rc;
  return ekv_launch_project_append(L, cache, cv, x, seq_id, pos, T, (cudaStream_t)stream);
}

extern "C" int elitekv_absorb_query(const elitekv_layer* L, const void* q, const int32_t* q_pos,
                                    int32_t B, void* q_rope, void* q_abs, elitekv_stream_t stream) {
  if (!L || !q || !q_pos || !q_abs || B < 0 || (L->r > 0 && !q_rope)) return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)q & 15) || ((uintptr_t)q_abs & 15) || ((uintptr_t)q_rope & 3))
    return ELITEKV_ERR_INVALID_ARG;
  int rc = ekv_launch_absorb(L, q, q_pos, B, q_rope, q_abs, (cudaStream_t)stream);
  return rc;
}

extern "C" int elitekv_decode_workspace_size(const elitekv_layer* L, int32_t B, size_t* bytes) {
  if (!L || !bytes || B <= 0) return ELITEKV_ERR_INVALID_ARG;
  const int items = max_items_any(L, B);
  if (items <= 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  *bytes = carve(L, B, items).total;
  return ELITEKV_OK;
}

extern "C" int elitekv_decode_plan_info(const elitekv_layer* L, const elitekv_cache* cache, int32_t B,
                                        int32_t info[5]) {
  if (!L || !info || B <= 0) return ELITEKV_ERR_INVALID_ARG;
  const int kernel = select_kernel(L, cache);
  if (kernel < 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  info[0] = kernel;
  info[1] = plan_tile_for(kernel);
  info[2] = workers_for(L, kernel);
  info[3] = max_items_for(L, B, kernel);
  info[4] = item_overhead_for(kernel);
  return ELITEKV_OK;
}

namespace {

// Plan, split-K kernel and combine of one attention call.  With `plan_stream` set, the plan is
// launched there (beside whatever runs on `st`), `ev_join` is recorded behind it and `st` waits
// for that event before the split-K kernel; `before_kernel` (may be empty) is enqueued on `st`
// in between, i.e. beside the plan.
template <class Fn>
int decode_impl(const elitekv_layer* L, const elitekv_cache* cache, const void* q_rope, const void* q_abs,
                const int32_t* seq_lens, int32_t B, void* workspace, size_t workspace_bytes, void* out,
                cudaStream_t st, cudaStream_t plan_stream, Fn before_kernel, int rows = 1) {
  if (!L || !cache || !q_abs || !seq_lens || !workspace || !out || B <= 0 || (L->r > 0 && !q_rope))
    return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)q_abs & 15) || ((uintptr_t)out & 3)) return ELITEKV_ERR_INVALID_ARG;
  if (B > cache->n_seqs || rows < 1 || rows > ELITEKV_MAX_QUERY_ROWS) return ELITEKV_ERR_INVALID_ARG;
  int kernel = select_kernel(L, cache);
  if (rows > 1) {
    // several query rows run on the two-pass tensor-core kernel only (one block per row and head
    // group walks the same tiles at the same time, so the rows share the tile through L2)
    if (L->decode_kernel != 0 && L->decode_kernel != 2) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
    kernel = ekv_tc_supported(L, cache) ? 2 : -1;
  }
  if (kernel < 0) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  CacheView cv;
  int rc = ekv_make_view(cache, &cv);
  if (rc != ELITEKV_OK) return rc;
  const int max_items = max_items_for(L, B, kernel, rows);
  const Carve cw = carve(L, B, max_items, rows);
  if (((uintptr_t)workspace & 255) || workspace_bytes < cw.total) return ELITEKV_ERR_WORKSPACE_TOO_SMALL;
  unsigned char* base = (unsigned char*)workspace;
  DecodeScratch ws;
  ws.rows = rows;
  ws.seq_lens = seq_lens;
  ws.max_items = max_items;
  ws.items = (int32_t*)(base + cw.off_items);
  ws.seq_first = (int32_t*)(base + cw.off_first);
  ws.part_ml = (float*)(base + cw.off_ml);
  ws.part_acc = (float*)(base + cw.off_acc);
  ws.slice_out = (float*)(base + cw.off_slice);
  ws.counters = (int32_t*)(base + cw.off_cnt);
  ws.n_counters = ekv_combine_counters(L, B) * rows;
  ws.worker_first = (int32_t*)(base + cw.off_wfirst);
  ws.n_workers = workers_for(L, kernel, rows);
  // tokens one sequence can hold: longer lengths are reported by the plan kernel and clamped
  const long long max_len = cv.page_table ? (long long)cv.max_pages_per_seq << cv.page_shift : cv.max_ctx;
  cudaStream_t ps = plan_stream ? plan_stream : st;
  if (ws.n_workers > 0)
    rc = ekv_launch_plan_balanced(seq_lens, B, plan_tile_for(kernel), ws.n_workers, max_items, ws.items, ws.seq_first,
                                  ws.worker_first, ws.counters, ws.n_counters, max_len, L->d_status,
                                  item_overhead_for(kernel), ps);
  else
    rc = ekv_launch_plan(seq_lens, B, plan_tile_for(kernel), max_items, ws.items, ws.seq_first,
                         ws.counters, ws.n_counters, max_len, L->d_status, ps);
  int rc_mid = ELITEKV_OK;
  if (plan_stream) {
    // the join is enqueued whatever happened above, so that the side stream never stays forked
    if (cudaEventRecord(L->ev_join, plan_stream) != cudaSuccess) return ELITEKV_ERR_CUDA;
    rc_mid = before_kernel();
    if (cudaStreamWaitEvent(st, L->ev_join, 0) != cudaSuccess) return ELITEKV_ERR_CUDA;
  }
  if (rc != ELITEKV_OK) return rc;
  if (rc_mid != ELITEKV_OK) return rc_mid;
  EkvProfile* prof = (L->prof && L->prof->enabled && L->prof->count < kProfileSlots) ? L->prof : nullptr;
  if (prof) EKV_CUDA_OK(cudaEventRecord(prof->ev[2 * prof->count], st));
  rc = kernel == 3   ? ekv_launch_decode_rt(L, cache, cv, q_rope, q_abs, B, ws, st)
       : kernel == 2 ? ekv_launch_decode_tc(L, cache, cv, q_rope, q_abs, B, ws, st)
                     : ekv_launch_decode_generic(L, cache, cv, q_rope, q_abs, B, ws, st);
  if (rc != ELITEKV_OK) return rc;
  if (prof) {
    EKV_CUDA_OK(cudaEventRecord(prof->ev[2 * prof->count + 1], st));
    prof->count++;
  }
  return ekv_launch_combine(L, B, ws, out, st);
}

}  // namespace

extern "C" int elitekv_decode(const elitekv_layer* L, const elitekv_cache* cache,
                              const void* q_rope, const void* q_abs, const int32_t* seq_lens,
                              int32_t B, void* workspace, size_t workspace_bytes, void* out,
                              elitekv_stream_t stream) {
  return decode_impl(L, cache, q_rope, q_abs, seq_lens, B, workspace, workspace_bytes, out,
                     (cudaStream_t)stream, nullptr, [] { return (int)ELITEKV_OK; });
}

extern "C" int elitekv_decode_step(const elitekv_layer* L, const elitekv_cache* cache, const void* k_e,
                                   const void* c, const int32_t* seq_id, const int32_t* pos,
                                   const void* q, const int32_t* seq_lens, int32_t B, void* q_rope,
                                   void* q_abs, void* workspace, size_t workspace_bytes, void* out,
                                   elitekv_stream_t stream) {
  if (!L || !cache || B <= 0) return ELITEKV_ERR_INVALID_ARG;
  if (!c || !seq_id || !pos || !q || !q_abs || !seq_lens || !workspace || !out) return ELITEKV_ERR_INVALID_ARG;
  if (L->r > 0 && (!k_e || !q_rope)) return ELITEKV_ERR_INVALID_ARG;
  if (((uintptr_t)k_e & 15) || ((uintptr_t)c & 15) || ((uintptr_t)q & 15) || ((uintptr_t)q_abs & 15) ||
      ((uintptr_t)q_rope & 3))
    return ELITEKV_ERR_INVALID_ARG;
  CacheView cv;
  int rc = ekv_make_view(cache, &cv);
  if (rc != ELITEKV_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // fork: the append (writes the cache) and, behind it, the plan (reads only the lengths) run
  // on the layer's second stream, beside the query preparation on the caller's stream
  EKV_CUDA_OK(cudaEventRecord(L->ev_fork, st));
  EKV_CUDA_OK(cudaStreamWaitEvent(L->side, L->ev_fork, 0));
  const int rc_append = ekv_launch_append(L, cache, cv, k_e, c, seq_id, pos, B, L->side);
  rc = decode_impl(L, cache, q_rope, q_abs, seq_lens, B, workspace, workspace_bytes, out, st, L->side,
                   [&] { return ekv_launch_absorb(L, q, pos, B, q_rope, q_abs, st); });
  if (rc != ELITEKV_OK) {
    // a call that gave up before its own join: bring the side stream back all the same
    cudaEventRecord(L->ev_join, L->side);
    cudaStreamWaitEvent(st, L->ev_join, 0);
  }
  return rc_append != ELITEKV_OK ? rc_append : rc;
}

extern "C" int elitekv_attend_rows_workspace_size(const elitekv_layer* L, int32_t B, int32_t m, size_t* bytes) {
  if (!L || !bytes || B <= 0 || m < 1 || m > ELITEKV_MAX_QUERY_ROWS) return ELITEKV_ERR_INVALID_ARG;
  if (!ekv_tc_supported(L, nullptr)) return ELITEKV_ERR_UNSUPPORTED_SHAPE;
  *bytes = carve(L, B, ekv_tc_max_items(L, B, m), m).total;
  return ELITEKV_OK;
}

extern "C" int elitekv_attend_rows(const elitekv_layer* L, const elitekv_cache* cache, const void* q_rope,
                                   const void* q_abs, const int32_t* seq_lens, int32_t B, int32_t m,
                                   void* workspace, size_t workspace_bytes, void* out,
                                   elitekv_stream_t stream) {
  return decode_impl(L, cache, q_rope, q_abs, seq_lens, B, workspace, workspace_bytes, out,
                     (cudaStream_t)stream, nullptr, [] { return (int)ELITEKV_OK; }, m);
}
