/* elitekv.h -- C ABI of the EliteKV decode-attention library for NVIDIA B200 (sm_100a).
 *
 * EliteKV (arXiv 2503.01586) shrinks the KV cache of a RoPE multi-head-attention layer in two
 * steps.  RoPElite (Section 3.1) keeps the rotary embedding only on r "elite" 2-D chunks per
 * head (each head has its own index set I_r^e); J-LRD (Section 3.2) replaces the remaining key
 * dims of all heads and the values of all heads by ONE latent vector c = x A^kv per token, from
 * which they are up-projected by B^kv = [B^k_J, B^v_J].  Per token and layer the cache therefore
 * holds 2 r n_h rotated key elements plus d_c latent elements (end of Section 3.2).
 *
 * Notation used below (the paper's):
 *   n_h heads, d_h head dim, r elite chunks per head, d_c latent width,
 *   W_uk = B^k_J  [d_c][n_h (d_h - 2r)]   head h owns columns [h (d_h-2r), (h+1)(d_h-2r))
 *   W_uv = B^v_J  [d_c][n_h d_h]          head h owns columns [h d_h, (h+1) d_h)
 *   theta_i = rope_base^(-2 i / d_h), chunk i = dims (2i, 2i+1)            (Section 2.2)
 *
 * One decode step of a layer is   elitekv_append -> elitekv_absorb_query -> elitekv_decode,
 * or the single call elitekv_decode_step, which overlaps the independent parts.
 *
 * General rules
 *   - Pointers are DEVICE pointers unless a comment says "host".  All floating-point tensors
 *     are bf16, row-major, densely packed, with the shapes given; index tensors are int32.
 *   - The caller owns every buffer.  The library allocates device memory only inside
 *     elitekv_layer_create (tables and repacked weights, released by elitekv_layer_destroy).
 *   - Every call only enqueues work on `stream` and returns; lengths, positions and page
 *     tables are read on the device, so a step can be replayed from a CUDA graph.
 *   - Every function returns 0 on success or a negative elitekv_status.  Nothing throws, exits
 *     or asserts on the device.  Invalid arguments are rejected before anything is launched.
 *     Faults that only the device can see (a position beyond max_pos, a page id outside the
 *     pool, a wait that ran out) are recorded in a status word and the offending access is
 *     skipped; elitekv_check_status reads that word.
 */
#ifndef ELITEKV_H_
#define ELITEKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* elitekv_stream_t;   /* a cudaStream_t */
typedef struct elitekv_layer elitekv_layer;     /* opaque */

typedef enum {
  ELITEKV_OK = 0,
  ELITEKV_ERR_INVALID_ARG = -1,
  ELITEKV_ERR_UNSUPPORTED_SHAPE = -2,
  ELITEKV_ERR_WORKSPACE_TOO_SMALL = -3,
  ELITEKV_ERR_CUDA = -4,
  ELITEKV_ERR_TIMEOUT = -5,       /* a bounded device-side wait ran out            */
  ELITEKV_ERR_BAD_PAGE = -6,      /* page id outside [0, num_pages)                */
  ELITEKV_ERR_BAD_POSITION = -7,  /* position outside [0, max_pos) or the cache    */
  ELITEKV_ERR_STATIC_SCRATCH_EXCEEDED = -8  /* elitekv_decode_static: batch/shape needs more
                                               scratch than ELITEKV_STATIC_SCRATCH_BYTES     */
} elitekv_status;

/* Layer description (Sections 3.1 and 3.2).  Host struct; elite_idx is a HOST pointer, the
 * weights are DEVICE pointers that must stay valid until elitekv_layer_create returns. */
typedef struct {
  int32_t n_h, d_h, r, d_c;
  const int32_t* elite_idx;   /* host [n_h][r]: chunk ids of I_r^e per head, distinct, each in
                                 [0, d_h/2).  Their order is the order of the chunks inside a
                                 cached rope row and inside k_e / q_rope.                     */
  float rope_base;            /* 10000 for LLaMA2                                              */
  float softmax_scale;        /* 0 selects 1/sqrt(d_h) (Section 2.1)                           */
  int32_t pair_mode;          /* how chunk i maps to query dims: 0 = (2i, 2i+1) as in Section
                                 2.2; 1 = (i, i + d_h/2).  Keys arrive already paired.         */
  const void* W_uk;           /* bf16 [d_c][n_h*(d_h-2r)]  (B^k_J)                             */
  const void* W_uv;           /* bf16 [d_c][n_h*d_h]       (B^v_J)                             */
  int32_t max_pos;            /* positions are in [0, max_pos)                                 */
  const float* cos_sin;       /* optional DEVICE fp32 [max_pos][d_h/2][2] = (cos, sin) of
                                 pos*theta_i.  NULL: the library tabulates them itself in double
                                 precision at create time.  With a caller table the rotated
                                 values are a pure function of the table (each product and sum
                                 rounded separately in fp32, then bf16 nearest-even).          */
  int32_t decode_kernel;      /* 0 = choose by shape; 1 = generic CUDA-core kernel; 2 = tcgen05
                                 kernel that streams each 128-token tile twice (scores, then
                                 values); 3 = tcgen05 kernel that keeps a 64-token tile
                                 resident in shared memory between the two products.  2 and 3
                                 fail with UNSUPPORTED_SHAPE when the shape is not covered.    */
  /* Only for elitekv_project_append (all three 0 / NULL otherwise): the projections that make
   * the cache row of a token from its hidden state x (Section 3.2, Eq. 2). */
  int32_t d;                  /* model width                                                   */
  const void* W_ke;           /* bf16 [d][n_h*2r]  columns of W^k of the elite chunks, head by
                                 head in the order of elite_idx, (even, odd) inside a chunk    */
  const void* W_down;         /* bf16 [d][d_c]     A^kv  (separated latents: [A^k | A^v])      */
  /* Separated low-rank decomposition (S-LRD, Section 3.2): keys and values have latents of
   * their own.  0: joint latent (J-LRD, everything above as written).  d_ck > 0: a latent row
   * of the cache is [c_k (d_ck) | c_v (d_cv = d_c - d_ck)]; scores read c_k only, outputs c_v
   * only; W_uk is B^k_S, bf16 [d_ck][n_h*(d_h-2r)], W_uv is B^v_S, bf16 [d_cv][n_h*d_h]; q_abs
   * is [B][n_h][d_ck].  d_ck and d_cv must be multiples of 8 (the tcgen05 two-pass kernel wants
   * multiples of 128; the resident-tile kernel does not serve separated latents).  The cache
   * costs 2 r n_h + d_ck + d_cv elements per token. */
  int32_t d_ck;
} elitekv_params;

/* The two cache planes.  Contiguous (page_table == NULL): sequence s, position p live in row
 * s*max_ctx + p.  Paged: row page_table[s][p / page_size]*page_size + p % page_size.  A rope
 * row is [n_h][r][2] (head-major, chunk order of elite_idx, (even, odd)); a latent row is
 * [d_c].  This struct lives on the HOST; its pointer members are DEVICE pointers. */
typedef struct {
  void* rope;                  /* bf16 [rows][n_h*2r]                                          */
  void* latent;                /* bf16 [rows][d_c]                                             */
  const int32_t* page_table;   /* int32 [n_seqs][max_pages_per_seq] or NULL                    */
  int32_t page_size;           /* tokens per page (64 in the benchmarks), power of two         */
  int32_t max_pages_per_seq;
  int64_t num_pages;           /* paged: pages in the pool (rows = num_pages*page_size)        */
  int64_t max_ctx;             /* contiguous: rows per sequence                                */
  int32_t n_seqs;              /* sequences the cache (and page table) is laid out for         */
} elitekv_cache;

/* Validates the description (r <= d_h/2, distinct in-range indices, d_c % 8 == 0, ...), copies
 * the index sets, tabulates (cos, sin) and repacks W_uk for the absorption kernel.  Must be
 * called with the target device current.  `*out` is written only on success. */
int elitekv_layer_create(const elitekv_params* params, elitekv_layer** out);
int elitekv_layer_destroy(elitekv_layer* layer);

/* Cache append (Section 3.1: the rotated elite chunks are stored once, at append time;
 * Section 3.2: one latent shared by all heads).
 * For each of the T new tokens: rotate chunk j of head h by R(pos * theta_{idx[h][j]})
 * (Eq. 1a; (x0,x1) -> (x0 cos - x1 sin, x0 sin + x1 cos)) and write the rope row and the
 * latent row to the token's cache row.  The rotation happens here once; decode never rotates
 * keys again.
 *   k_e    bf16  [T][n_h][r][2]  un-rotated elite key chunks (x W^k_{e,h})
 *   c      bf16  [T][d_c]        latent (x A^kv), copied bit for bit
 *   seq_id int32 [T], pos int32 [T] (0-based position inside the sequence)
 * Tokens must target distinct rows.  T == 0 is a no-op. */
int elitekv_append(const elitekv_layer* layer, const elitekv_cache* cache, const void* k_e,
                   const void* c, const int32_t* seq_id, const int32_t* pos, int64_t T,
                   elitekv_stream_t stream);

/* Projection fused with the cache append (Section 3.2: k_e = x W^k_e, c = x A^kv; Section 3.1:
 * rotation of the elite chunks at the token's position): what elitekv_append does, starting
 * from the hidden states, in one kernel -- x [T][d] . [W^k_e | A^kv] on the tensor cores (fp32
 * accumulation), rotation and the single rounding to bf16 in the epilogue, rows written straight
 * into the cache.  k_e and c never exist in memory.
 *   x bf16 [T][d], 16-byte aligned;  seq_id, pos int32 [T] as for elitekv_append.
 * Needs a layer created with d, W_ke and W_down; d a multiple of 64 and both n_h*2r and d_c
 * multiples of 128 (ELITEKV_ERR_UNSUPPORTED_SHAPE otherwise).  Stored values differ from
 * elitekv_append(bf16(x W^k_e), bf16(x A^kv)) by the intermediate rounding only. */
int elitekv_project_append(const elitekv_layer* layer, const elitekv_cache* cache, const void* x,
                           const int32_t* seq_id, const int32_t* pos, int64_t T,
                           elitekv_stream_t stream);

/* Query preparation (score equation of Section 3.1; absorption of B^k, Section 5).
 *   q      bf16  [B][n_h][d_h]  un-rotated queries,  q_pos int32 [B]
 *   q_rope bf16  [B][n_h][2r]   elite chunks of q rotated at q_pos
 *   q_abs  bf16  [B][n_h][d_c]  (separated latents: [B][n_h][d_ck])  q_nope[b,h,:] . W_uk,h^T, q_nope = the other d_h-2r dims of
 *                               q[b,h] in ascending order; fp32 accumulation. */
int elitekv_absorb_query(const elitekv_layer* layer, const void* q, const int32_t* q_pos,
                         int32_t B, void* q_rope, void* q_abs, elitekv_stream_t stream);

/* Scratch needed by elitekv_decode for a batch of B sequences (split-K partial results and
 * the work plan).  It depends on the layer shape, on B and on the device, not on the lengths. */
int elitekv_decode_workspace_size(const elitekv_layer* layer, int32_t B, size_t* bytes);

/* Decode attention over the compressed cache (Sections 2.1, 3.1, 3.2, 5):
 *   s[b,h,t] = q_rope[b,h] . k_rope[t,h] + q_abs[b,h] . c[t]        t < seq_lens[b]
 *   p = softmax(scale * s),   o[b,h] = (sum_t p[b,h,t] c[t]) . W_uv,h
 * seq_lens[b] counts the cached tokens INCLUDING the one just appended (the query attends to
 * its own token).  seq_lens[b] == 0 gives a zero row.
 *   out bf16 [B][n_h][d_h];  workspace: 256-byte aligned, at least
 *   elitekv_decode_workspace_size bytes, private to this call until the stream reaches its end.
 * Launches: plan, split-K attention, combine + up-projection.  The three kernels are launched
 * with programmatic stream serialisation: each may start its private set-up while the kernel
 * before it on the stream drains, but reads and writes nothing shared before every earlier
 * kernel on the stream has completed, so the usual stream order holds for the caller (two
 * calls may share one workspace on one stream). */
int elitekv_decode(const elitekv_layer* layer, const elitekv_cache* cache, const void* q_rope,
                   const void* q_abs, const int32_t* seq_lens, int32_t B, void* workspace,
                   size_t workspace_bytes, void* out, elitekv_stream_t stream);

/* One whole decode step of a layer in one call (Sections 3.1, 3.2, 5): token b (cache entries
 * k_e[b], c[b]) is appended to sequence seq_id[b] at position pos[b], the query q[b] is
 * prepared at that same position (elitekv_absorb_query with q_pos = pos) into the caller's
 * q_rope / q_abs buffers, and elitekv_decode runs over seq_lens (the lengths INCLUDING the new
 * tokens).  Arguments, shapes, alignment and errors are those of the three calls; the result
 * is bit-identical to calling them in order.  The append and the work plan depend only on the
 * new tokens and the lengths, so they run on a stream the layer owns, beside the query
 * preparation on `stream`, and are joined before the attention kernel; to the caller the call
 * behaves like work enqueued on `stream` alone (it may be captured in a CUDA graph).  Two
 * threads must not run steps of the same layer object at the same time. */
int elitekv_decode_step(const elitekv_layer* layer, const elitekv_cache* cache, const void* k_e,
                        const void* c, const int32_t* seq_id, const int32_t* pos, const void* q,
                        const int32_t* seq_lens, int32_t B, void* q_rope, void* q_abs,
                        void* workspace, size_t workspace_bytes, void* out, elitekv_stream_t stream);

/* Several query rows per sequence over the cache, with the causal rule (Section 3.1: the score
 * equation holds for any query position m and key position n): a chunk of a prefill, or the
 * draft tokens of speculative decoding.  The m new tokens of every sequence are in the cache
 * already (elitekv_append / elitekv_project_append); seq_lens[b] counts them.  Query row i of
 * sequence b sits at position seq_lens[b] - m + i and attends to the cached tokens at positions
 * <= its own, i.e. to the first seq_lens[b] - (m - 1 - i) tokens; a row that sees none gives a
 * zero row.
 *   q_rope bf16 [B][m][n_h][2r], q_abs bf16 [B][m][n_h][d_c]: elitekv_absorb_query on the B*m
 *          rows with q_pos[b*m + i] = seq_lens[b] - m + i
 *   out    bf16 [B][m][n_h][d_h]
 *   workspace: as for elitekv_decode, sized by elitekv_attend_rows_workspace_size(B, m)
 * 1 <= m <= ELITEKV_MAX_QUERY_ROWS.  Runs on the two-pass tcgen05 kernel only (shapes it does
 * not cover, or a layer created with decode_kernel 1 or 3: ELITEKV_ERR_UNSUPPORTED_SHAPE): one
 * block per query row and head group walks the same token tiles at the same time, so a tile
 * comes from HBM once and the other rows read it from L2.  m = 1 is elitekv_decode. */
#define ELITEKV_MAX_QUERY_ROWS 16
int elitekv_attend_rows_workspace_size(const elitekv_layer* layer, int32_t B, int32_t m, size_t* bytes);
int elitekv_attend_rows(const elitekv_layer* layer, const elitekv_cache* cache, const void* q_rope,
                        const void* q_abs, const int32_t* seq_lens, int32_t B, int32_t m,
                        void* workspace, size_t workspace_bytes, void* out, elitekv_stream_t stream);

/* RoPElite search (Algorithm 1, Section 3.1) on calibration activations: which r chunks of every
 * head keep their rotation.  Q, K: bf16 [n_heads][n][d_h], un-rotated queries and keys of a
 * calibration sequence of n tokens (token t at position t), heads of all layers side by side;
 * d_h is 64 or 128.  A round computes, per head and per chunk j not yet chosen, the L1 distance
 * over all causal pairs (query position m, key position <= m) between the pre-softmax scores
 * q K^T with RoPE on every chunk and with RoPE on the chosen chunks plus j only; the first
 * minimum joins the head's list.
 *   elitekv_ropelite_distances: one round for given lists.  elite_mask: uint64 [n_heads], bit i
 *     set = chunk i already chosen (NULL: none).  dist: fp32 [n_heads][d_h/2], +inf at chosen
 *     chunks.
 *   elitekv_ropelite_search: r rounds.  elite_idx: int32 [n_heads][r], chunks in the order
 *     chosen (the order elitekv_params.elite_idx wants).  dist_trace: optional fp32
 *     [r][n_heads][d_h/2], the distances of every round.
 * Sums are fp32 and added in a fixed order (results do not depend on scheduling).  workspace:
 * 256-byte aligned, elitekv_ropelite_workspace_size bytes. */
int elitekv_ropelite_workspace_size(int32_t n_heads, int32_t n, int32_t d_h, size_t* bytes);
int elitekv_ropelite_distances(const void* Q, const void* K, int32_t n_heads, int32_t n, int32_t d_h,
                               float rope_base, const uint64_t* elite_mask, void* workspace,
                               size_t workspace_bytes, float* dist, elitekv_stream_t stream);
int elitekv_ropelite_search(const void* Q, const void* K, int32_t n_heads, int32_t n, int32_t d_h,
                            float rope_base, int32_t r, void* workspace, size_t workspace_bytes,
                            int32_t* elite_idx, float* dist_trace, elitekv_stream_t stream);

/* Decode attention without any allocation (the paper has no counterpart; this is a packaging
 * variant of elitekv_decode).  For callers that must not, or cannot, call cudaMalloc: engines
 * that give all device memory to one arena up front, plugins running inside another
 * framework's step, latency-critical loops.  Same arguments and result as elitekv_decode, minus
 * the workspace: the scratch lives in a device array of ELITEKV_STATIC_SCRATCH_BYTES inside the
 * library, which every GPU that loads the library holds until the process exits.
 *   - Returns ELITEKV_ERR_STATIC_SCRATCH_EXCEEDED, launching nothing, when
 *     elitekv_decode_workspace_size(layer, B) exceeds ELITEKV_STATIC_SCRATCH_BYTES
 *     (a 7B-shaped layer at 75 % reduction with B = 16 needs about 31 MiB).
 *   - Calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - The first call on a device looks up the array's device address
 *     (cudaGetSymbolAddress, with the layer's device current); make that first call before
 *     any stream capture begins.  The layer's device must be the current device.
 *   - All calls share the one array, which keeps the previous call's contents (nothing in it
 *     needs clearing between calls).  Two calls whose kernels can overlap on the GPU -- other
 *     streams, other host threads, other layers -- race on it: order them on one stream. */
#define ELITEKV_STATIC_SCRATCH_BYTES (48u << 20)
int elitekv_decode_static(const elitekv_layer* layer, const elitekv_cache* cache,
                          const void* q_rope, const void* q_abs, const int32_t* seq_lens,
                          int32_t B, void* out, elitekv_stream_t stream);

/* Work plan of the split-K kernel, exported for inspection (the paper has no counterpart: it
 * is this library's load balancer for ragged batches).  Cuts the batch's token tiles into at
 * most `max_items` pieces of near-equal size, never across a sequence.
 *   items int32 [max_items][4] = (sequence, first token, token count, 0);  unused entries have
 *   sequence = -1.   seq_first_item int32 [B+1]: items of sequence b are
 *   [seq_first_item[b], seq_first_item[b+1]). */
int elitekv_plan(const int32_t* seq_lens, int32_t B, int32_t tile_tokens, int32_t max_items,
                 int32_t* items, int32_t* seq_first_item, elitekv_stream_t stream);

/* The plan of the kernels whose blocks are persistent workers (the paper has no counterpart),
 * exported for inspection.  Worker w owns the global tile range [w*total/n, (w+1)*total/n),
 * n = min(n_workers, total) (integer division; later workers stay idle); an item is the part
 * of one sequence inside one worker's range, so items come out ordered by sequence and worker.
 *   items int32 [max_items][4] = (sequence, first token, token count, worker), unused entries
 *   sequence = -1;  seq_first_item int32 [B+1];  worker_first int32 [n_workers+1]: items of
 *   worker w are [worker_first[w], worker_first[w+1]).  max_items >= B + n_workers.
 * item_overhead_tiles (>= 0): empty tiles counted in front of every sequence when the ranges
 * are cut, the price of starting one more item; 0 gives the plain equal-tile cut. */
int elitekv_plan_workers(const int32_t* seq_lens, int32_t B, int32_t tile_tokens, int32_t n_workers,
                         int32_t item_overhead_tiles, int32_t max_items, int32_t* items,
                         int32_t* seq_first_item, int32_t* worker_first, elitekv_stream_t stream);

/* Which split-K kernel and plan elitekv_decode uses for this layer, cache layout (may be NULL:
 * shape-only answer) and batch (the paper has no counterpart).  info is a HOST array:
 * info[0] = kernel (1, 2, 3 as in elitekv_params.decode_kernel), info[1] = tokens per plan tile,
 * info[2] = persistent workers (0: the plain plan of elitekv_plan), info[3] = plan capacity,
 * info[4] = item_overhead_tiles of elitekv_plan_workers. */
int elitekv_decode_plan_info(const elitekv_layer* layer, const elitekv_cache* cache, int32_t B,
                             int32_t info[5]);

/* Synchronises `stream`, returns the layer's device status word (0 or a negative
 * elitekv_status recorded by a kernel) and clears it. */
int elitekv_check_status(const elitekv_layer* layer, elitekv_stream_t stream);

/* The two detail words and the fault count that the last elitekv_check_status of this layer
 * read together with the code it returned (host array; e.g. sequence and length for
 * BAD_POSITION, sequence and page id for BAD_PAGE, worker | wait code << 16 for TIMEOUT). */
int elitekv_last_status_detail(const elitekv_layer* layer, int32_t detail[3]);

/* Self-test of the bounded waits (the paper has no counterpart).  Launches one small block that
 * initialises a shared-memory barrier nobody will ever arrive on and waits for it with each of
 * the library's wait helpers (single thread, whole warp, group with a leader), every wait
 * limited to `poll_limit` probes.  Each wait must give up: the kernel then records
 * ELITEKV_ERR_TIMEOUT in the layer's status word (detail[0] = bit mask of the helpers that gave
 * up as they should: 7 when all three did) and the block exits normally.  It touches no
 * tensor memory, issues no copy and leaves the device usable.  poll_limit in [1, 2^20]. */
int elitekv_selftest_bounded_wait(const elitekv_layer* layer, uint32_t poll_limit,
                                  elitekv_stream_t stream);

/* Comparator: uncompressed RoPE multi-head attention decode (Sections 2.1 and 2.2) over a
 * contiguous cache of rotated keys and values.
 *   q_hat bf16 [B][n_h][d_h] rotated query;  K_hat, V bf16 [B][max_ctx][n_h][d_h];
 *   out bf16 [B][n_h][d_h];  scale 0 selects 1/sqrt(d_h). */
int elitekv_mha_workspace_size(int32_t B, int32_t n_h, int32_t d_h, size_t* bytes);
int elitekv_mha_decode(const void* q_hat, const void* K_hat, const void* V,
                       const int32_t* seq_lens, int32_t B, int32_t n_h, int32_t d_h,
                       int64_t max_ctx, float scale, void* workspace, size_t workspace_bytes,
                       void* out, elitekv_stream_t stream);

/* Timing aid (the paper has no counterpart).  While enabled, elitekv_decode brackets its
 * split-K attention kernel with a pair of CUDA events on the caller's stream (up to 512 calls
 * between collections).  elitekv_profile_collect waits for the recorded events, returns the
 * summed kernel time in milliseconds and the number of launches it covers, and starts over. */
int elitekv_profile_enable(elitekv_layer* layer, int32_t on);
int elitekv_profile_collect(elitekv_layer* layer, float* total_ms, int32_t* launches);

const char* elitekv_strerror(int status);

#ifdef __cplusplus
}
#endif
#endif /* ELITEKV_H_ */
