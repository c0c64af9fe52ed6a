/*
 * ilre_recall.h -- C ABI of the B200 (sm_100a) implementation of ILRe's token-recall path.
 *
 * The path is the part of the paper's pipeline that runs once per request at the retrieval
 * layer l_R (Section 3.3, bullets "Calculate A^C ..." and "Apply Algorithm 1 ..."):
 *
 *   Eq. 4   s[h,i,t] = q[i,h,:] . K[t, kv(h), :] / sqrt(d_h),  softmax over the L context keys
 *   Eq. 5   A^C[t]   = max over all query heads h and query tokens i of that softmax
 *   Alg. 1  "Context Allocation": strided max pooling (size = stride = m_i), stride-1
 *           window pooling (size n_j), top-K_m per (m_i, n_j) combination, an even budget
 *           split B_c over the combinations with de-duplication ("next-highest-ranked
 *           candidate"), and an ascending sort of the chosen positions.
 *
 * All pointers whose name ends in _dev are device pointers on the handle's device; _host
 * pointers are host pointers.  No torch or C++ types cross this boundary.  Every function
 * returns ILRE_OK (0) or a negative ilre_status code; nothing is launched when argument
 * validation fails.  The library never falls back to the CPU.
 */
#ifndef ILRE_RECALL_H_
#define ILRE_RECALL_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ilre_recall ilre_recall_t;   /* opaque; owns workspace, events, nothing else */

enum ilre_status {
  ILRE_OK = 0,
  ILRE_ERR_INVALID_ARG = -1,  /* null pointer, L < 1, q_len < 1, a pooling size < 1, ...    */
  ILRE_ERR_UNSUPPORTED = -2,  /* head_dim != 128, n_q_heads % n_kv_heads != 0, not sm_100,  */
                              /* reduce_op != 0                                              */
  ILRE_ERR_CAPACITY = -3,     /* L, q_len, budget or #combinations above the create() caps  */
  ILRE_ERR_BUDGET = -4,       /* budget > L - n_sink                                         */
  ILRE_ERR_ALIGNMENT = -5,    /* key cache or query base address not 16-byte aligned         */
  ILRE_ERR_CUDA = -6,         /* a CUDA runtime/driver call failed                           */
  ILRE_ERR_DEVICE_WAIT = -7,  /* a bounded wait inside a kernel gave up (see _status)        */
  ILRE_ERR_QUOTA = -8,        /* a combination ran out of candidates (cannot happen for valid */
                              /* inputs; reported by _status)                                */
  ILRE_ERR_NOMEM = -9         /* workspace allocation failed in create()                     */
};

/* Capacities fixed at create(); run() never allocates. */
typedef struct {
  int32_t n_kv_heads;        /* e.g. 8                                                       */
  int32_t n_q_heads;         /* e.g. 32; query head h reads kv head h / (n_q/n_kv)           */
  int32_t head_dim;          /* must be 128                                                  */
  int64_t max_L;             /* largest context length, < 2^31 - 256                         */
  int32_t max_q_len;         /* largest number of query tokens                               */
  int32_t max_budget;        /* largest budget B, <= 16382                                   */
  int32_t max_combinations;  /* largest N_M * N_A, e.g. 48                                   */
  int32_t device;            /* CUDA device ordinal                                          */
  int32_t host_staging;      /* != 0: also allocate device staging for ilre_recall_run_host  */
} ilre_recall_config_t;

/* Pooling spec of Algorithm 1.  The arrays are host memory, read before run() returns. */
typedef struct {
  int32_t n_max;             /* N_M */
  const int32_t* max_sizes;  /* m_i: MaxPooling size == stride; {1} switches it off           */
  int32_t n_win;             /* N_A */
  const int32_t* win_sizes;  /* n_j: stride-1 window; covers cells [c - n/2, c - n/2 + n-1]  */
  int32_t win_op;            /* 0 = average (Algorithm 1; zero padding, divisor n), 1 = max   */
  int32_t reduce_op;         /* 0 = max over (head, query token) (Eq. 5); others reserved    */
  int32_t n_sink;            /* S: leading positions always returned, excluded from pooling  */
} ilre_pool_spec_t;

/*
 * Create a handle on cfg->device: allocates all device workspace (row statistics, packed
 * query, scores, pooled arrays [max_combinations][max_L], candidate lists, bitmap, status).
 * *out is set only on success.  The handle may be used from one host thread and one stream
 * at a time.
 */
int ilre_recall_create(const ilre_recall_config_t* cfg, ilre_recall_t** out);

/*
 * One recall (Eq. 4, Eq. 5, Algorithm 1), asynchronous on cuda_stream (a cudaStream_t passed
 * as void*; NULL = default stream).  Does not synchronise.
 *   k_cache_dev   bf16 [L][n_kv_heads][128], RoPE already applied, 16-byte aligned; read only
 *   query_dev     bf16 [q_len][n_q_heads][128], 16-byte aligned; read only
 *   budget        B, 0 <= B <= L - n_sink
 *   out_idx_dev   int32 [n_sink + budget]: chosen context positions, ascending (may be NULL when
 *                 n_sink + budget = 0: the result is empty)
 *   out_scores_dev  optional fp32 [L]: A^C of Eq. 5 (NULL to skip)
 * The call only encodes two tensor maps on the host and launches kernels on cuda_stream (no
 * allocation, no synchronisation), so it may be captured into a CUDA graph and replayed.
 * Ranking inside a combination is (pooled value descending, cell index ascending); K_m =
 * B/m + 1 (+1 when L - n_sink is not a multiple of m), B_c = B/N_c with the remainder given
 * to the first combinations in loop order (max sizes outer, window sizes inner).
 */
int ilre_recall_run(ilre_recall_t* h,
                    const void* k_cache_dev, int64_t L,
                    const void* query_dev, int32_t q_len,
                    int32_t budget, const ilre_pool_spec_t* spec,
                    int32_t* out_idx_dev, float* out_scores_dev,
                    void* cuda_stream);

/*
 * Same computation from HOST buffers (handle created with host_staging != 0): copies the
 * key cache and query to device staging, runs, copies the indices (and scores if asked)
 * back, and synchronises the stream before returning.  For throughput the host buffers
 * should be page-locked.  Contexts of more than 65536 positions are uploaded in up to 16 pieces
 * on an internal stream while the row statistics of the pieces already on the device are
 * computed; the pieces' statistics are merged as those of key shards are, so the scores may
 * differ from ilre_recall_run's in the rounding order of the softmax denominator (a few fp32
 * ulps).
 */
int ilre_recall_run_host(ilre_recall_t* h,
                         const void* k_cache_host, int64_t L,
                         const void* query_host, int32_t q_len,
                         int32_t budget, const ilre_pool_spec_t* spec,
                         int32_t* out_idx_host, float* out_scores_host,
                         void* cuda_stream);

/*
 * Key-range sharded recall (the context's keys split by position over several GPUs, as the
 * key cache of a long context is when it does not fit, or is not produced on, one device).
 * Eq. 4's softmax runs over ALL keys, so a shard needs every shard's row statistics before it
 * can score its own positions; Eq. 5 and Algorithm 1 then need every position's score.  The
 * three calls below are the per-rank steps, with one all-gather between each pair (the caller
 * owns the exchange; the library never talks to a peer):
 *
 *   1. ilre_recall_shard_stats: for this shard's keys, per query row r = i * n_q_heads + h,
 *      stats_out_dev[r] = (max_t x_rt, sum_t 2^(x_rt - max)) with x = log2(e) q.k / sqrt(128),
 *      fp32 pairs [q_len * n_q_heads][2].
 *      -> all-gather into stats_all_dev [n_shards][q_len * n_q_heads][2] (any shard order).
 *   2. ilre_recall_shard_scores: A^C (Eq. 5) of this shard's positions under the softmax over
 *      all shards' keys: scores_out_dev fp32 [L_shard].  Also publishes the global per-row lse
 *      (ilre_recall_copy_row_lse).
 *      -> all-gather into scores [L] in position order.
 *   3. ilre_recall_allocate: Algorithm 1 on given scores (fp32 [L], finite and >= 0; read
 *      only): out_idx_dev int32 [n_sink + budget] ascending.  Every rank may run it (the result
 *      is the same everywhere) or one rank may and broadcast the indices.
 *
 * With one shard the three calls give exactly what ilre_recall_run gives.  With several, the
 * scores differ from the unsharded run only in the rounding order of the softmax denominator
 * (a few fp32 ulps).  L_shard, q_len, budget, spec: as for ilre_recall_run, against the
 * handle's capacities.  Asynchronous on cuda_stream; workspace rule as for ilre_recall_run.
 */
int ilre_recall_shard_stats(ilre_recall_t* h, const void* k_shard_dev, int64_t L_shard,
                            const void* query_dev, int32_t q_len, float* stats_out_dev,
                            void* cuda_stream);
int ilre_recall_shard_scores(ilre_recall_t* h, const void* k_shard_dev, int64_t L_shard,
                             const void* query_dev, int32_t q_len, const float* stats_all_dev,
                             int32_t n_shards, float* scores_out_dev, void* cuda_stream);
int ilre_recall_allocate(ilre_recall_t* h, const float* scores_dev, int64_t L, int32_t budget,
                         const ilre_pool_spec_t* spec, int32_t* out_idx_dev, void* cuda_stream);

/*
 * Streaming chunked prefill attention of one chunk in a layer before the retrieval layer
 * (Section 3.1, Eq. 2 with the Lambda-shaped mask; Section 3.3, the step for layers 1..l_R-1,
 * where only S sink and W sliding-window rows of K and V are kept between chunks):
 *   out[j, h, :] = sum_k softmax_k(q[j, h, :] . k[k, kv(h), :] / sqrt(128)) v[k, kv(h), :],
 *   k = 0 .. n_prefix + j,
 * where the first n_prefix rows of k/v are the cached sink and sliding-window tokens, visible to
 * every query, and the following chunk_len rows the chunk's own, visible causally.  The caller
 * keeps the cache (sink S, window W) and lays the rows out in that order.
 *   q_dev    bf16 [chunk_len][n_q_heads][128]             (RoPE applied)
 *   k_dev    bf16 [n_prefix + chunk_len][n_kv_heads][128] (RoPE applied)
 *   v_dev    bf16 [n_prefix + chunk_len][n_kv_heads][128]
 *   out_dev  bf16 [chunk_len][n_q_heads][128]
 * All 16-byte aligned.  Products on the tensor cores with fp32 accumulation; the probabilities
 * are rounded to bf16 before they multiply the values (as the output is).  Asynchronous on
 * cuda_stream; bounded waits report through ilre_recall_status.
 */
int ilre_recall_chunk_attention(ilre_recall_t* h, const void* q_dev, const void* k_dev,
                                const void* v_dev, int32_t chunk_len, int32_t n_prefix,
                                void* out_dev, void* cuda_stream);

/*
 * Key-cache fill of the retrieval layer (Section 3.3, the step at layer l_R: the context's key
 * states are computed chunk by chunk into a cache pre-allocated for all L positions; Eq. 1 with
 * the positional encoding of Eq. 3):
 *   K[pos0 + t, g, :] = R(pos0 + t) (x[t, :] . W_K[g*128 : (g+1)*128, :]^T + b[g*128 : (g+1)*128])
 * for t = 0 .. n_tok-1 and every kv head g, where R(p) is RoPE at position p in the
 * rotate-half layout (pair (c, c + 64) turns by p * rope_theta^(-2c/128)).  One call fills the
 * rows [pos0, pos0 + n_tok) of the cache, e.g. one prefill chunk.
 *   x_dev        bf16 [n_tok][d_model] hidden states entering the key projection
 *   w_k_dev      bf16 [n_kv_heads * 128][d_model], one row per output channel
 *   bias_dev     bf16 [n_kv_heads * 128] or NULL
 *   k_cache_dev  bf16 [L][n_kv_heads][128]; rows outside [pos0, pos0 + n_tok) are not touched
 * d_model must be a multiple of 64 (ILRE_ERR_UNSUPPORTED), pos0 + n_tok <= L <= max_L
 * (ILRE_ERR_CAPACITY), all three tensors 16-byte aligned.  bf16 x bf16 products accumulate in
 * fp32 on the tensor cores; bias, rotation in fp32 from angle tables built in double precision;
 * one rounding to bf16.  Asynchronous on cuda_stream; bounded waits report through
 * ilre_recall_status.  The handle keeps the angle tables between calls (they depend on
 * rope_theta only); a call on another stream than the one that built them waits for the build
 * on the device, but calls with different rope_theta on one handle must not overlap.  Under
 * CUDA-graph capture: a call that would have to build the tables returns ILRE_ERR_UNSUPPORTED
 * (make one call with this rope_theta before the capture), and a captured call does not wait
 * for a build issued on another stream: launch the graph behind that build.
 */
int ilre_recall_fill_keys(ilre_recall_t* h, const void* x_dev, int64_t n_tok, int32_t d_model,
                          const void* w_k_dev, const void* bias_dev, int64_t pos0,
                          double rope_theta, void* k_cache_dev, int64_t L, void* cuda_stream);

/*
 * Dual Chunk Attention re-rotation of the retrieval layer's cached keys (Section 3.3, Eq. 7),
 * to be applied before ilre_recall_run when DCA is on:
 *   K~[t] = R(D_i) K[t]  for every position t of chunk i < N_C - 1,  D_i = (N_C - 1 - i) * chunk_size,
 * where chunk 1 holds the n_sink sink tokens plus chunk_size tokens, every later chunk
 * chunk_size tokens (the last possibly fewer), N_C = ceil((L - n_sink) / chunk_size), and R(D)
 * is the RoPE rotation by D positions in the rotate-half layout (channel pair (c, c + 64) turns
 * by D * rope_theta^(-2c/128)).  The last two chunks stay as they are.
 *   k_cache_dev  bf16 [L][n_kv_heads][128], 16-byte aligned
 *   k_out_dev    same shape; may be k_cache_dev itself (in place) or a separate buffer, in
 *                which case the unrotated chunks are copied
 * Arithmetic: fp32 from an angle table computed in double precision, one rounding to bf16
 * (nearest even).  Asynchronous on cuda_stream.  At most 8192 + 2 chunks
 * (ILRE_ERR_CAPACITY beyond).  The handle keeps the angle table between calls; a call on
 * another stream waits on the device for the table's build, but calls that need different
 * tables (chunk size, theta, more rows) must not overlap on one handle.  Under CUDA-graph
 * capture: a call that would have to (re)build the table returns ILRE_ERR_UNSUPPORTED (make one
 * call with these arguments before the capture), and a captured call does not wait for a build
 * issued on another stream: launch the graph behind that build.
 */
int ilre_recall_rerope_keys(ilre_recall_t* h, const void* k_cache_dev, void* k_out_dev,
                            int64_t L, int32_t chunk_size, int32_t n_sink, double rope_theta,
                            void* cuda_stream);

/*
 * Dual Chunk Attention in the layers before the retrieval layer (Eq. 6): the sink keys as the
 * prefill of chunk i sees them, K^{S,i} = R^{i-2}(D_C) K^S for i > 2 (chunk_index is 1-based;
 * the first two chunks see the cached keys, which are then only copied).  The power of the
 * rotation is applied as one rotation by (chunk_index - 2) * chunk_size positions to the
 * CACHED sink keys (keep them; do not feed a rotated copy back in), so the result is rounded
 * to bf16 once.  R(D) as in ilre_recall_rerope_keys.
 *   k_sink_dev  bf16 [n_sink][n_kv_heads][128], 16-byte aligned; read only
 *   k_out_dev   bf16 [n_sink][n_kv_heads][128]; may be k_sink_dev (in place)
 * chunk_index <= 8194 (ILRE_ERR_CAPACITY beyond).  Shares the handle's angle table with
 * ilre_recall_rerope_keys: calls on one handle must not overlap, and alternating between
 * different chunk sizes rebuilds the table.  Asynchronous on cuda_stream.
 */
int ilre_recall_rerope_sinks(ilre_recall_t* h, const void* k_sink_dev, void* k_out_dev,
                             int32_t n_sink, int32_t chunk_size, int32_t chunk_index,
                             double rope_theta, void* cuda_stream);

/*
 * The compressed prompt (Algorithm 1's last line, C~ = C[I], and Section 3.3's last step):
 *   out[i] = input_ids[idx[i]] for i < n_idx, then the n_query ids of the query part.
 * All pointers are int32 arrays on the current device; idx is what ilre_recall_run returned.
 * A position outside [0, L) yields -1.  No handle; asynchronous on cuda_stream.
 */
int ilre_gather_input_ids(const int32_t* input_ids_dev, int64_t L, const int32_t* idx_dev,
                          int32_t n_idx, const int32_t* query_ids_dev, int32_t n_query,
                          int32_t* out_ids_dev, void* cuda_stream);

/*
 * Offline choice of the retrieval layer l_R (Section 3.3, first paragraph, with the retrieval
 * task of Appendix A.1): the recall is run once per candidate layer on a context with planted
 * key phrases; a phrase counts as retrieved only if every one of its positions was recalled
 * (exact match); a layer's recall rate is its share of retrieved phrases; l_R is the layer
 * with the smallest index among those with the highest rate.
 *   idx_dev         int32 [n_layers][n_idx]: each layer's recalled positions, ascending,
 *                   without repeats (ilre_recall_run's output, one row per layer)
 *   span_begin_dev  int32 [n_spans]: first position of each phrase
 *   span_len_dev    int32 [n_spans]: its length, >= 1
 *   hits_out_dev    int32 [n_layers][n_spans]: recalled positions inside each phrase (NULL to skip)
 *   full_out_dev    int32 [n_layers]: phrases retrieved completely (rate = this / n_spans)
 *   layer_out_dev   int32 [1]: the chosen layer's row index
 * All pointers on the current device.  n_layers <= 1024 (ILRE_ERR_CAPACITY beyond).  No handle;
 * asynchronous on cuda_stream.
 */
int ilre_layer_recall(const int32_t* idx_dev, int32_t n_layers, int32_t n_idx,
                      const int32_t* span_begin_dev, const int32_t* span_len_dev, int32_t n_spans,
                      int32_t* hits_out_dev, int32_t* full_out_dev, int32_t* layer_out_dev,
                      void* cuda_stream);

/*
 * Row statistics of the last run (Eq. 4's softmax denominator): copies
 * lse[i * n_q_heads + h] = log(sum_t exp(s[h,i,t])) (natural log, fp32) for the q_len rows
 * of that run into out_lse_dev, asynchronously on cuda_stream.
 */
int ilre_recall_copy_row_lse(ilre_recall_t* h, float* out_lse_dev, int32_t q_len,
                             void* cuda_stream);

/*
 * Device status word of the handle.  Synchronises the stream of the last run, then returns
 * ILRE_OK, ILRE_ERR_DEVICE_WAIT or ILRE_ERR_QUOTA, and clears the word.
 */
int ilre_recall_status(ilre_recall_t* h);

/*
 * SM clock, in MHz, that the row-statistics kernel of the last run with profiling on really ran
 * at: SM cycles of its first CTA over the global timer's nanoseconds (0 if no such run yet).
 * Under the board's power cap this is well below the clock the driver reports.  Measurement
 * aid; the paper has no counterpart.  Synchronises the last run's stream.
 */
int ilre_recall_sm_clock(ilre_recall_t* h, float* mhz_out_host);

/*
 * Stage timing.  With profiling on, run() records CUDA events between its stages on the
 * caller's stream (the events of the 32 most recent runs are kept).  Switching profiling on
 * resets the history.  ilre_recall_stage_times synchronises on those events and writes up to
 * n entries, each the mean over the recorded runs (milliseconds), in this order:
 *   0 prepare (query packing, clears)   1 row statistics (QK^T + online softmax)
 *   2 scores (statistics merge, QK^T + max over rows)
 *   3 Algorithm 1 (A^C from the maxima, pooling, top-K_m selection and ranking, allocation,
 *     ascending output; one kernel)
 * Returns the number of entries written, or a negative status.
 */
int ilre_recall_set_profiling(ilre_recall_t* h, int32_t on);
int ilre_recall_stage_times(ilre_recall_t* h, float* ms_host, int32_t n);

/*
 * Failure-detection self test.  Every wait inside the kernels (mbarrier waits of the TMA /
 * tensor-core pipelines, the grid barrier of the Algorithm 1 kernel) is bounded: a wait that
 * runs past its spin budget records a code in the handle's status word, its CTA leaves the
 * kernel in an orderly way (no trap, tensor memory released), and ilre_recall_status returns
 * ILRE_ERR_DEVICE_WAIT after the caller's next synchronisation.  This call lets a test reach
 * that path without faulting anything: it sets the spin budget of the following runs on this
 * handle and makes ONE wait impossible to complete,
 *   ILRE_SELFTEST_GRID_BARRIER      the grid barrier of the Algorithm 1 kernel waits for one
 *                                   CTA more than the grid has;
 *   ILRE_SELFTEST_MISSING_KEY_TILE  the TMA producer of the row-statistics kernel leaves out
 *                                   the last key tile of every CTA, so the tensor-core thread
 *                                   waits for a tile that never arrives;
 *   ILRE_SELFTEST_OFF               normal operation.
 * wait_cycle_limit is the spin budget in SM clock cycles (0 = the default of 2^31, about a
 * second).  The outputs of a run with an injected failure are unspecified; after
 * ilre_recall_selftest_wait(h, 0, ILRE_SELFTEST_OFF) the handle works as before.  The paper
 * has no counterpart; host-side, changes only the handle.
 */
#define ILRE_SELFTEST_OFF 0
#define ILRE_SELFTEST_GRID_BARRIER 1
#define ILRE_SELFTEST_MISSING_KEY_TILE 2
int ilre_recall_selftest_wait(ilre_recall_t* h, int64_t wait_cycle_limit, int32_t what);

/* Debugging aid (the paper has no counterpart): every workspace buffer of the handle is followed
 * by a 256-byte guard zone filled with a pattern when the handle is created; no kernel may write
 * there.  Waits for the device to go idle, reads the zones back and returns how many of them no
 * longer hold the pattern (0 = none: no kernel of any call so far wrote past the end of a
 * workspace buffer), or a negative ILRE_ERR_* code (a null handle: ILRE_ERR_INVALID_ARG).  Host
 * call; synchronises; meant for tests, not for the hot path. */
int ilre_recall_check_guards(ilre_recall_t* h);

/* Number of kernel launches issued by the last run(). */
int ilre_recall_last_launch_count(ilre_recall_t* h);

int ilre_recall_destroy(ilre_recall_t* h);

/*
 * Top-k of a score array without any allocation (the paper has no counterpart: this is a
 * convenience for callers that are not allowed to allocate device memory, e.g. code running
 * under a framework-owned memory pool or in a thread that must not hit cudaMalloc's implicit
 * synchronisation).  No handle is needed.  Returns the k positions with the highest scores,
 * equal scores ranked by lower position, as ascending int32 positions -- what
 * ilre_recall_run returns for one max kernel of size 1, one window of size 1 and no sink.
 *   scores_dev   fp32 [L] on the CURRENT device; 1 <= L <= ILRE_NOALLOC_MAX_L; no NaNs
 *                (-0.0 and +0.0 count as equal; a NaN would rank by its bit pattern)
 *   out_idx_dev  int32 [k] on the current device; 0 <= k <= L
 * Larger L is rejected with ILRE_ERR_CAPACITY, k > L with ILRE_ERR_BUDGET; nothing is launched
 * then.  The call is asynchronous on cuda_stream and calls no cudaMalloc/cudaFree.  Its scratch
 * (a bitmap of ILRE_NOALLOC_MAX_L bits = 128 KiB) is a fixed __device__ array inside the
 * library, resident on every GPU that loads the library until the process exits, and SHARED
 * by all calls: two calls that overlap on the same GPU (different streams or threads) race;
 * serialise them.  The first call on each device looks the array's address up (this may load
 * the library's device code), so make that first call before starting any stream capture.
 */
#define ILRE_NOALLOC_MAX_L 1048576
int ilre_topk_positions_noalloc(const float* scores_dev, int64_t L, int32_t k,
                                int32_t* out_idx_dev, void* cuda_stream);

const char* ilre_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ILRE_RECALL_H_ */
