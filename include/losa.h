/*
 * losa.h — C ABI of the LoSA per-denoising-step attention hot path (sm_100a).
 *
 * LoSA (locality-aware sparse attention for block-wise diffusion language models) runs, for every
 * attention layer and every denoising step of a block of B tokens, the workflow of the paper's
 * method-overview figure (Section 4):
 *
 *   (1) losa_select_active      per-token change of the queries since the previous step (Eq. 1,
 *                               Section 3.2); the m tokens that changed most are "active", the rest
 *                               "stable" (Section 4.1).
 *   (2) losa_page_scores_topk   QUEST page selection (Section 2.3) for the active queries only:
 *                               an upper bound of q.k per page from per-page min/max keys, top-k
 *                               pages per (token, query head) (Section 4.2).
 *   (3) losa_page_union         one deduplicated page list per (sequence, KV head): the union of
 *                               Section 4.2 / 4.4, which is what bounds the "KV Inflation" of
 *                               Section 3.1.
 *   (4) losa_sparse_prefix_attn prefix attention statistics (o_p, L_p) of Section 2.2 for the
 *                               active tokens over the union; stable tokens keep their cached
 *                               statistics (reuse rule / update rule, Section 4.2).  With every
 *                               token active and every page listed this is the dense first step
 *                               ("Initialization Workflow", Section 4.2).
 *   (5) losa_block_attn_merge   dense bidirectional attention inside the block and the
 *                               online-softmax merge with the prefix part (Section 4.3).
 *   (6) losa_update_prefix_cache keep the queries for the next step's Eq. 1 (Section 4.3); when a
 *                               block is finalised, append its K/V to the paged prefix cache
 *                               (Section 2.1) and refresh the page summaries (Section 2.3).
 *
 * Conventions
 *   - Every pointer named below is a DEVICE pointer unless it is a struct passed by address, a
 *     `losa_ctx*`, an `out` size, or explicitly marked "host".  The library never allocates device
 *     memory: the caller owns every buffer, including the workspace, and keeps it alive until the
 *     work enqueued on the stream has completed.
 *   - Every call validates its arguments on the host first and launches nothing when it fails.
 *   - Every call is asynchronous on the CUDA stream passed as `void* stream` (a `cudaStream_t`;
 *     NULL is the legacy default stream).  Per-step quantities (number of active tokens, prefix
 *     lengths, union sizes, step counters) live in device memory and are never read back, so a
 *     sequence of calls has a fixed launch configuration for a given context.
 *   - Kernels never trap.  A kernel that meets an out-of-range index or gives up on a bounded wait
 *     records LOSA_ERR_BOUNDS / LOSA_ERR_TIMEOUT in a device status word, skips the access and
 *     returns; losa_poll_status() reads that word.
 *   - Index conventions: tokens are 0-based inside the block; pages are LOGICAL page numbers,
 *     0-based inside a sequence (page p holds prefix tokens p*g .. p*g+g-1); `page_table` maps them
 *     to physical pages of the shared pool.  Padding entries of index lists are -1.
 *   - Element type `dtype` applies to Q, K, V, the page summaries, the Eq. 1 input and the final
 *     output.  The cached statistics (o_p, L_p), page scores, Delta and every LSE are fp32; index
 *     arrays are int32.  L_p and the merged LSE are natural logarithms of the sum of
 *     exp(sm_scale * q.k) (Section 2.2 with sm_scale = 1/sqrt(d)).
 *   - Supported shapes: head_dim in {64, 128}; page_size in {16, 32, 64}; block_size 1..64;
 *     n_q_heads a multiple of n_kv_heads with at most 16 query heads per KV head; device pointers
 *     16-byte aligned.  Anything else returns LOSA_ERR_UNSUPPORTED.
 */
#ifndef LOSA_H_
#define LOSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LOSA_OK                 0
#define LOSA_ERR_INVALID_ARG   -1   /* null pointer, bad enum, size out of range                 */
#define LOSA_ERR_UNSUPPORTED   -2   /* shape / dtype / stride / alignment the kernels do not cover */
#define LOSA_ERR_CUDA          -3   /* a CUDA runtime or driver call failed; see losa_last_cuda_error */
#define LOSA_ERR_TIMEOUT       -4   /* device: a bounded wait ran out (reported by losa_poll_status) */
#define LOSA_ERR_BOUNDS        -5   /* device: an index outside its range was met and skipped     */

#define LOSA_F32   0
#define LOSA_BF16  1

#define LOSA_KV_NATIVE    0
#define LOSA_KV_FP8_E4M3  1

#define LOSA_MAX_BLOCK 64

/* Problem shape of one attention layer (Section 2.1): B block tokens attend to a paged prefix. */
typedef struct {
  int32_t batch;              /* N  sequences handled by one call                               */
  int32_t n_q_heads;          /* H_q                                                            */
  int32_t n_kv_heads;         /* H_kv (grouped-query attention: G = H_q / H_kv heads per KV head) */
  int32_t head_dim;           /* d                                                              */
  int32_t block_size;         /* B  tokens of the block being denoised                          */
  int32_t page_size;          /* g  tokens per KV page (Section 2.3)                             */
  int32_t max_pages_per_seq;  /* P_max: row length of page_table and of union_pages             */
  int32_t dtype;              /* LOSA_F32 or LOSA_BF16                                          */
  float   sm_scale;           /* score scale, 1/sqrt(d) in Section 2.2                           */
} losa_shape_t;

/* Paged prefix KV cache K_p, V_p of Section 2.1 plus the per-page min/max keys of Section 2.3.
 * The struct itself lives in host memory and is read during the call; the pointers are device. */
typedef struct {
  void*          k_pages;      /* [n_phys_pages, H_kv, g, d] elements, strides below             */
  void*          v_pages;      /* same layout and strides as k_pages                             */
  int64_t        stride_page;  /* in elements; byte strides must be multiples of 16              */
  int64_t        stride_head;  /* in elements                                                    */
  int64_t        stride_tok;   /* in elements; the d elements of one token are contiguous        */
  void*          kmin;         /* [n_phys_pages, H_kv, d] element-wise min key of each page      */
  void*          kmax;         /* [n_phys_pages, H_kv, d] element-wise max key of each page      */
  const int32_t* page_table;   /* [N, P_max] physical page of each logical page                  */
  int32_t*       kv_len;       /* [N] prefix tokens L_s of each sequence                         */
  int32_t        n_phys_pages; /* pages in the pool                                              */
  int32_t        kv_format;    /* LOSA_KV_NATIVE: k_pages / v_pages hold `dtype` elements;       */
                               /* LOSA_KV_FP8_E4M3: one byte per element (strides in bytes) and  */
                               /* the scales below; summaries stay `dtype` (bf16 contexts only)  */
  float*         k_scale;      /* [n_phys_pages, H_kv] power-of-two scale of each key page       */
  float*         v_scale;      /* [n_phys_pages, H_kv] likewise for the values; NULL when native */
} losa_kv_t;

/* Per-block LoSA cache (Section 4.3 / "Memory overhead" in Section 4.5): B(d+1) scalars per head
 * and sequence, plus the previous step's queries and a step counter. Host struct, device pointers. */
#define LOSA_STATE_F32  0
#define LOSA_STATE_BF16 1
typedef struct {
  void*    q_prev;  /* [N, B, H_q, d] queries of the previous step (dtype)                       */
  void*    o_p;     /* [N, B, H_q, d] cached prefix attention output: fp32, or bf16 (o_p_format)  */
  float*   lse_p;   /* [N, B, H_q]    cached prefix log-normaliser L_p (fp32)                     */
  int32_t* step;    /* [N] denoising steps done for the current block; 0 = no valid cache        */
  int32_t  o_p_format;  /* LOSA_STATE_F32 (0, the default) or LOSA_STATE_BF16: o_p is STORED rounded to
                           bf16 (ties to even) and every use - the merge of the same step, the reuse in
                           later steps - sees the stored value (the paper quotes this cache in FP16,
                           Section 4.5); bf16 contexts only                                       */
} losa_state_t;

typedef struct losa_ctx losa_ctx;

/* Size in bytes of the device workspace a context of this shape needs (page-score scratch,
 * split-KV partial results, counters, the status word).  Host-only; `out` is a host pointer. */
int32_t losa_workspace_bytes(const losa_shape_t* shape, size_t* out);

/* Creates a context (host memory only) bound to a caller-owned, 256-byte aligned device workspace
 * of at least losa_workspace_bytes() bytes on the current device.  Clears the workspace's counters
 * and status word with a synchronous memset.  A context serves one stream at a time. */
int32_t losa_create(const losa_shape_t* shape, void* workspace, size_t workspace_bytes, losa_ctx** out);

/* Frees the context's host memory.  The workspace stays the caller's. */
int32_t losa_destroy(losa_ctx* ctx);

/* Synchronises `stream`, then returns the first device-side error recorded since the last poll
 * (LOSA_ERR_TIMEOUT or LOSA_ERR_BOUNDS) and clears it, or LOSA_OK. */
int32_t losa_poll_status(losa_ctx* ctx, void* stream);

/* Bound of the waits inside the bf16 stage-4 kernel (its warps hand work to one another through
 * shared-memory barriers), in SM clock cycles; `cycles` <= 0 restores the default of about one
 * second.  A wait that outlasts the bound makes its thread block record LOSA_ERR_TIMEOUT, wait
 * (again within a bound) for the page copies and tensor-core instructions it had already started,
 * release its tensor memory and return: the launch ends normally, the step's results are
 * meaningless, and the context stays usable.  A bound of a few cycles makes every launch end this
 * way, which is how the path is exercised without starving any barrier.  Host-side switch; takes
 * effect for calls issued after it returns (a captured graph keeps the bound it was captured with). */
int32_t losa_set_wait_limit(losa_ctx* ctx, int64_t cycles);

/* The CUDA error code (cudaError_t or CUresult value) behind the last LOSA_ERR_CUDA, else 0. */
int32_t losa_last_cuda_error(const losa_ctx* ctx);

/* Number of kernels this context has launched so far (host counter, for accounting). */
int64_t losa_launch_count(const losa_ctx* ctx);

/* Timing aid.  With `enable` != 0 every later losa_sparse_prefix_attn records a pair of CUDA events
 * (owned by the context) on its stream immediately before and after its main kernel — not around
 * the small combine kernel that follows.  losa_stage4_last_ms waits for the second event and
 * returns the time between the two in milliseconds (host pointer).  Do not enable while a stream
 * capture is in progress. */
int32_t losa_profile_stage4(losa_ctx* ctx, int32_t enable);
int32_t losa_stage4_last_ms(losa_ctx* ctx, float* out_ms);

/* Stage 1 — locality score and locality pruning (Eq. 1 in Section 3.2; Section 4.1).
 *   x_cur, x_prev [N, B, row_width] (dtype): the representation whose change is measured, this
 *       step's and the previous step's (queries flattened over heads: row_width = H_q*d; hidden
 *       states of any width that is a multiple of 8 work as well).
 *   Delta[s,i] = mean_c (x_cur[s,i,c] - x_prev[s,i,c])^2, accumulated in fp64.
 *   m_per_seq [N] int32 or NULL: how many tokens to keep active; NULL or a negative entry means
 *       all B; values above B are clamped.
 *   step [N] int32 or NULL: where step[s] == 0 (first step of a block, no cache) all B tokens are
 *       active whatever m says.
 *   active_idx [N, B] int32 out: the active tokens of each sequence in ascending order, then -1.
 *       The m tokens with the largest Delta are chosen; equal Delta goes to the lower token index.
 *   n_active [N] int32 out.   delta_opt [N, B] fp32 out or NULL.
 *   Inputs must be finite.  A Delta that is NaN (NaN or opposite infinities in a row) is ranked as
 *   +inf, so that the ranking stays a total order and n_active never exceeds m; what the definition
 *   would select in that case is left open. */
int32_t losa_select_active(losa_ctx* ctx, const void* x_cur, const void* x_prev, int32_t row_width,
                           const int32_t* m_per_seq, const int32_t* step, int32_t* active_idx,
                           int32_t* n_active, float* delta_opt, void* stream);

/* Stage 1, threshold variant (the rule behind the appendix's locality heat maps, which mark the
 * tokens that carry half of a layer's total change: tau = 0.5).  Delta and the ranking are those of
 * losa_select_active; the active set is the shortest leading part of the ranking whose Delta add up
 * to at least tau times the sum of Delta over the block (both sums taken over the ranking in order,
 * in fp64).  A block whose queries did not change at all has no active token.
 *   tau in (0, 1] (host value); anything else returns LOSA_ERR_INVALID_ARG.
 *   m_cap_opt [N] int32 or NULL: an upper bound on the count per sequence (negative = none).
 *   step[s] == 0 makes every token of sequence s active, as in losa_select_active.
 *   All other arguments and outputs are those of losa_select_active. */
int32_t losa_select_active_tau(losa_ctx* ctx, const void* x_cur, const void* x_prev, int32_t row_width,
                               double tau, const int32_t* m_cap_opt, const int32_t* step, int32_t* active_idx,
                               int32_t* n_active, float* delta_opt, void* stream);

/* Stage 1 without any allocation (the paper has no counterpart; this is a deployment aid).
 * Some programs that embed this library are not allowed to obtain device memory once they are
 * running: an inference server whose memory pool was carved up at start-up and whose allocator is
 * owned by the host framework, a plug-in running under a fixed memory budget, or code on a path
 * where cudaMalloc's implicit device-wide synchronisation is unacceptable.  Such callers cannot
 * provide the workspace a context needs.  For them this entry point runs stage 1 exactly as
 * losa_select_active does, but keeps its scratch (one fp64 score per block token and one counter
 * per sequence) in a fixed array inside the library image instead of a caller workspace.  It needs
 * no context, and it calls no cudaMalloc, cudaFree or other allocating routine.
 *   shape: only batch, block_size and dtype are read.  batch must be at most 64 (the size the fixed
 *       array was built for); a larger batch returns LOSA_ERR_UNSUPPORTED and launches nothing.
 *   All other arguments, outputs and tie rules are those of losa_select_active.
 *   The array costs about 33 KB on every GPU that loads the library, for the life of the process.
 *   The first call on a device looks up the array's device address (once per device, with that
 *   device current); make that first call before starting any stream capture.
 *   All calls on a device share the one array, which keeps the previous call's contents (this call
 *   clears the counters it relies on).  Two calls that overlap on the GPU — different streams, or
 *   different host threads without ordering between their streams — race on it: serialise them. */
int32_t losa_select_active_static(const losa_shape_t* shape, const void* x_cur, const void* x_prev,
                                  int32_t row_width, const int32_t* m_per_seq, const int32_t* step,
                                  int32_t* active_idx, int32_t* n_active, float* delta_opt,
                                  void* stream);

/* Stage 2 — QUEST page scores and top-k for the active queries (Section 2.3; Section 4.2).
 *   q [N, B, H_q, d] (dtype).  For every active token i, query head h and logical page p < P_s
 *   (P_s = ceil(L_s / g)), with kappa = h / G:
 *       U(p) = sum_j max(q_j * kmin[p,kappa,j], q_j * kmax[p,kappa,j])
 *            = sum_j (max(q_j, 0) * kmax[p,kappa,j] + min(q_j, 0) * kmin[p,kappa,j])     (kmin <= kmax)
 *   evaluated in fp32 in a fixed order, because it decides integer page ids: for each run of 8
 *   consecutive j an accumulator starts at +0 and takes, j ascending, first
 *   acc = fma(max(q_j,0), kmax_j, acc), then acc = fma(min(q_j,0), kmin_j, acc) (fused, round to
 *   nearest); the d/8 run sums are combined by the butterfly c[i] <- c[i] + c[i xor off],
 *   off = d/16 .. 1; finally + 0.0f.
 *   topk_pages [N, B, H_q, k] int32 out: the min(k, P_s) pages with the largest U, ordered by
 *       (U descending, page ascending), then -1.  Rows of stable tokens, and of sequences whose
 *       step[s] == 0 (their union is "all pages" anyway), are not written.
 *   topk_scores_opt [N, B, H_q, k] fp32 out or NULL: U of the listed pages (padding untouched).
 *   step [N] or NULL as in stage 1.  k >= 1 (pages, not tokens). */
int32_t losa_page_scores_topk(losa_ctx* ctx, const void* q, const losa_kv_t* kv,
                              const int32_t* active_idx, const int32_t* n_active,
                              const int32_t* step, int32_t k, int32_t* topk_pages,
                              float* topk_scores_opt, void* stream);

/* Stage 2, pooled selector — one list per (token, KV head) instead of one per query head.  The
 *   paper leaves the selector open (Section 2.3); with grouped-query attention the G heads of a KV
 *   head read the same pages, so this variant scores a page once per KV head: the pooled score is
 *   the largest of the G heads' U(p) (each evaluated exactly as above), the min(k, P_s) pages are
 *   taken by (pooled score descending, page ascending), and the list is stored for every head of
 *   the group, so topk_pages / topk_scores_opt keep the layout above and stage 3 is unchanged.  The
 *   union of a KV head then holds at most n_active * k pages instead of n_active * G * k.  With
 *   G = 1 the result is that of losa_page_scores_topk.  Same arguments and errors. */
int32_t losa_page_scores_topk_pooled(losa_ctx* ctx, const void* q, const losa_kv_t* kv,
                                     const int32_t* active_idx, const int32_t* n_active,
                                     const int32_t* step, int32_t k, int32_t* topk_pages,
                                     float* topk_scores_opt, void* stream);

/* Stage 2, tensor-core selector (bf16 only) - the page scores as one GEMM [q+ | q-] x [kmax | kmin] on
 *   the tensor cores, top-k on its fp32 results.  The paper calls its method independent of the
 *   selector (Section 2.3) and fixes no arithmetic; this variant gives up the fixed summation order of
 *   losa_page_scores_topk, so its lists are not comparable entry by entry.  What holds instead: a
 *   list has min(k, P_s) distinct pages of 0 .. P_s-1, then -1, and every listed page's score (in
 *   exact arithmetic) is at least the k-th largest exact score minus 2^-11 times the largest
 *   sum_j |t_j| over the pages (t_j the terms of U).  Lists are ordered by the tensor-core score
 *   (descending, page ascending); topk_scores_opt receives those scores.  Same arguments and errors;
 *   fp32 contexts return LOSA_ERR_UNSUPPORTED. */
int32_t losa_page_scores_topk_mma(losa_ctx* ctx, const void* q, const losa_kv_t* kv,
                                  const int32_t* active_idx, const int32_t* n_active,
                                  const int32_t* step, int32_t k, int32_t* topk_pages,
                                  float* topk_scores_opt, void* stream);

/* Selector used by losa_denoise_step / losa_denoise_step_host on this context: 0 (default) = one
 *   list per query head, non-zero = the pooled selector.  Host-side switch; takes effect for calls
 *   issued after it returns. */
int32_t losa_set_pooled_selection(losa_ctx* ctx, int32_t on);

/* Selector of stage 2 inside losa_denoise_step / losa_denoise_step_host, by name:
 *   LOSA_SELECTOR_EXACT  one list per query head in the fixed fp32 order (losa_page_scores_topk; default)
 *   LOSA_SELECTOR_POOLED one list per KV head (losa_page_scores_topk_pooled; the same as
 *                        losa_set_pooled_selection(ctx, 1))
 *   LOSA_SELECTOR_MMA    page scores as a GEMM on the tensor cores, lists valid under the relaxed rule
 *                        (losa_page_scores_topk_mma; bf16 contexts, else LOSA_ERR_UNSUPPORTED)
 * Host-only; LOSA_ERR_INVALID_ARG for another value. */
#define LOSA_SELECTOR_EXACT  0
#define LOSA_SELECTOR_POOLED 1
#define LOSA_SELECTOR_MMA    2
int32_t losa_set_step_selector(losa_ctx* ctx, int32_t selector);

/* Stage 3 — union of the selections (Section 4.2, Section 4.4).
 *   union_pages [N, H_kv, P_max] int32 out: for each sequence and KV head, the distinct logical
 *       pages selected by any active token through any of the G query heads of that KV head,
 *       ascending, then -1.   union_count [N, H_kv] int32 out.
 *   Where step[s] == 0 the list is every page 0 .. P_s-1 (dense first step, Section 4.2). */
int32_t losa_page_union(losa_ctx* ctx, const int32_t* topk_pages, const int32_t* active_idx,
                        const int32_t* n_active, int32_t k, const int32_t* kv_len,
                        const int32_t* step, int32_t* union_pages, int32_t* union_count,
                        void* stream);

/* Stage 4 — paged sparse prefix attention for the active tokens (Section 2.2; Section 4.2).
 *   For every active token i and head h, over the valid tokens t (t < L_s) of the pages listed
 *   for KV head h / G:  s_t = sm_scale * <q, k_t>;  L_p = log sum_t exp(s_t);
 *   o_p = sum_t exp(s_t - L_p) v_t.  Writes state->o_p and state->lse_p rows of active tokens
 *   only; rows of stable tokens are neither read nor written.  An empty list gives L_p = -inf,
 *   o_p = 0.  Uses the context's workspace for split-KV partial results. */
int32_t losa_sparse_prefix_attn(losa_ctx* ctx, const void* q, const losa_kv_t* kv,
                                const int32_t* active_idx, const int32_t* n_active,
                                const int32_t* union_pages, const int32_t* union_count,
                                losa_state_t* state, void* stream);

/* Stage 5 — dense in-block attention and the online-softmax merge (Section 4.3, Section 2.2).
 *   k_blk, v_blk [N, B, H_kv, d] (dtype): this step's block keys / values.  For every block token
 *   and head: (o_b, L_b) over the B block keys with no mask; L = log(e^{L_p} + e^{L_b});
 *   out = e^{L_p - L} o_p + e^{L_b - L} o_b.
 *   out [N, B, H_q, d] (dtype).   lse_out_opt [N, B, H_q] fp32 or NULL. */
int32_t losa_block_attn_merge(losa_ctx* ctx, const void* q, const void* k_blk, const void* v_blk,
                              const losa_state_t* state, void* out, float* lse_out_opt,
                              void* stream);

/* Stage 6 — cache maintenance (Section 4.3; Section 2.1).
 *   finalize_block == 0: q_prev <- q, step[s] += 1.
 *   finalize_block != 0: the block's k_blk, v_blk [N, B, H_kv, d] are written to prefix positions
 *       L_s .. L_s+B-1 through page_table (whose entries for those pages must already name free
 *       physical pages), kmin/kmax of every touched page are recomputed over its valid tokens,
 *       kv_len[s] += B and step[s] = 0, so that the next block starts with a dense first step. */
int32_t losa_update_prefix_cache(losa_ctx* ctx, losa_kv_t* kv, losa_state_t* state, const void* q,
                                 const void* k_blk, const void* v_blk, int32_t finalize_block,
                                 void* stream);

/* FP8 K/V pages (bf16 contexts) — an extension of the cache format; the paper names quantised
 * attention as orthogonal to the method (Section 6) and quotes the cached state in FP16
 * (Section 4.5, "Memory overhead").  A cache with kv_format = LOSA_KV_FP8_E4M3 stores every K / V
 * element as one E4M3 byte (largest finite value 448) and one scale per (physical page, KV head) and
 * tensor:  amax = largest |x| over the page's valid tokens;  scale = 2^e with e the smallest integer
 * such that amax <= 448 * 2^e, clamped to [-6, 7];  code = round-to-nearest-even of x / scale,
 * saturated at +-448;  the value every stage works with is scale * value(code) (exact in bf16 and
 * fp16).  Slots of a page past the prefix's end hold code 0.  Stage 4 streams half the bytes; its
 * arithmetic is that of the bf16 path on the dequantised values (fp16 operands, fp32 accumulation),
 * so its results are held to the bf16 tolerances against the definition evaluated on the
 * dequantised cache.  Stages 2, 3, 5 are unchanged (the summaries are those of the dequantised
 * keys); block finalisation re-quantises every touched page from its dequantised old rows and the
 * new rows together.  Inputs must satisfy |x| <= 448 * 2^7 (larger magnitudes saturate).
 *
 * losa_quantize_kv_pages: src is a native bf16 cache, dst an FP8 cache with the same page_table,
 *   kv_len and n_phys_pages; writes dst's codes and scales for every logical page p < P_s of every
 *   sequence and dst's kmin / kmax. */
int32_t losa_quantize_kv_pages(losa_ctx* ctx, const losa_kv_t* src, losa_kv_t* dst, void* stream);

/* Set-up helper — per-page min/max keys of Section 2.3 for the whole prefix: kmin/kmax of every
 * logical page p < P_s over its valid tokens. */
int32_t losa_build_page_summaries(losa_ctx* ctx, losa_kv_t* kv, void* stream);

/* Device buffers a whole-step call needs besides its inputs and outputs (caller-owned). */
typedef struct {
  void *d_q, *d_k_blk, *d_v_blk, *d_out;  /* staging of the host variant; unused by losa_denoise_step */
  int32_t *active_idx, *n_active;      /* [N,B], [N]                     */
  int32_t *topk_pages;                 /* [N,B,H_q,k]                    */
  int32_t *union_pages, *union_count;  /* [N,H_kv,P_max], [N,H_kv]       */
} losa_step_buffers_t;

/* One whole layer-step (the method-overview workflow of Section 4, stages 1-6 with
 * finalize_block = 0) in one call, with the same results as the six calls in order: the index
 * buffers of `buf` receive what stages 1-3 produce, state->o_p / lse_p what stage 4 produces,
 * out / lse_out_opt what stage 5 produces; q_prev and step are updated as by stage 6.
 * Being one call, it may schedule freely inside: the in-block attention of stage 5 (which needs
 * nothing from stages 1-4) runs on a second stream owned by the context and is joined before a
 * final merge kernel that also keeps the queries; where stage 2 runs the candidate refinement
 * (bf16, k <= 512) that kernel also writes stage 3's union.  All work is ordered after prior work on
 * `stream` and complete when `stream` reaches the end of the call's work; the call can be captured
 * in a CUDA graph after one un-captured call on the context (which creates the second stream). */
int32_t losa_denoise_step(losa_ctx* ctx, const void* q, const void* k_blk, const void* v_blk, void* out,
                          float* lse_out_opt, losa_kv_t* kv, losa_state_t* state,
                          const losa_step_buffers_t* buf, const int32_t* m_per_seq, int32_t k,
                          void* stream);

/* The same whole layer-step from HOST buffers: copies q, k_blk, v_blk [dtype] from host memory to
 * the device staging buffers d_q, d_k_blk, d_v_blk of `buf`, runs losa_denoise_step on them with
 * d_out as output, and copies d_out back to the host buffer h_out.  Does not synchronise.  All
 * h_* pointers are HOST pointers (pinned for true asynchrony); everything else is device memory
 * owned by the caller.  m_per_seq as in stage 1; k as in stage 2. */
int32_t losa_denoise_step_host(losa_ctx* ctx, const void* h_q, const void* h_k_blk,
                               const void* h_v_blk, void* h_out, losa_kv_t* kv, losa_state_t* state,
                               const losa_step_buffers_t* buf, const int32_t* m_per_seq, int32_t k,
                               void* stream);

#ifdef __cplusplus
}
#endif
#endif  /* LOSA_H_ */
