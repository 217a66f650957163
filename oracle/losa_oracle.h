/*
 * losa_oracle.h — CPU oracle of the LoSA per-denoising-step attention path.
 *
 * TEST INFRASTRUCTURE, not product code: a plain, slow, step-by-step restatement of what the
 * paper defines, in fp64 (page scores additionally in the fixed fp32 order the library's interface
 * states, because that arithmetic decides integer page ids).  Nothing here is shared with the CUDA
 * library; only tests, the smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * All pointers are HOST pointers.  Element buffers hold either fp32 or bf16 bit patterns
 * (dtype 0 / 1), in the same layouts the library's interface uses, so that both sides can be fed
 * the same bytes.  State (o_p, L_p) and outputs are fp64.
 *
 * Pins (tests/test_oracle_*.py): brute-force dense softmax attention when every token is active
 * and every page selected; LSE merge vs softmax over the concatenation; bit-exact reuse for stable
 * tokens; page-score upper-bound property and its reduction to exact top-k keys at page size 1;
 * union-size inequalities; invariance under physical page permutation; the threshold rule and the
 * pooled selector each by a worked example with exact arithmetic and a numpy re-derivation.  No
 * function here is "parity unpinned".
 */
#ifndef LOSA_ORACLE_H_
#define LOSA_ORACLE_H_
#include <stdint.h>

typedef struct {
  int32_t batch, n_q_heads, n_kv_heads, head_dim, block_size, page_size, max_pages_per_seq, dtype;
  double  sm_scale;
} oracle_shape_t;

typedef struct {
  void *k_pages, *v_pages;                       /* [n_phys, H_kv, g, d], strides in elements */
  int64_t stride_page, stride_head, stride_tok;
  void *kmin, *kmax;                             /* [n_phys, H_kv, d] */
  const int32_t* page_table;                     /* [N, P_max] */
  int32_t* kv_len;                               /* [N] */
} oracle_kv_t;

int oracle_num_threads(void);

/* Section 2.3: element-wise min / max key of every logical page over its valid tokens. */
void oracle_build_page_summaries(const oracle_shape_t* sh, oracle_kv_t* kv);

/* Eq. 1 (Section 3.2) + Section 4.1. */
void oracle_select_active(const oracle_shape_t* sh, const void* x_cur, const void* x_prev,
                          int32_t row_width, const int32_t* m_per_seq, const int32_t* step,
                          int32_t* active_idx, int32_t* n_active, double* delta);

/* Threshold variant (appendix figures, tau = 0.5): the shortest leading part of the ranking whose
 * Delta add up to at least tau times the block's total; m_cap (optional, per sequence) bounds it. */
void oracle_select_active_tau(const oracle_shape_t* sh, const void* x_cur, const void* x_prev,
                              int32_t row_width, double tau, const int32_t* m_cap, const int32_t* step,
                              int32_t* active_idx, int32_t* n_active, double* delta);

/* Section 2.3 page upper bound for one (sequence, token, head): fp32 in the interface's fixed
 * order (u32, may be NULL) and plain fp64 (u64, may be NULL); P_s entries each. */
void oracle_page_scores_one(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                            int32_t s, int32_t tok, int32_t head, float* u32, double* u64);

/* Section 2.3 / 4.2: top-k pages per active (token, head). */
void oracle_page_scores_topk(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                             const int32_t* active_idx, const int32_t* n_active,
                             const int32_t* step, int32_t k, int32_t* topk_pages,
                             float* topk_scores);

/* Selector variant for grouped-query attention: a page's pooled score is the largest of the upper
 * bounds of the G heads of its KV head; one top-k list per (token, KV head), stored for every head
 * of the group (same layout as above).  Not in the paper, which leaves the selector open
 * (Section 2.3). */
void oracle_page_scores_topk_pooled(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                                    const int32_t* active_idx, const int32_t* n_active,
                                    const int32_t* step, int32_t k, int32_t* topk_pages,
                                    float* topk_scores);

/* Section 4.2 / 4.4: union per (sequence, KV head). */
/* FP8 (E4M3) K/V pages with one power-of-two scale per (physical page, KV head) and tensor; see the
 * definition in losa_oracle.c.  codes: [n_phys, H_kv, g, d] bytes; scales: [n_phys, H_kv] fp32. */
double oracle_fp8_decode(uint8_t code);
uint8_t oracle_fp8_encode(double y);
void oracle_fp8_quantize_pages(const oracle_shape_t* sh, const oracle_kv_t* src, uint8_t* k_codes, uint8_t* v_codes,
                               float* k_scale, float* v_scale);
void oracle_fp8_dequantize_pages(const oracle_shape_t* sh, const uint8_t* k_codes, const uint8_t* v_codes,
                                 const float* k_scale, const float* v_scale, oracle_kv_t* dst);
void oracle_fp8_append_block(const oracle_shape_t* sh, const int32_t* page_table, int32_t* kv_len,
                             uint8_t* k_codes, uint8_t* v_codes, float* k_scale, float* v_scale,
                             const void* k_blk, const void* v_blk);

/* bf16 state (extension; Section 4.5 quotes the cache in FP16): o_p is stored rounded to bf16 (ties to
 * even), L_p unchanged.  Rounds the rows of the active tokens in place. */
double oracle_round_bf16(double x);
void oracle_round_state_bf16(const oracle_shape_t* sh, double* o_p, const int32_t* active_idx,
                             const int32_t* n_active);

/* Relaxed validity of page lists produced with another arithmetic than the fixed fp32 order: number of
 * (active token, head) lists that are not "min(k, P) distinct in-range pages, each with fp64 bound >=
 * the k-th largest fp64 bound - eps * (largest sum of term magnitudes)", then -1 padding. */
int64_t oracle_check_topk_relaxed(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                                  const int32_t* active_idx, const int32_t* n_active,
                                  const int32_t* step, int32_t k, const int32_t* topk_pages, double eps);

void oracle_page_union(const oracle_shape_t* sh, const int32_t* topk_pages,
                       const int32_t* active_idx, const int32_t* n_active, int32_t k,
                       const int32_t* kv_len, const int32_t* step, int32_t* union_pages,
                       int32_t* union_count);

/* Section 2.2 prefix statistics over the union for active tokens; others untouched (Section 4.2). */
void oracle_sparse_prefix_attn(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                               const int32_t* active_idx, const int32_t* n_active,
                               const int32_t* union_pages, const int32_t* union_count,
                               double* o_p, double* lse_p);

/* Section 4.3: dense in-block attention and the merge with (o_p, L_p). */
void oracle_block_attn_merge(const oracle_shape_t* sh, const void* q, const void* k_blk,
                             const void* v_blk, const double* o_p, const double* lse_p,
                             double* out, double* lse_out);

/* Section 4.3 / 2.1: keep queries; on finalise append the block's K/V and refresh summaries. */
void oracle_update_prefix_cache(const oracle_shape_t* sh, oracle_kv_t* kv, void* q_prev,
                                int32_t* step, const void* q, const void* k_blk,
                                const void* v_blk, int32_t finalize_block);

#endif
