// Host-side launchers of the stage kernels.  Each enqueues on `st`, validates nothing (the C-ABI
// layer in api.cu has done so) and returns LOSA_OK or LOSA_ERR_CUDA.
#pragma once
#include "common.cuh"

namespace losa {

int32_t launch_select_active(losa_ctx* c, const void* x_cur, const void* x_prev, int32_t row_width,
                             const int32_t* m_per_seq, const int32_t* step, int32_t* active_idx,
                             int32_t* n_active, float* delta_opt, cudaStream_t st, double tau = 0.0,
                             int32_t* slot_map_opt = nullptr);

int32_t launch_page_scores_topk(losa_ctx* c, const void* q, const losa_kv_t* kv,
                                const int32_t* active_idx, const int32_t* n_active,
                                const int32_t* step, int32_t k, int32_t* topk_pages,
                                float* topk_scores_opt, cudaStream_t st, int selector = 0, bool after_stage1 = false,
                                int32_t* union_pages = nullptr, int32_t* union_count = nullptr, bool* union_done = nullptr);
// union_pages / union_count / union_done (all three or none): where the selection can also write stage 3's
// union (the bf16 candidate refinement, bitmaps of at most 256 words), it does so and sets *union_done;
// otherwise *union_done is false and the caller launches stage 3 itself.
// after_stage1: the kernel launched just before on `st` is stage 1 of the same step (see launch_page_bounds)
// selector: 0 = one exact list per query head, 1 = pooled over the heads of a KV head, 2 = tensor-core scores (relaxed rule, bf16)
constexpr int kSelectorExact = 0, kSelectorPooled = 1, kSelectorMma = 2;

// Stage 2, first half: fp32 page scores of the active queries into the workspace's score rows.
int32_t launch_page_scores(losa_ctx* c, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                           const int32_t* n_active, const int32_t* step, cudaStream_t st);

// bf16: (lower, upper) bounds of the page scores from the tensor cores, as float2 per (row, page), for
// the selection that evaluates the exact score of the surviving candidates only.
// With approx_only the tensor-core value itself is written as an fp32 score row (relaxed selector).
int32_t launch_page_bounds(losa_ctx* c, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                           const int32_t* n_active, const int32_t* step, cudaStream_t st, bool approx_only = false,
                           bool after_stage1 = false);
// after_stage1: the previous kernel on `st` is stage 1 of the same step, which releases its dependents only
// after everything before it has completed: the kernel then takes its work list and first copies (kv_len,
// step, page table, summaries - nothing stage 1 writes) before stage 1 ends.

int32_t launch_page_union(losa_ctx* c, const int32_t* topk_pages, const int32_t* active_idx,
                          const int32_t* n_active, int32_t k, const int32_t* kv_len,
                          const int32_t* step, int32_t* union_pages, int32_t* union_count,
                          cudaStream_t st);

int32_t launch_sparse_prefix_attn(losa_ctx* c, const void* q, const losa_kv_t* kv,
                                  const int32_t* active_idx, const int32_t* n_active,
                                  const int32_t* union_pages, const int32_t* union_count,
                                  losa_state_t* state, cudaStream_t st, bool defer_combine = false);
// Whole-step path: with defer_combine the bf16 main kernel leaves its partial records unmerged and
// launch_attn_finish merges them, merges with the in-block part, writes the output, keeps the
// queries and bumps the step (one kernel instead of combine + merge_commit).
bool finish_fuses_combine(const losa_ctx* c);
int32_t launch_attn_finish(losa_ctx* c, const void* q, const int32_t* active_idx, const int32_t* n_active, const int32_t* slot_map,
                           losa_state_t* state, void* out, float* lse_out_opt, cudaStream_t st);

int32_t launch_block_attn_merge(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk,
                                const losa_state_t* state, void* out, float* lse_out_opt,
                                cudaStream_t st);

// Whole-step path: in-block attention alone (o_b, L_b into the workspace), then merge with the
// prefix statistics, write the output, keep the queries and bump the step counters.
int32_t launch_block_attn(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk, cudaStream_t st);
int32_t launch_merge_commit(losa_ctx* c, const void* q, losa_state_t* state, void* out, float* lse_out_opt,
                            cudaStream_t st);

int32_t launch_update_prefix_cache(losa_ctx* c, losa_kv_t* kv, losa_state_t* state, const void* q,
                                   const void* k_blk, const void* v_blk, int32_t finalize_block,
                                   cudaStream_t st);

int32_t launch_build_page_summaries(losa_ctx* c, losa_kv_t* kv, cudaStream_t st);

// FP8 (E4M3) K/V pages, one power-of-two scale per (physical page, KV head) and tensor (bf16 contexts):
// quantise a bf16 pool page by page (codes, scales, summaries of the dequantised keys); summaries of
// an FP8 pool; block append with re-quantisation of the touched pages.
int32_t launch_fp8_quantize(losa_ctx* c, const losa_kv_t* src, losa_kv_t* dst, cudaStream_t st);
int32_t launch_fp8_summaries(losa_ctx* c, losa_kv_t* kv, cudaStream_t st);
int32_t launch_fp8_append(losa_ctx* c, losa_kv_t* kv, const void* k_blk, const void* v_blk, cudaStream_t st);

// Largest k and page count the top-k kernel's shared memory allows for this context.
int32_t topk_max_sortable(const losa_ctx* c);

}  // namespace losa
