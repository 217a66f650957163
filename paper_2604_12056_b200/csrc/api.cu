// C-ABI layer of the LoSA library: argument validation, context and workspace bookkeeping.
// Every entry point validates on the host and launches nothing when validation fails.
#include <cstdlib>
#include <cstring>
#include <new>

#include "kernels.h"

using namespace losa;

namespace {

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int32_t check_shape(const losa_shape_t* sh) {
  if (!sh) return LOSA_ERR_INVALID_ARG;
  if (sh->batch < 1 || sh->batch > 1024 || sh->n_q_heads < 1 || sh->n_kv_heads < 1 || sh->head_dim < 1 ||
      sh->block_size < 1 || sh->block_size > LOSA_MAX_BLOCK || sh->page_size < 1 ||
      sh->max_pages_per_seq < 0 || !(sh->sm_scale > 0.f))
    return LOSA_ERR_INVALID_ARG;
  if (sh->dtype != LOSA_F32 && sh->dtype != LOSA_BF16) return LOSA_ERR_INVALID_ARG;
  if (sh->head_dim != 64 && sh->head_dim != 128) return LOSA_ERR_UNSUPPORTED;
  if (sh->page_size != 16 && sh->page_size != 32 && sh->page_size != 64) return LOSA_ERR_UNSUPPORTED;
  if (sh->n_q_heads % sh->n_kv_heads != 0 || sh->n_q_heads / sh->n_kv_heads > 16) return LOSA_ERR_UNSUPPORTED;
  return LOSA_OK;
}

int32_t make_layout(const losa_shape_t* sh, int n_ctas, WorkspaceLayout* L) {
  const int G = sh->n_q_heads / sh->n_kv_heads;
  L->n_row_groups = (sh->block_size * G + kRowsPerGroup - 1) / kRowsPerGroup;
  L->n_segments = sh->batch * sh->n_kv_heads * L->n_row_groups;
  if (L->n_segments > kMaxSegments) return LOSA_ERR_UNSUPPORTED;
  L->n_ctas = n_ctas;
  L->n_slots = n_ctas + L->n_segments;
  L->score_stride = static_cast<int32_t>(align_up(static_cast<size_t>(sh->max_pages_per_seq > 0 ? sh->max_pages_per_seq : 1), 64));
  size_t off = 0;
  L->status = off;   off = align_up(off + 16, 256);
  L->counters = off; off = align_up(off + sizeof(uint32_t) * sh->batch, 256);
  L->seg_prefix = off; off = align_up(off + sizeof(int32_t) * (kMaxSegments + 1), 256);
  L->slot_map = off; off = align_up(off + sizeof(int32_t) * sh->batch * sh->block_size, 256);
  L->union_bits = off;
  off = align_up(off + sizeof(uint32_t) * static_cast<size_t>(sh->batch) * sh->n_kv_heads * ((sh->max_pages_per_seq + 31) / 32), 256);
  L->union_tickets = off; off = align_up(off + sizeof(uint32_t) * sh->batch * sh->n_kv_heads, 256);
  L->delta = off;    off = align_up(off + sizeof(double) * sh->batch * sh->block_size, 256);
  L->scores = off;
  off = align_up(off + 2 * sizeof(float) * static_cast<size_t>(sh->batch) * sh->block_size * sh->n_q_heads * L->score_stride, 256);
  L->partials = off;
  off = align_up(off + sizeof(float) * static_cast<size_t>(L->n_slots) * kRowsPerGroup * (sh->head_dim + 2), 256);
  const size_t rows = static_cast<size_t>(sh->batch) * sh->block_size * sh->n_q_heads;
  L->block_o = off;   off = align_up(off + sizeof(float) * rows * sh->head_dim, 256);
  L->block_lse = off; off = align_up(off + sizeof(float) * rows, 256);
  L->total = off;
  return LOSA_OK;
}

// Number of CTAs of the split-KV kernels: one per SM of the current device.  Without a device
// (size queries on a CPU-only host) the B200 count is assumed.
int current_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
    return n;
  (void)cudaGetLastError();
  return 148;
}

// The cached prefix output is fp32, or - in bf16 contexts - stored rounded to bf16.
int32_t check_state_format(const losa_ctx* c, const losa_state_t* st) {
  if (st->o_p_format != LOSA_STATE_F32 && st->o_p_format != LOSA_STATE_BF16) return LOSA_ERR_INVALID_ARG;
  if (st->o_p_format == LOSA_STATE_BF16 && c->shape.dtype != LOSA_BF16) return LOSA_ERR_UNSUPPORTED;
  return LOSA_OK;
}

int32_t check_kv(const losa_ctx* c, const losa_kv_t* kv, bool need_summaries) {
  if (!kv || !kv->k_pages || !kv->v_pages || !kv->page_table || !kv->kv_len) return LOSA_ERR_INVALID_ARG;
  if (need_summaries && (!kv->kmin || !kv->kmax)) return LOSA_ERR_INVALID_ARG;
  if (kv->n_phys_pages < 1) return LOSA_ERR_INVALID_ARG;
  const losa_shape_t& sh = c->shape;
  if (kv->kv_format != LOSA_KV_NATIVE && kv->kv_format != LOSA_KV_FP8_E4M3) return LOSA_ERR_INVALID_ARG;
  const bool fp8 = kv->kv_format == LOSA_KV_FP8_E4M3;
  if (fp8 && (!kv->k_scale || !kv->v_scale)) return LOSA_ERR_INVALID_ARG;
  if (fp8 && sh.dtype != LOSA_BF16) return LOSA_ERR_UNSUPPORTED;
  const int64_t es = fp8 ? 1 : (sh.dtype == LOSA_BF16 ? 2 : 4);
  if (kv->stride_tok < sh.head_dim || kv->stride_head < 1 || kv->stride_page < 1) return LOSA_ERR_INVALID_ARG;
  if ((kv->stride_tok * es) % 16 || (kv->stride_head * es) % 16 || (kv->stride_page * es) % 16) return LOSA_ERR_UNSUPPORTED;
  if (!aligned16(kv->k_pages) || !aligned16(kv->v_pages) || (kv->kmin && !aligned16(kv->kmin)) ||
      (kv->kmax && !aligned16(kv->kmax)))
    return LOSA_ERR_UNSUPPORTED;
  return LOSA_OK;
}

cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

}  // namespace

extern "C" {

int32_t losa_workspace_bytes(const losa_shape_t* shape, size_t* out) {
  if (!out) return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_shape(shape);
  if (rc != LOSA_OK) return rc;
  WorkspaceLayout L;
  rc = make_layout(shape, current_sm_count(), &L);
  if (rc != LOSA_OK) return rc;
  *out = L.total;
  return LOSA_OK;
}

int32_t losa_create(const losa_shape_t* shape, void* workspace, size_t workspace_bytes, losa_ctx** out) {
  if (!out) return LOSA_ERR_INVALID_ARG;
  *out = nullptr;
  int32_t rc = check_shape(shape);
  if (rc != LOSA_OK) return rc;
  if (!workspace) return LOSA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LOSA_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LOSA_ERR_CUDA;
  losa_ctx* c = new (std::nothrow) losa_ctx();
  if (!c) return LOSA_ERR_INVALID_ARG;
  std::memset(c, 0, sizeof(*c));
  c->shape = *shape;
  c->device = dev;
  c->ws = static_cast<char*>(workspace);
  cudaError_t e = cudaDeviceGetAttribute(&c->n_sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) { delete c; return LOSA_ERR_CUDA; }
  rc = make_layout(shape, c->n_sms, &c->lay);
  if (rc == LOSA_OK && workspace_bytes < c->lay.total) rc = LOSA_ERR_INVALID_ARG;
  if (rc == LOSA_OK && shape->max_pages_per_seq > topk_max_sortable(c)) rc = LOSA_ERR_UNSUPPORTED;
  if (rc != LOSA_OK) { delete c; return rc; }
  // status word, arrival counters and page bitmaps start at zero
  e = cudaMemset(c->ws, 0, c->lay.delta);
  if (e != cudaSuccess) { delete c; return LOSA_ERR_CUDA; }
  *out = c;
  return LOSA_OK;
}

int32_t losa_destroy(losa_ctx* ctx) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  if (ctx->ev_begin) cudaEventDestroy(ctx->ev_begin);
  if (ctx->ev_end) cudaEventDestroy(ctx->ev_end);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
  delete ctx;
  return LOSA_OK;
}

int32_t losa_poll_status(losa_ctx* ctx, void* stream) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  LOSA_CUDA_TRY(ctx, cudaStreamSynchronize(as_stream(stream)));
  int32_t st = 0;
  LOSA_CUDA_TRY(ctx, cudaMemcpy(&st, status_ptr(ctx), sizeof(st), cudaMemcpyDeviceToHost));
  if (st != 0) LOSA_CUDA_TRY(ctx, cudaMemset(status_ptr(ctx), 0, sizeof(st)));
  return st;
}

int32_t losa_profile_stage4(losa_ctx* ctx, int32_t enable) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  if (enable && !ctx->ev_begin) {
    LOSA_CUDA_TRY(ctx, cudaEventCreate(&ctx->ev_begin));
    LOSA_CUDA_TRY(ctx, cudaEventCreate(&ctx->ev_end));
  }
  ctx->profile = enable ? 1 : 0;
  return LOSA_OK;
}

int32_t losa_stage4_last_ms(losa_ctx* ctx, float* out_ms) {
  if (!ctx || !out_ms || !ctx->ev_begin) return LOSA_ERR_INVALID_ARG;
  LOSA_CUDA_TRY(ctx, cudaEventSynchronize(ctx->ev_end));
  LOSA_CUDA_TRY(ctx, cudaEventElapsedTime(out_ms, ctx->ev_begin, ctx->ev_end));
  return LOSA_OK;
}

int32_t losa_set_wait_limit(losa_ctx* ctx, int64_t cycles) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  ctx->wait_cycles = cycles > 0 ? cycles : 0;
  return LOSA_OK;
}

int32_t losa_last_cuda_error(const losa_ctx* ctx) { return ctx ? ctx->last_cuda_error : 0; }
int64_t losa_launch_count(const losa_ctx* ctx) { return ctx ? ctx->launches : 0; }

int32_t losa_select_active(losa_ctx* ctx, const void* x_cur, const void* x_prev, int32_t row_width,
                           const int32_t* m_per_seq, const int32_t* step, int32_t* active_idx,
                           int32_t* n_active, float* delta_opt, void* stream) {
  if (!ctx || !x_cur || !x_prev || !active_idx || !n_active || row_width < 1) return LOSA_ERR_INVALID_ARG;
  if (row_width % 8 != 0 || !aligned16(x_cur) || !aligned16(x_prev)) return LOSA_ERR_UNSUPPORTED;
  return launch_select_active(ctx, x_cur, x_prev, row_width, m_per_seq, step, active_idx, n_active, delta_opt, as_stream(stream));
}

int32_t losa_select_active_tau(losa_ctx* ctx, const void* x_cur, const void* x_prev, int32_t row_width,
                               double tau, const int32_t* m_cap_opt, const int32_t* step, int32_t* active_idx,
                               int32_t* n_active, float* delta_opt, void* stream) {
  if (!ctx || !x_cur || !x_prev || !active_idx || !n_active || row_width < 1 || !(tau > 0.0) || tau > 1.0)
    return LOSA_ERR_INVALID_ARG;
  if (row_width % 8 != 0 || !aligned16(x_cur) || !aligned16(x_prev)) return LOSA_ERR_UNSUPPORTED;
  return launch_select_active(ctx, x_cur, x_prev, row_width, m_cap_opt, step, active_idx, n_active, delta_opt, as_stream(stream), tau);
}

int32_t losa_page_scores_topk(losa_ctx* ctx, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                              const int32_t* n_active, const int32_t* step, int32_t k, int32_t* topk_pages,
                              float* topk_scores_opt, void* stream) {
  if (!ctx || !q || !active_idx || !n_active || !topk_pages || k < 1) return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, true);
  if (rc != LOSA_OK) return rc;
  if (!aligned16(q)) return LOSA_ERR_UNSUPPORTED;
  return launch_page_scores_topk(ctx, q, kv, active_idx, n_active, step, k, topk_pages, topk_scores_opt, as_stream(stream));
}

int32_t losa_page_scores_topk_pooled(losa_ctx* ctx, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                                     const int32_t* n_active, const int32_t* step, int32_t k, int32_t* topk_pages,
                                     float* topk_scores_opt, void* stream) {
  if (!ctx || !q || !active_idx || !n_active || !topk_pages || k < 1) return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, true);
  if (rc != LOSA_OK) return rc;
  if (!aligned16(q)) return LOSA_ERR_UNSUPPORTED;
  return launch_page_scores_topk(ctx, q, kv, active_idx, n_active, step, k, topk_pages, topk_scores_opt, as_stream(stream), kSelectorPooled);
}

int32_t losa_page_scores_topk_mma(losa_ctx* ctx, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                                  const int32_t* n_active, const int32_t* step, int32_t k, int32_t* topk_pages,
                                  float* topk_scores_opt, void* stream) {
  if (!ctx || !q || !active_idx || !n_active || !topk_pages || k < 1) return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, true);
  if (rc != LOSA_OK) return rc;
  if (!aligned16(q) || ctx->shape.dtype != LOSA_BF16) return LOSA_ERR_UNSUPPORTED;
  return launch_page_scores_topk(ctx, q, kv, active_idx, n_active, step, k, topk_pages, topk_scores_opt, as_stream(stream), kSelectorMma);
}

int32_t losa_set_pooled_selection(losa_ctx* ctx, int32_t on) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  ctx->pooled_selection = on ? 1 : 0;
  return LOSA_OK;
}

int32_t losa_set_step_selector(losa_ctx* ctx, int32_t selector) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  if (selector != LOSA_SELECTOR_EXACT && selector != LOSA_SELECTOR_POOLED && selector != LOSA_SELECTOR_MMA)
    return LOSA_ERR_INVALID_ARG;
  if (selector == LOSA_SELECTOR_MMA && ctx->shape.dtype != LOSA_BF16) return LOSA_ERR_UNSUPPORTED;
  ctx->pooled_selection = selector;                  // the codes are those of launch_page_scores_topk
  return LOSA_OK;
}

int32_t losa_page_union(losa_ctx* ctx, const int32_t* topk_pages, const int32_t* active_idx,
                        const int32_t* n_active, int32_t k, const int32_t* kv_len, const int32_t* step,
                        int32_t* union_pages, int32_t* union_count, void* stream) {
  if (!ctx || !topk_pages || !active_idx || !n_active || !kv_len || !union_pages || !union_count || k < 1)
    return LOSA_ERR_INVALID_ARG;
  return launch_page_union(ctx, topk_pages, active_idx, n_active, k, kv_len, step, union_pages, union_count, as_stream(stream));
}

int32_t losa_sparse_prefix_attn(losa_ctx* ctx, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                                const int32_t* n_active, const int32_t* union_pages, const int32_t* union_count,
                                losa_state_t* state, void* stream) {
  if (!ctx || !q || !active_idx || !n_active || !union_pages || !union_count || !state || !state->o_p || !state->lse_p)
    return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, false);
  if (rc == LOSA_OK) rc = check_state_format(ctx, state);
  if (rc != LOSA_OK) return rc;
  if (!aligned16(q) || !aligned16(state->o_p)) return LOSA_ERR_UNSUPPORTED;
  return launch_sparse_prefix_attn(ctx, q, kv, active_idx, n_active, union_pages, union_count, state, as_stream(stream));
}

int32_t losa_block_attn_merge(losa_ctx* ctx, const void* q, const void* k_blk, const void* v_blk,
                              const losa_state_t* state, void* out, float* lse_out_opt, void* stream) {
  if (!ctx || !q || !k_blk || !v_blk || !state || !state->o_p || !state->lse_p || !out) return LOSA_ERR_INVALID_ARG;
  const int32_t rc = check_state_format(ctx, state);
  if (rc != LOSA_OK) return rc;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out) || !aligned16(state->o_p)) return LOSA_ERR_UNSUPPORTED;
  return launch_block_attn_merge(ctx, q, k_blk, v_blk, state, out, lse_out_opt, as_stream(stream));
}

int32_t losa_update_prefix_cache(losa_ctx* ctx, losa_kv_t* kv, losa_state_t* state, const void* q,
                                 const void* k_blk, const void* v_blk, int32_t finalize_block, void* stream) {
  if (!ctx || !state || !state->step) return LOSA_ERR_INVALID_ARG;
  if (!finalize_block) {
    if (!q || !state->q_prev) return LOSA_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(state->q_prev)) return LOSA_ERR_UNSUPPORTED;
  } else {
    if (!k_blk || !v_blk) return LOSA_ERR_INVALID_ARG;
    int32_t rc = check_kv(ctx, kv, true);
    if (rc != LOSA_OK) return rc;
  }
  return launch_update_prefix_cache(ctx, kv, state, q, k_blk, v_blk, finalize_block, as_stream(stream));
}

int32_t losa_quantize_kv_pages(losa_ctx* ctx, const losa_kv_t* src, losa_kv_t* dst, void* stream) {
  if (!ctx || !src || !dst) return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, src, false);
  if (rc == LOSA_OK) rc = check_kv(ctx, dst, true);
  if (rc != LOSA_OK) return rc;
  if (src->kv_format != LOSA_KV_NATIVE || dst->kv_format != LOSA_KV_FP8_E4M3 || src->n_phys_pages != dst->n_phys_pages)
    return LOSA_ERR_INVALID_ARG;
  return launch_fp8_quantize(ctx, src, dst, as_stream(stream));
}

int32_t losa_build_page_summaries(losa_ctx* ctx, losa_kv_t* kv, void* stream) {
  if (!ctx) return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, true);
  if (rc != LOSA_OK) return rc;
  return launch_build_page_summaries(ctx, kv, as_stream(stream));
}

int32_t losa_denoise_step(losa_ctx* ctx, const void* q, const void* k_blk, const void* v_blk, void* out,
                          float* lse_out_opt, losa_kv_t* kv, losa_state_t* state, const losa_step_buffers_t* buf,
                          const int32_t* m_per_seq, int32_t k, void* stream) {
  if (!ctx || !q || !k_blk || !v_blk || !out || !buf || !state || !state->step || !state->q_prev || !state->o_p ||
      !state->lse_p || k < 1)
    return LOSA_ERR_INVALID_ARG;
  if (!buf->active_idx || !buf->n_active || !buf->topk_pages || !buf->union_pages || !buf->union_count)
    return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, true);
  if (rc == LOSA_OK) rc = check_state_format(ctx, state);
  if (rc != LOSA_OK) return rc;
  if (!aligned16(q) || !aligned16(k_blk) || !aligned16(v_blk) || !aligned16(out) || !aligned16(state->q_prev) ||
      !aligned16(state->o_p))
    return LOSA_ERR_UNSUPPORTED;
  if (!ctx->side_stream) {
    // lowest priority: when CTAs of both streams are pending, those of stages 1-4 go first
    int prio_lo = 0, prio_hi = 0;
    LOSA_CUDA_TRY(ctx, cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi));
    LOSA_CUDA_TRY(ctx, cudaStreamCreateWithPriority(&ctx->side_stream, cudaStreamNonBlocking, prio_lo));
    LOSA_CUDA_TRY(ctx, cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming));
    LOSA_CUDA_TRY(ctx, cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming));
  }
  cudaStream_t st = as_stream(stream);
  const losa_shape_t& sh = ctx->shape;
  // fork: the in-block attention needs nothing from stages 1-4
  LOSA_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_fork, st));
  LOSA_CUDA_TRY(ctx, cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0));
  rc = launch_block_attn(ctx, q, k_blk, v_blk, ctx->side_stream);
  if (rc != LOSA_OK) return rc;
  LOSA_CUDA_TRY(ctx, cudaEventRecord(ctx->ev_join, ctx->side_stream));
  int32_t* slot_map = reinterpret_cast<int32_t*>(ctx->ws + ctx->lay.slot_map);
  rc = launch_select_active(ctx, q, state->q_prev, sh.n_q_heads * sh.head_dim, m_per_seq, state->step,
                            buf->active_idx, buf->n_active, nullptr, st, 0.0, slot_map);
  bool union_done = false;                              // stage 3 written by the selection kernel itself
  if (rc == LOSA_OK) rc = launch_page_scores_topk(ctx, q, kv, buf->active_idx, buf->n_active, state->step, k, buf->topk_pages, nullptr, st, ctx->pooled_selection, true, buf->union_pages, buf->union_count, &union_done);
  if (rc == LOSA_OK && !union_done) rc = launch_page_union(ctx, buf->topk_pages, buf->active_idx, buf->n_active, k, kv->kv_len, state->step, buf->union_pages, buf->union_count, st);
  if (rc == LOSA_OK) rc = launch_sparse_prefix_attn(ctx, q, kv, buf->active_idx, buf->n_active, buf->union_pages, buf->union_count, state, st, true);
  // join (also when a launch above failed: the forked kernel must not be left reading the caller's
  // buffers, nor a capture be left with an unjoined branch), then one pass over the rows: (merge of
  // the partial records,) merge with the block part, commit
  const cudaError_t joined = cudaStreamWaitEvent(st, ctx->ev_join, 0);
  if (rc != LOSA_OK) return rc;
  LOSA_CUDA_TRY(ctx, joined);
  if (finish_fuses_combine(ctx)) return launch_attn_finish(ctx, q, buf->active_idx, buf->n_active, slot_map, state, out, lse_out_opt, st);
  return launch_merge_commit(ctx, q, state, out, lse_out_opt, st);
}

int32_t losa_denoise_step_host(losa_ctx* ctx, const void* h_q, const void* h_k_blk, const void* h_v_blk,
                               void* h_out, losa_kv_t* kv, losa_state_t* state, const losa_step_buffers_t* buf,
                               const int32_t* m_per_seq, int32_t k, void* stream) {
  if (!ctx || !h_q || !h_k_blk || !h_v_blk || !h_out || !buf || !state || !state->step || !state->q_prev)
    return LOSA_ERR_INVALID_ARG;
  if (!buf->d_q || !buf->d_k_blk || !buf->d_v_blk || !buf->d_out || !buf->active_idx || !buf->n_active ||
      !buf->topk_pages || !buf->union_pages || !buf->union_count)
    return LOSA_ERR_INVALID_ARG;
  int32_t rc = check_kv(ctx, kv, true);
  if (rc != LOSA_OK) return rc;
  const losa_shape_t& sh = ctx->shape;
  const size_t es = sh.dtype == LOSA_BF16 ? 2 : 4;
  const size_t qb = static_cast<size_t>(sh.batch) * sh.block_size * sh.n_q_heads * sh.head_dim * es;
  const size_t kb = static_cast<size_t>(sh.batch) * sh.block_size * sh.n_kv_heads * sh.head_dim * es;
  cudaStream_t st = as_stream(stream);
  LOSA_CUDA_TRY(ctx, cudaMemcpyAsync(buf->d_q, h_q, qb, cudaMemcpyHostToDevice, st));
  LOSA_CUDA_TRY(ctx, cudaMemcpyAsync(buf->d_k_blk, h_k_blk, kb, cudaMemcpyHostToDevice, st));
  LOSA_CUDA_TRY(ctx, cudaMemcpyAsync(buf->d_v_blk, h_v_blk, kb, cudaMemcpyHostToDevice, st));
  rc = losa_denoise_step(ctx, buf->d_q, buf->d_k_blk, buf->d_v_blk, buf->d_out, nullptr, kv, state, buf, m_per_seq, k, stream);
  if (rc != LOSA_OK) return rc;
  LOSA_CUDA_TRY(ctx, cudaMemcpyAsync(h_out, buf->d_out, qb, cudaMemcpyDeviceToHost, st));
  return LOSA_OK;
}

}  // extern "C"
