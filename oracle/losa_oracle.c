/*
 * losa_oracle.c — CPU oracle of the LoSA per-denoising-step attention path (see losa_oracle.h).
 *
 * TEST INFRASTRUCTURE.  Every function follows one passage of the paper, stated above it, with no
 * blocking, fusion or reordering beyond that passage.  fp64 throughout, except the page score,
 * which is also produced in the fp32 order fixed by the library's interface because it decides
 * integer page ids.  Build: gcc -O2 -std=c11 -fopenmp -ffp-contract=off (no fast-math).
 */
#include "losa_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---------- element access: fp32 or bf16 bit patterns ---------- */

#define ORACLE_MAX_BLOCK 1024

static inline size_t esize(int dtype) { return dtype == 1 ? 2 : 4; }

static inline float ld_f32(const void* p, int dtype, int64_t i) {
  if (dtype == 1) {
    uint32_t bits = ((uint32_t)((const uint16_t*)p)[i]) << 16;
    float f;
    memcpy(&f, &bits, 4);
    return f;
  }
  return ((const float*)p)[i];
}
static inline double ld(const void* p, int dtype, int64_t i) { return (double)ld_f32(p, dtype, i); }

static inline void cp_elem(void* dst, int64_t di, const void* src, int64_t si, int dtype, int64_t n) {
  size_t e = esize(dtype);
  memcpy((char*)dst + (size_t)di * e, (const char*)src + (size_t)si * e, (size_t)n * e);
}

static inline int pages_of(int32_t len, int32_t g) { return (len + g - 1) / g; }

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* offset (in elements) of token `slot` of physical page `phys`, KV head `kh` */
static inline int64_t kv_off(const oracle_kv_t* kv, int32_t phys, int32_t kh, int32_t slot) {
  return (int64_t)phys * kv->stride_page + (int64_t)kh * kv->stride_head +
         (int64_t)slot * kv->stride_tok;
}

/* ---------- Section 2.3: per-page min and max keys ---------- */

static void summarise_page(const oracle_shape_t* sh, oracle_kv_t* kv, int32_t s, int32_t p) {
  const int g = sh->page_size, d = sh->head_dim, Hkv = sh->n_kv_heads;
  int valid = kv->kv_len[s] - p * g;
  if (valid > g) valid = g;
  if (valid <= 0) return;
  const int32_t phys = kv->page_table[(int64_t)s * sh->max_pages_per_seq + p];
  for (int kh = 0; kh < Hkv; ++kh) {
    for (int j = 0; j < d; ++j) {
      int tmin = 0, tmax = 0;
      double vmin = ld(kv->k_pages, sh->dtype, kv_off(kv, phys, kh, 0) + j), vmax = vmin;
      for (int t = 1; t < valid; ++t) {
        double v = ld(kv->k_pages, sh->dtype, kv_off(kv, phys, kh, t) + j);
        if (v < vmin) { vmin = v; tmin = t; }
        if (v > vmax) { vmax = v; tmax = t; }
      }
      int64_t so = ((int64_t)phys * Hkv + kh) * d + j;
      cp_elem(kv->kmin, so, kv->k_pages, kv_off(kv, phys, kh, tmin) + j, sh->dtype, 1);
      cp_elem(kv->kmax, so, kv->k_pages, kv_off(kv, phys, kh, tmax) + j, sh->dtype, 1);
    }
  }
}

void oracle_build_page_summaries(const oracle_shape_t* sh, oracle_kv_t* kv) {
  for (int s = 0; s < sh->batch; ++s) {
    const int P = pages_of(kv->kv_len[s], sh->page_size);
#pragma omp parallel for schedule(static)
    for (int p = 0; p < P; ++p) summarise_page(sh, kv, s, p);
  }
}

/* ---------- Eq. 1 (Section 3.2) and locality pruning (Section 4.1) ----------
 * Delta_i = mean over the row of (x_cur - x_prev)^2; the m tokens with the largest Delta are
 * active.  Ties go to the lower token index (the paper gives no tie rule).  step == 0, no m, or
 * m < 0: every token is active ("Initialization Workflow", Section 4.2). */
void oracle_select_active(const oracle_shape_t* sh, const void* x_cur, const void* x_prev,
                          int32_t row_width, const int32_t* m_per_seq, const int32_t* step,
                          int32_t* active_idx, int32_t* n_active, double* delta) {
  const int B = sh->block_size;
  double* dl = (double*)malloc(sizeof(double) * (size_t)B);
  for (int s = 0; s < sh->batch; ++s) {
    for (int i = 0; i < B; ++i) {
      const int64_t row = ((int64_t)s * B + i) * row_width;
      double acc = 0.0;
      for (int c = 0; c < row_width; ++c) {
        double df = ld(x_cur, sh->dtype, row + c) - ld(x_prev, sh->dtype, row + c);
        acc += df * df;
      }
      dl[i] = acc / (double)row_width;
      if (delta) delta[(int64_t)s * B + i] = dl[i];
    }
    int m = m_per_seq ? m_per_seq[s] : -1;
    if (m < 0 || m > B || (step && step[s] == 0)) m = B;
    int cnt = 0;
    for (int i = 0; i < B; ++i) {
      /* rank of token i under (Delta descending, index ascending) */
      int rank = 0;
      for (int j = 0; j < B; ++j)
        if (dl[j] > dl[i] || (dl[j] == dl[i] && j < i)) ++rank;
      if (rank < m) active_idx[(int64_t)s * B + cnt++] = i; /* i ascends, so the list is sorted */
    }
    n_active[s] = cnt;
    for (int i = cnt; i < B; ++i) active_idx[(int64_t)s * B + i] = -1;
  }
  free(dl);
}

/* ---------- threshold variant of the pruning rule (appendix, locality heat maps with tau = 0.5) ----------
 * Tokens are ranked as above; the active set is the shortest leading part of the ranking whose
 * Delta values add up to at least tau times the sum over the block ("the boundary where the
 * cumulative normalised MSE reaches 50% of the total").  Both sums run over the ranking in order.
 * A block whose Delta are all zero has no active token.  m_cap (optional) bounds the count from
 * above; step == 0 makes every token active. */
void oracle_select_active_tau(const oracle_shape_t* sh, const void* x_cur, const void* x_prev,
                              int32_t row_width, double tau, const int32_t* m_cap, const int32_t* step,
                              int32_t* active_idx, int32_t* n_active, double* delta) {
  const int B = sh->block_size;
  double* dl = (double*)malloc(sizeof(double) * (size_t)B);
  double* sorted = (double*)malloc(sizeof(double) * (size_t)B);
  int* rank = (int*)malloc(sizeof(int) * (size_t)B);
  for (int s = 0; s < sh->batch; ++s) {
    for (int i = 0; i < B; ++i) {
      const int64_t row = ((int64_t)s * B + i) * row_width;
      double acc = 0.0;
      for (int c = 0; c < row_width; ++c) {
        double df = ld(x_cur, sh->dtype, row + c) - ld(x_prev, sh->dtype, row + c);
        acc += df * df;
      }
      dl[i] = acc / (double)row_width;
      if (delta) delta[(int64_t)s * B + i] = dl[i];
    }
    for (int i = 0; i < B; ++i) {
      int r = 0;
      for (int j = 0; j < B; ++j)
        if (dl[j] > dl[i] || (dl[j] == dl[i] && j < i)) ++r;
      rank[i] = r;
      sorted[r] = dl[i];
    }
    int m;
    if (step && step[s] == 0) {
      m = B;
    } else {
      double total = 0.0;
      for (int r = 0; r < B; ++r) total += sorted[r];
      const double thr = tau * total;
      double cum = 0.0;
      m = 0;
      while (m < B && cum < thr) cum += sorted[m++];
      if (m_cap && m_cap[s] >= 0 && m_cap[s] < m) m = m_cap[s];
    }
    int cnt = 0;
    for (int i = 0; i < B; ++i)
      if (rank[i] < m) active_idx[(int64_t)s * B + cnt++] = i;
    n_active[s] = cnt;
    for (int i = cnt; i < B; ++i) active_idx[(int64_t)s * B + i] = -1;
  }
  free(dl);
  free(sorted);
  free(rank);
}

/* ---------- Section 2.3: query-dependent upper bound of the attention score per page ----------
 * For a page with element-wise key bounds kmin <= k <= kmax, q.k <= sum_j max(q_j kmin_j,
 * q_j kmax_j) — the tightest bound those summaries allow.  The 1/sqrt(d) factor is omitted: it
 * does not change the ranking. */

/* fp32 in the order the library's interface fixes (the paper fixes none).  Since kmin <= kmax,
 * max(q kmin, q kmax) = max(q,0) kmax + min(q,0) kmin, one of the two terms being zero.  Each run
 * of 8 consecutive j: acc = +0, then for j ascending acc = fma(max(q_j,0), kmax_j, acc) followed by
 * acc = fma(min(q_j,0), kmin_j, acc); the d/8 run sums are combined by c[i] <- c[i] + c[i xor off],
 * off = d/16 .. 1; then + 0.0f.  fmaf is the correctly rounded fused operation. */
static float page_bound_f32(const float* q, const float* lo, const float* hi, int d) {
  float c[64], n[64];
  const int nc = d / 8;
  for (int r = 0; r < nc; ++r) {
    float acc = 0.0f;
    for (int jj = 0; jj < 8; ++jj) {
      const int j = r * 8 + jj;
      const float qp = (q[j] > 0.0f) ? q[j] : 0.0f;
      const float qn = (q[j] < 0.0f) ? q[j] : 0.0f;
      acc = fmaf(qp, hi[j], acc);
      acc = fmaf(qn, lo[j], acc);
    }
    c[r] = acc;
  }
  for (int off = nc / 2; off >= 1; off /= 2) {
    for (int i = 0; i < nc; ++i) n[i] = c[i] + c[i ^ off];
    for (int i = 0; i < nc; ++i) c[i] = n[i];
  }
  return c[0] + 0.0f;
}

static double page_bound_f64(const float* q, const float* lo, const float* hi, int d) {
  double acc = 0.0;
  for (int j = 0; j < d; ++j) {
    const double a = (double)q[j] * (double)lo[j], b = (double)q[j] * (double)hi[j];
    acc += (a > b) ? a : b;
  }
  return acc;
}

void oracle_page_scores_one(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                            int32_t s, int32_t tok, int32_t head, float* u32, double* u64) {
  const int d = sh->head_dim, Hkv = sh->n_kv_heads, G = sh->n_q_heads / Hkv;
  const int kh = head / G;
  const int P = pages_of(kv->kv_len[s], sh->page_size);
  float qv[512], lo[512], hi[512];
  const int64_t qo = (((int64_t)s * sh->block_size + tok) * sh->n_q_heads + head) * d;
  for (int j = 0; j < d; ++j) qv[j] = ld_f32(q, sh->dtype, qo + j);
  for (int p = 0; p < P; ++p) {
    const int32_t phys = kv->page_table[(int64_t)s * sh->max_pages_per_seq + p];
    const int64_t so = ((int64_t)phys * Hkv + kh) * d;
    for (int j = 0; j < d; ++j) {
      lo[j] = ld_f32(kv->kmin, sh->dtype, so + j);
      hi[j] = ld_f32(kv->kmax, sh->dtype, so + j);
    }
    if (u32) u32[p] = page_bound_f32(qv, lo, hi, d);
    if (u64) u64[p] = page_bound_f64(qv, lo, hi, d);
  }
}

/* ---------- FP8 K/V pages (extension: the paper names quantised attention as orthogonal to the
 * method, Section 6, and quotes its cached state in FP16, Section 4.5 "Memory overhead") ----------
 * Format: E4M3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; largest finite value 448;
 * no infinities).  One scale per (physical page, KV head) and tensor, a power of two:
 *   amax = largest |x| over the page's valid tokens and d dimensions,
 *   scale = 2^e, e = the smallest integer with amax <= 448 * 2^e, clamped to [-6, 7]  (amax = 0: e = -6),
 *   code  = round-to-nearest-even of x / scale onto the E4M3 grid, saturated at +-448,
 *   dequantised value = scale * value(code)   (exact in bf16 and fp16: four significant bits).
 * Slots of a page past the prefix's end get code 0.  Appending a block re-quantises every touched
 * page from the dequantised old values and the new rows together (the scale may have to grow). */
double oracle_fp8_decode(uint8_t code) {
  const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0) v = ldexp((double)m, -9);                  /* subnormal: m * 2^-3 * 2^-6 */
  else v = ldexp(1.0 + m / 8.0, e - 7);
  return sign ? -v : v;
}
uint8_t oracle_fp8_encode(double y) {
  const uint8_t sign = (y < 0.0 || (y == 0.0 && signbit(y))) ? 0x80 : 0;
  double a = fabs(y);
  if (!(a == a)) return 0x7f;                             /* NaN in, NaN out (never produced from finite inputs) */
  if (a >= 448.0) return sign | 0x7e;                     /* saturate: 0x7e = 448 */
  double r;
  int ex;
  if (a < ldexp(1.0, -6)) {                               /* subnormal range, step 2^-9 */
    r = nearbyint(ldexp(a, 9));                           /* ties to even (default rounding mode) */
    if (r >= 8.0) return sign | 0x08;                     /* rounded up to the first normal, 2^-6 */
    return sign | (uint8_t)r;
  }
  (void)frexp(a, &ex);                                    /* a = f * 2^ex, f in [0.5, 1)  =>  2^(ex-1) <= a < 2^ex */
  int e = ex - 1;                                         /* binade of a */
  r = nearbyint(ldexp(a, 3 - e));                         /* a / 2^(e-3): in [8, 16], ties to even */
  if (r >= 16.0) { r = 8.0; e += 1; }
  if (e > 8 || (e == 8 && r > 14.0)) return sign | 0x7e;
  return sign | (uint8_t)(((e + 7) << 3) | ((int)r - 8));
}
static int fp8_scale_exp(double amax) {
  if (!(amax > 0.0)) return -6;
  int e = -6;
  while (e < 7 && amax > ldexp(448.0, e)) ++e;
  return e;
}
/* quantises n valid token rows (read through get(ctx, t, j)) of one (page, KV head) into codes[g][d] */
typedef double (*fp8_get_fn)(const void* ctx, int t, int j);
static float fp8_quantize_rows(fp8_get_fn get, const void* ctx, int n, int g, int d, uint8_t* codes) {
  double amax = 0.0;
  for (int t = 0; t < n; ++t)
    for (int j = 0; j < d; ++j) { const double a = fabs(get(ctx, t, j)); if (a > amax) amax = a; }
  const int e = fp8_scale_exp(amax);
  for (int t = 0; t < g; ++t)
    for (int j = 0; j < d; ++j) codes[(int64_t)t * d + j] = t < n ? oracle_fp8_encode(ldexp(get(ctx, t, j), -e)) : 0;
  return (float)ldexp(1.0, e);
}
typedef struct { const void* base; int dtype; int64_t off, stride_tok; } fp8_src_t;
static double fp8_get_pool(const void* c, int t, int j) {
  const fp8_src_t* s = (const fp8_src_t*)c;
  return ld(s->base, s->dtype, s->off + (int64_t)t * s->stride_tok + j);
}
void oracle_fp8_quantize_pages(const oracle_shape_t* sh, const oracle_kv_t* src, uint8_t* k_codes, uint8_t* v_codes,
                               float* k_scale, float* v_scale) {
  const int Hkv = sh->n_kv_heads, g = sh->page_size, d = sh->head_dim;
  for (int s = 0; s < sh->batch; ++s) {
    const int L = src->kv_len[s], P = pages_of(L, g);
    for (int p = 0; p < P; ++p) {
      const int32_t phys = src->page_table[(int64_t)s * sh->max_pages_per_seq + p];
      const int n = (L - p * g) < g ? (L - p * g) : g;
      for (int kh = 0; kh < Hkv; ++kh) {
        const int64_t co = ((int64_t)phys * Hkv + kh) * g * d;
        fp8_src_t ks = {src->k_pages, sh->dtype, kv_off(src, phys, kh, 0), src->stride_tok};
        fp8_src_t vs = {src->v_pages, sh->dtype, kv_off(src, phys, kh, 0), src->stride_tok};
        k_scale[(int64_t)phys * Hkv + kh] = fp8_quantize_rows(fp8_get_pool, &ks, n, g, d, k_codes + co);
        v_scale[(int64_t)phys * Hkv + kh] = fp8_quantize_rows(fp8_get_pool, &vs, n, g, d, v_codes + co);
      }
    }
  }
}
/* writes scale * value(code) of the valid tokens of every logical page into dst's pools (element dtype) */
static void st_elem(void* p, int dtype, int64_t i, double v) {
  if (dtype == 1) {                                       /* bf16: the values written here are exact in bf16 */
    float f = (float)v;
    uint32_t u;
    memcpy(&u, &f, 4);
    ((uint16_t*)p)[i] = (uint16_t)(u >> 16);
  } else {
    ((float*)p)[i] = (float)v;
  }
}
void oracle_fp8_dequantize_pages(const oracle_shape_t* sh, const uint8_t* k_codes, const uint8_t* v_codes,
                                 const float* k_scale, const float* v_scale, oracle_kv_t* dst) {
  const int Hkv = sh->n_kv_heads, g = sh->page_size, d = sh->head_dim;
  for (int s = 0; s < sh->batch; ++s) {
    const int L = dst->kv_len[s], P = pages_of(L, g);
    for (int p = 0; p < P; ++p) {
      const int32_t phys = dst->page_table[(int64_t)s * sh->max_pages_per_seq + p];
      const int n = (L - p * g) < g ? (L - p * g) : g;
      for (int kh = 0; kh < Hkv; ++kh) {
        const int64_t co = ((int64_t)phys * Hkv + kh) * g * d;
        const double ksc = k_scale[(int64_t)phys * Hkv + kh], vsc = v_scale[(int64_t)phys * Hkv + kh];
        for (int t = 0; t < n; ++t)
          for (int j = 0; j < d; ++j) {
            st_elem(dst->k_pages, sh->dtype, kv_off(dst, phys, kh, t) + j, ksc * oracle_fp8_decode(k_codes[co + (int64_t)t * d + j]));
            st_elem(dst->v_pages, sh->dtype, kv_off(dst, phys, kh, t) + j, vsc * oracle_fp8_decode(v_codes[co + (int64_t)t * d + j]));
          }
      }
    }
  }
}
typedef struct { const uint8_t* codes; double scale; int n_old; const void* blk; int dtype; int64_t blk_off; int blk_stride; int d; } fp8_mix_t;
static double fp8_get_mix(const void* c, int t, int j) {
  const fp8_mix_t* m = (const fp8_mix_t*)c;
  if (t < m->n_old) return m->scale * oracle_fp8_decode(m->codes[(int64_t)t * m->d + j]);
  return ld(m->blk, m->dtype, m->blk_off + (int64_t)(t - m->n_old) * m->blk_stride + j);
}
/* block finalisation on an FP8 cache: appends the block's rows at prefix positions L_s .. L_s+B-1 and
 * re-quantises every touched page; kv_len[s] += B.  (Summaries and the step counter are the caller's.) */
void oracle_fp8_append_block(const oracle_shape_t* sh, const int32_t* page_table, int32_t* kv_len,
                             uint8_t* k_codes, uint8_t* v_codes, float* k_scale, float* v_scale,
                             const void* k_blk, const void* v_blk) {
  const int B = sh->block_size, Hkv = sh->n_kv_heads, g = sh->page_size, d = sh->head_dim;
  uint8_t* tmp = (uint8_t*)malloc((size_t)g * d);
  for (int s = 0; s < sh->batch; ++s) {
    const int L0 = kv_len[s];
    for (int p = L0 / g; p <= (L0 + B - 1) / g; ++p) {
      const int32_t phys = page_table[(int64_t)s * sh->max_pages_per_seq + p];
      const int n_old = L0 > p * g ? L0 - p * g : 0;                 /* tokens the page already holds */
      const int last = (L0 + B) < (p + 1) * g ? (L0 + B) : (p + 1) * g;
      const int n_new = last - (p * g + n_old);
      const int first_blk = p * g + n_old - L0;                      /* block row of the first new token */
      for (int kh = 0; kh < Hkv; ++kh) {
        const int64_t co = ((int64_t)phys * Hkv + kh) * g * d, so = (int64_t)phys * Hkv + kh;
        for (int which = 0; which < 2; ++which) {
          uint8_t* codes = (which ? v_codes : k_codes) + co;
          float* scale = (which ? v_scale : k_scale) + so;
          fp8_mix_t mx = {codes, n_old ? (double)*scale : 1.0, n_old, which ? v_blk : k_blk, sh->dtype,
                          (((int64_t)s * B + first_blk) * Hkv + kh) * d, Hkv * d, d};
          const float sc = fp8_quantize_rows(fp8_get_mix, &mx, n_old + n_new, g, d, tmp);
          memcpy(codes, tmp, (size_t)g * d);
          *scale = sc;
        }
      }
    }
    kv_len[s] = L0 + B;
  }
  free(tmp);
}

/* ---------- bf16 state (extension of the cached statistics' format) ----------
 * The paper quotes the per-block cache in FP16 (memory overhead, Section 4.5); the interface keeps it in
 * fp32 by default.  With the bf16 state the cached prefix output o_p of a token is STORED rounded to
 * bf16 - eight significant bits, ties to even, subnormals below 2^-126 on the 2^-133 grid - and every
 * later use (the merge of the same step, the reuse in later steps) sees the rounded value; L_p stays as
 * it is.  oracle_round_state_bf16 rounds, in place, the rows stage 4 has just written: those of the
 * active tokens. */
double oracle_round_bf16(double x) {
  if (x == 0.0 || !(x == x) || isinf(x)) return x;
  int ex;
  (void)frexp(fabs(x), &ex);                              /* 2^(ex-1) <= |x| < 2^ex */
  int e = ex - 1;
  if (e < -126) e = -126;                                 /* subnormal range: fixed step 2^-133 */
  const double r = nearbyint(ldexp(x, 7 - e));            /* |x| / 2^(e-7) in [128, 256): ties to even */
  return ldexp(r, e - 7);                                 /* (256 * 2^(e-7) = 2^(e+1): the next binade, still exact) */
}
void oracle_round_state_bf16(const oracle_shape_t* sh, double* o_p, const int32_t* active_idx,
                             const int32_t* n_active) {
  const int B = sh->block_size, H = sh->n_q_heads, d = sh->head_dim;
  for (int s = 0; s < sh->batch; ++s)
    for (int a = 0; a < n_active[s]; ++a) {
      double* row = o_p + ((int64_t)s * B + active_idx[(int64_t)s * B + a]) * H * d;
      for (int64_t i = 0; i < (int64_t)H * d; ++i) row[i] = oracle_round_bf16(row[i]);
    }
}

/* ---------- Section 2.3: relaxed validity of a page list (selector variants with their own arithmetic) ----------
 * The paper fixes no arithmetic for the page bound, and calls the method independent of the
 * selector.  A selector that evaluates U(p) = sum_j max(q_j kmin_j, q_j kmax_j) in another order
 * or precision than the fixed fp32 order cannot be compared list by list; it is checked against
 * this rule instead, in fp64:
 *   a list of (token, head) is VALID iff it holds exactly min(k, P_s) distinct pages of
 *   0 .. P_s - 1 followed by -1 padding, and every listed page p has
 *       U64(p) >= T - eps * Smax,
 *   where T is the min(k, P_s)-th largest U64 over all pages and Smax = max_p sum_j |t_j(p)|,
 *   t_j = the larger of q_j kmin_j and q_j kmax_j (the magnitude rounding errors scale with).
 * With eps = 0 the only valid lists are the exact top-k sets (up to ties).  Order inside a list is
 * not part of the rule.  Returns the number of invalid lists over the active (token, head) pairs
 * of the sequences whose step is not 0. */
static double page_bound_abs_f64(const float* q, const float* lo, const float* hi, int d) {
  double acc = 0.0;
  for (int j = 0; j < d; ++j) {
    const double a = (double)q[j] * (double)lo[j], b = (double)q[j] * (double)hi[j];
    acc += fabs((a > b) ? a : b);
  }
  return acc;
}
static int cmp_double_desc(const void* a, const void* b) {
  const double x = *(const double*)a, y = *(const double*)b;
  return (x < y) - (x > y);
}
int64_t oracle_check_topk_relaxed(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                                  const int32_t* active_idx, const int32_t* n_active,
                                  const int32_t* step, int32_t k, const int32_t* topk_pages, double eps) {
  const int B = sh->block_size, Hq = sh->n_q_heads, d = sh->head_dim, Hkv = sh->n_kv_heads, G = Hq / Hkv;
  int64_t bad = 0;
  for (int s = 0; s < sh->batch; ++s) {
    if (step && step[s] == 0) continue;
    const int P = pages_of(kv->kv_len[s], sh->page_size);
    const int kk = k < P ? k : P;
    for (int a = 0; a < n_active[s]; ++a) {
      const int tok = active_idx[(int64_t)s * B + a];
      for (int h = 0; h < Hq; ++h) {
        const int32_t* list = topk_pages + (((int64_t)s * B + tok) * Hq + h) * k;
        double* u = (double*)malloc(sizeof(double) * (P > 0 ? P : 1));
        double* sorted = (double*)malloc(sizeof(double) * (P > 0 ? P : 1));
        char* seen = (char*)calloc(P > 0 ? P : 1, 1);
        float qv[512], lo[512], hi[512];
        const int64_t qo = (((int64_t)s * B + tok) * Hq + h) * d;
        for (int j = 0; j < d; ++j) qv[j] = ld_f32(q, sh->dtype, qo + j);
        double smax = 0.0;
        for (int p = 0; p < P; ++p) {
          const int32_t phys = kv->page_table[(int64_t)s * sh->max_pages_per_seq + p];
          const int64_t so = ((int64_t)phys * Hkv + h / G) * d;
          for (int j = 0; j < d; ++j) {
            lo[j] = ld_f32(kv->kmin, sh->dtype, so + j);
            hi[j] = ld_f32(kv->kmax, sh->dtype, so + j);
          }
          u[p] = page_bound_f64(qv, lo, hi, d);
          const double sa = page_bound_abs_f64(qv, lo, hi, d);
          if (sa > smax) smax = sa;
          sorted[p] = u[p];
        }
        qsort(sorted, P, sizeof(double), cmp_double_desc);
        int ok = 1;
        for (int j = 0; j < k; ++j) {
          const int32_t p = list[j];
          if (j < kk) {
            if (p < 0 || p >= P || seen[p]) { ok = 0; break; }
            seen[p] = 1;
            if (u[p] < sorted[kk - 1] - eps * smax) { ok = 0; break; }
          } else if (p != -1) {
            ok = 0;
            break;
          }
        }
        bad += ok ? 0 : 1;
        free(u); free(sorted); free(seen);
      }
    }
  }
  return bad;
}

/* ---------- Section 2.3 / 4.2: top-k pages for the active queries only ----------
 * I_{i,h} = the min(k, P_s) pages with the largest bound, ordered (bound descending, page
 * ascending).  Every (token, query head) is one query.  Sequences at step 0 are skipped. */
typedef struct { float u; int32_t p; } scored_t;
static int cmp_scored(const void* a, const void* b) {
  const scored_t *x = (const scored_t*)a, *y = (const scored_t*)b;
  if (x->u > y->u) return -1;
  if (x->u < y->u) return 1;
  return (x->p > y->p) - (x->p < y->p);
}

void oracle_page_scores_topk(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                             const int32_t* active_idx, const int32_t* n_active,
                             const int32_t* step, int32_t k, int32_t* topk_pages,
                             float* topk_scores) {
  const int B = sh->block_size, Hq = sh->n_q_heads;
  for (int s = 0; s < sh->batch; ++s) {
    if (step && step[s] == 0) continue;
    const int P = pages_of(kv->kv_len[s], sh->page_size);
    const int work = n_active[s] * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int w = 0; w < work; ++w) {
      const int tok = active_idx[(int64_t)s * B + w / Hq], h = w % Hq;
      float* u = (float*)malloc(sizeof(float) * (size_t)(P > 0 ? P : 1));
      scored_t* sc = (scored_t*)malloc(sizeof(scored_t) * (size_t)(P > 0 ? P : 1));
      oracle_page_scores_one(sh, q, kv, s, tok, h, u, NULL);
      for (int p = 0; p < P; ++p) { sc[p].u = u[p]; sc[p].p = p; }
      qsort(sc, (size_t)P, sizeof(scored_t), cmp_scored);
      const int64_t o = (((int64_t)s * B + tok) * Hq + h) * k;
      for (int j = 0; j < k; ++j) {
        topk_pages[o + j] = (j < P) ? sc[j].p : -1;
        if (topk_scores && j < P) topk_scores[o + j] = sc[j].u;
      }
      free(u);
      free(sc);
    }
  }
}

/* ---------- Selector variant: one list per (token, KV head) ---------------------------------
 * Section 2.3 calls the method independent of the selector.  With grouped-query attention the G
 * heads of a KV head read the same pages, so this variant scores a page once per KV head: the
 * pooled score is the largest of the G heads' upper bounds (each in the interface's fixed fp32
 * order), the k best pages by (pooled score descending, page ascending) are chosen, and every
 * head of the group receives that list.  With G = 1 it is oracle_page_scores_topk. */
void oracle_page_scores_topk_pooled(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                                    const int32_t* active_idx, const int32_t* n_active,
                                    const int32_t* step, int32_t k, int32_t* topk_pages,
                                    float* topk_scores) {
  const int B = sh->block_size, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
  for (int s = 0; s < sh->batch; ++s) {
    if (step && step[s] == 0) continue;
    const int P = pages_of(kv->kv_len[s], sh->page_size);
    const int work = n_active[s] * Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (int w = 0; w < work; ++w) {
      const int tok = active_idx[(int64_t)s * B + w / Hkv], kh = w % Hkv;
      float* u = (float*)malloc(sizeof(float) * (size_t)(P > 0 ? P : 1));
      scored_t* sc = (scored_t*)malloc(sizeof(scored_t) * (size_t)(P > 0 ? P : 1));
      for (int gi = 0; gi < G; ++gi) {
        oracle_page_scores_one(sh, q, kv, s, tok, kh * G + gi, u, NULL);
        for (int p = 0; p < P; ++p) {
          if (gi == 0 || u[p] > sc[p].u) sc[p].u = u[p];
          sc[p].p = p;
        }
      }
      qsort(sc, (size_t)P, sizeof(scored_t), cmp_scored);
      for (int gi = 0; gi < G; ++gi) {
        const int64_t o = (((int64_t)s * B + tok) * Hq + kh * G + gi) * k;
        for (int j = 0; j < k; ++j) {
          topk_pages[o + j] = (j < P) ? sc[j].p : -1;
          if (topk_scores && j < P) topk_scores[o + j] = sc[j].u;
        }
      }
      free(u);
      free(sc);
    }
  }
}

/* ---------- Section 4.2 / 4.4: I = union over active tokens (and the G heads of a KV head) ---- */
void oracle_page_union(const oracle_shape_t* sh, const int32_t* topk_pages,
                       const int32_t* active_idx, const int32_t* n_active, int32_t k,
                       const int32_t* kv_len, const int32_t* step, int32_t* union_pages,
                       int32_t* union_count) {
  const int B = sh->block_size, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
  const int Pmax = sh->max_pages_per_seq;
  char* mark = (char*)malloc((size_t)(Pmax > 0 ? Pmax : 1));
  for (int s = 0; s < sh->batch; ++s) {
    const int P = pages_of(kv_len[s], sh->page_size);
    for (int kh = 0; kh < Hkv; ++kh) {
      memset(mark, 0, (size_t)(Pmax > 0 ? Pmax : 1));
      if (step && step[s] == 0) {
        for (int p = 0; p < P; ++p) mark[p] = 1;
      } else {
        for (int a = 0; a < n_active[s]; ++a) {
          const int tok = active_idx[(int64_t)s * B + a];
          for (int gi = 0; gi < G; ++gi)
            for (int j = 0; j < k; ++j) {
              const int32_t p = topk_pages[(((int64_t)s * B + tok) * Hq + kh * G + gi) * k + j];
              if (p >= 0 && p < P) mark[p] = 1;
            }
        }
      }
      int cnt = 0;
      int32_t* out = union_pages + ((int64_t)s * Hkv + kh) * Pmax;
      for (int p = 0; p < P; ++p)
        if (mark[p]) out[cnt++] = p;
      union_count[(int64_t)s * Hkv + kh] = cnt;
      for (int p = cnt; p < Pmax; ++p) out[p] = -1;
    }
  }
  free(mark);
}

/* ---------- Section 2.2: log-normaliser of one query over a list of scores ----------
 * L = log sum_t exp(s_t); the maximum is subtracted inside the exponentials only to keep them
 * finite.  The output then is o = (1 / e^L) sum_t exp(s_t) v_t = sum_t exp(s_t - L) v_t. */
static void log_normaliser(const double* sc, int n, double* L) {
  if (n == 0) { *L = -INFINITY; return; }
  double M = sc[0];
  for (int t = 1; t < n; ++t) if (sc[t] > M) M = sc[t];
  double sum = 0.0;
  for (int t = 0; t < n; ++t) sum += exp(sc[t] - M);
  *L = M + log(sum);
}

/* Section 4.2: all queries of the active set attend over the shared union of their KV head;
 * update rule for tokens in A; tokens outside A keep (o_p, L_p) untouched (reuse rule). */
void oracle_sparse_prefix_attn(const oracle_shape_t* sh, const void* q, const oracle_kv_t* kv,
                               const int32_t* active_idx, const int32_t* n_active,
                               const int32_t* union_pages, const int32_t* union_count,
                               double* o_p, double* lse_p) {
  const int B = sh->block_size, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
  const int d = sh->head_dim, g = sh->page_size, Pmax = sh->max_pages_per_seq;
  for (int s = 0; s < sh->batch; ++s) {
    const int len = kv->kv_len[s];
    const int work = n_active[s] * Hq;
#pragma omp parallel for schedule(dynamic, 1)
    for (int w = 0; w < work; ++w) {
      const int tok = active_idx[(int64_t)s * B + w / Hq], h = w % Hq, kh = h / G;
      const int cnt = union_count[(int64_t)s * Hkv + kh];
      const int32_t* list = union_pages + ((int64_t)s * Hkv + kh) * Pmax;
      const int64_t qo = (((int64_t)s * B + tok) * Hq + h) * d;
      double* sc = (double*)malloc(sizeof(double) * (size_t)(cnt * g + 1));
      int64_t* voff = (int64_t*)malloc(sizeof(int64_t) * (size_t)(cnt * g + 1));
      int n = 0;
      for (int u = 0; u < cnt; ++u) {
        const int p = list[u];
        const int32_t phys = kv->page_table[(int64_t)s * Pmax + p];
        for (int t = 0; t < g && p * g + t < len; ++t) {
          const int64_t ko = kv_off(kv, phys, kh, t);
          double dot = 0.0;
          for (int j = 0; j < d; ++j) dot += ld(q, sh->dtype, qo + j) * ld(kv->k_pages, sh->dtype, ko + j);
          sc[n] = sh->sm_scale * dot;
          voff[n] = ko;
          ++n;
        }
      }
      double L;
      log_normaliser(sc, n, &L);
      double* o = o_p + qo;
      for (int j = 0; j < d; ++j) o[j] = 0.0;
      for (int t = 0; t < n; ++t) {
        const double pw = exp(sc[t] - L);
        for (int j = 0; j < d; ++j) o[j] += pw * ld(kv->v_pages, sh->dtype, voff[t] + j);
      }
      lse_p[((int64_t)s * B + tok) * Hq + h] = L;
      free(sc);
      free(voff);
    }
  }
}

/* ---------- Section 4.3: dense in-block attention, then the online-softmax merge ----------
 * (o_b, L_b) over the B block keys, bidirectional (no mask).  Since exp(s) V = e^L o for each part
 * (Section 2.2), the attention over prefix and block together is
 * L = log(e^{L_p} + e^{L_b}),  out = e^{L_p - L} o_p + e^{L_b - L} o_b. */
void oracle_block_attn_merge(const oracle_shape_t* sh, const void* q, const void* k_blk,
                             const void* v_blk, const double* o_p, const double* lse_p,
                             double* out, double* lse_out) {
  const int B = sh->block_size, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, G = Hq / Hkv;
  const int d = sh->head_dim;
  const int work = sh->batch * B * Hq;
#pragma omp parallel for schedule(static)
  for (int w = 0; w < work; ++w) {
    const int s = w / (B * Hq), i = (w / Hq) % B, h = w % Hq, kh = h / G;
    const int64_t qo = (((int64_t)s * B + i) * Hq + h) * d;
    double sc[ORACLE_MAX_BLOCK];
    for (int t = 0; t < B; ++t) {
      const int64_t ko = (((int64_t)s * B + t) * Hkv + kh) * d;
      double dot = 0.0;
      for (int j = 0; j < d; ++j) dot += ld(q, sh->dtype, qo + j) * ld(k_blk, sh->dtype, ko + j);
      sc[t] = sh->sm_scale * dot;
    }
    double Lb;
    log_normaliser(sc, B, &Lb);
    const double Lp = lse_p[((int64_t)s * B + i) * Hq + h];
    const double M = (Lp > Lb) ? Lp : Lb;
    const double L = M + log(exp(Lp - M) + exp(Lb - M));
    const double wp = exp(Lp - L), wb = exp(Lb - L);
    for (int j = 0; j < d; ++j) {
      double ob = 0.0;
      for (int t = 0; t < B; ++t)
        ob += exp(sc[t] - Lb) * ld(v_blk, sh->dtype, (((int64_t)s * B + t) * Hkv + kh) * d + j);
      out[qo + j] = wp * o_p[qo + j] + wb * ob;
    }
    if (lse_out) lse_out[((int64_t)s * B + i) * Hq + h] = L;
  }
}

/* ---------- Section 4.3 (keep the queries for the next step) and Section 2.1 (the cache grows
 * by the finalised block) ---------- */
void oracle_update_prefix_cache(const oracle_shape_t* sh, oracle_kv_t* kv, void* q_prev,
                                int32_t* step, const void* q, const void* k_blk,
                                const void* v_blk, int32_t finalize_block) {
  const int B = sh->block_size, Hq = sh->n_q_heads, Hkv = sh->n_kv_heads, d = sh->head_dim;
  const int g = sh->page_size;
  if (!finalize_block) {
    cp_elem(q_prev, 0, q, 0, sh->dtype, (int64_t)sh->batch * B * Hq * d);
    for (int s = 0; s < sh->batch; ++s) step[s] += 1;
    return;
  }
  for (int s = 0; s < sh->batch; ++s) {
    const int L0 = kv->kv_len[s];
    for (int t = 0; t < B; ++t) {
      const int pos = L0 + t, p = pos / g, slot = pos % g;
      const int32_t phys = kv->page_table[(int64_t)s * sh->max_pages_per_seq + p];
      for (int kh = 0; kh < Hkv; ++kh) {
        const int64_t src = (((int64_t)s * B + t) * Hkv + kh) * d;
        cp_elem(kv->k_pages, kv_off(kv, phys, kh, slot), k_blk, src, sh->dtype, d);
        cp_elem(kv->v_pages, kv_off(kv, phys, kh, slot), v_blk, src, sh->dtype, d);
      }
    }
    kv->kv_len[s] = L0 + B;
    for (int p = L0 / g; p <= (L0 + B - 1) / g; ++p) summarise_page(sh, kv, s, p);
    step[s] = 0;
  }
}
