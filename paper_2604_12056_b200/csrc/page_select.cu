// Stages 2 and 3 — QUEST page scores, top-k per active query, union per KV head
// (Section 2.3, Section 4.2, Section 4.4).
//
//   (the page scores themselves are computed by the kernel in page_scores.cu)
//   topk_select_kernel : one 128-thread CTA per (sequence, active token, head); threshold search over
//                        64-bit keys (order-preserving score bits, inverted page id), see below.
//   topk_kernel        : budgets above 512 pages: one CTA per query sorts all keys with a
//                        shared-memory bitonic network.
//   topk_refine_kernel : bf16, k <= 512 (the default): candidates from tensor-core bounds, exact scores
//                        for those only; in the whole-step call it also writes stage 3's union.
//   union_kernel       : one CTA per (sequence, KV head) ORs the selected ids into a bitmap and
//                        emits the set bits in ascending order with a popcount scan.
#include <algorithm>

#include "kernels.h"

namespace losa {
namespace {

constexpr int kThreads = 256;

// One score row, or (pooled selector) the element-wise maximum of the `g` consecutive rows of a KV
// head's query heads.
template <bool POOLED>
struct RowView {
  const float* base;
  int g, stride;
  __device__ __forceinline__ float operator[](int p) const {
    float v = base[p];
    if (POOLED)
      for (int gi = 1; gi < g; ++gi) v = fmaxf(v, base[static_cast<size_t>(gi) * stride + p]);
    return v;
  }
};

__device__ __forceinline__ uint32_t order_bits(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float unorder_bits(uint32_t o) {
  return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}

__global__ void __launch_bounds__(kThreads)
topk_kernel(const float* __restrict__ scores, const int32_t* __restrict__ kv_len,
            const int32_t* __restrict__ active_idx, const int32_t* __restrict__ n_active,
            const int32_t* __restrict__ step, int32_t* __restrict__ topk_pages,
            float* __restrict__ topk_scores, int B, int Hq, int g, int k, int Pmax, int score_stride, int pool,
            int32_t* __restrict__ status) {
  grid_dep_wait();
  extern __shared__ __align__(16) unsigned long long keys[];
  const int h = blockIdx.x * pool, a = blockIdx.y, s = blockIdx.z;   // pooled: first head of the KV head
  if (step && step[s] == 0) return;
  int na = n_active[s];
  na = na > B ? B : na;
  if (a >= na) return;
  int tok = active_idx[s * B + a];
  if (tok < 0 || tok >= B) { set_status(status, LOSA_ERR_BOUNDS); return; }
  int P = pages_of(kv_len[s], g);
  if (P > Pmax) { set_status(status, LOSA_ERR_BOUNDS); P = Pmax; }
  const int tid = threadIdx.x;
  int n = 2;
  while (n < P) n <<= 1;
  const RowView<true> sc{scores + ((static_cast<size_t>(s) * B + a) * Hq + h) * score_stride, pool, score_stride};
  for (int p = tid; p < n; p += kThreads)
    keys[p] = (p < P) ? ((static_cast<unsigned long long>(order_bits(sc[p])) << 32) |
                         static_cast<unsigned long long>(0xffffffffu - static_cast<uint32_t>(p)))
                      : 0ull;
  __syncthreads();
  // bitonic network, descending
  for (int k2 = 2; k2 <= n; k2 <<= 1) {
    for (int j = k2 >> 1; j > 0; j >>= 1) {
      for (int t = tid; t < (n >> 1); t += kThreads) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int x = i | j;
        const unsigned long long ka = keys[i], kb = keys[x];
        const bool desc = (i & k2) == 0;
        if ((ka < kb) == desc) { keys[i] = kb; keys[x] = ka; }
      }
      __syncthreads();
    }
  }
  for (int gi = 0; gi < pool; ++gi) {                 // pooled: every head of the group gets the list
    const size_t o = ((static_cast<size_t>(s) * B + tok) * Hq + h + gi) * k;
    for (int j = tid; j < k; j += kThreads) {
      if (j < P) {
        const unsigned long long key = keys[j];
        topk_pages[o + j] = static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(key));
        if (topk_scores) topk_scores[o + j] = unorder_bits(static_cast<uint32_t>(key >> 32));
      } else {
        topk_pages[o + j] = -1;
      }
    }
  }
}

// ---- top-k by threshold search: one small CTA per query, O(P) work ---------------------------
// Keys are (order-preserving score bits, inverted page id), all distinct, so "the k largest keys"
// is the required answer with ties already broken.  The CTA histograms the score bits of the
// still-undecided range into 256 equal-width bins, finds the bin holding the k-th largest, takes
// every key above that bin, and either finishes by sorting "taken + threshold bin" (a few dozen
// keys) or narrows the range to the threshold bin and repeats.  A range of one value means the
// remaining candidates tie on the score: the lowest page ids win, taken in page order.
constexpr int kSelCap = 512;     // candidate keys a warp can sort; also the largest k of this path
constexpr int kSelBins = 256;

__device__ __forceinline__ unsigned long long make_key(uint32_t ob, int p) {
  return (static_cast<unsigned long long>(ob) << 32) |
         static_cast<unsigned long long>(0xffffffffu - static_cast<uint32_t>(p));
}

// One CTA of kSelThreads per query.  Thread t owns keys p = t + kSelThreads * i; with CACHED
// (P <= kSelThreads * kSelPerThread) their order bits stay in registers for the whole selection.
constexpr int kSelThreads = 128;
constexpr int kSelPerThread = 8;
constexpr int kSelSlots = 8;        // CTAs per (sequence, head): active slots are dealt out round-robin

template <bool CACHED, typename Row, typename F>
__device__ __forceinline__ void for_each_key(const uint32_t (&cache)[kSelPerThread], const Row& row,
                                             int P, int tid, F&& f) {
  if (CACHED) {
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i) {
      const int p = tid + kSelThreads * i;
      if (p < P) f(cache[i], p);
    }
  } else {
    for (int p = tid; p < P; p += kSelThreads) f(order_bits(row[p]), p);
  }
}

template <bool CACHED, typename Row>
__device__ __forceinline__ void topk_select_body(const Row& row, int P, int kk, int k,
                                                 int32_t* out_pages, float* out_scores, int n_out) {
  __shared__ unsigned long long cand[kSelCap];
  __shared__ int hist[kSelBins];
  __shared__ uint32_t s_red[2][kSelThreads / 32];
  __shared__ int s_ncand, s_bstar, s_above, s_thr;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t cache[kSelPerThread];
  if (CACHED) {
#pragma unroll
    for (int i = 0; i < kSelPerThread; ++i) {
      const int p = tid + kSelThreads * i;
      cache[i] = p < P ? order_bits(row[p]) : 0u;
    }
  }
  uint32_t lo = 0xffffffffu, hi = 0u;
  for_each_key<CACHED, Row>(cache, row, P, tid, [&](uint32_t ob, int) { lo = min(lo, ob); hi = max(hi, ob); });
  lo = __reduce_min_sync(0xffffffffu, lo);
  hi = __reduce_max_sync(0xffffffffu, hi);
  if (lane == 0) { s_red[0][warp] = lo; s_red[1][warp] = hi; }
  if (tid == 0) s_ncand = 0;
  __syncthreads();
#pragma unroll
  for (int w = 0; w < kSelThreads / 32; ++w) { lo = min(lo, s_red[0][w]); hi = max(hi, s_red[1][w]); }
  int need = kk;
  while (need > 0) {
    if (lo == hi) {
      // every remaining candidate has the same score: lowest pages first, in page order (rare;
      // one warp walks the pages so that the order is kept)
      if (warp == 0) {
        int ncand = s_ncand;
        const unsigned below = (1u << lane) - 1u;
        for (int base = 0; base < P && need > 0; base += 32) {
          const int p = base + lane;
          const bool hit = p < P && order_bits(row[p]) == lo;
          const unsigned bal = __ballot_sync(0xffffffffu, hit);
          const int rank = __popc(bal & below);
          if (hit && rank < need) cand[ncand + rank] = make_key(lo, p);
          const int taken = min(need, __popc(bal));
          ncand += taken;
          need -= taken;
        }
        if (lane == 0) s_ncand = ncand;
      }
      break;
    }
    const int width = 32 - __clz(hi - lo);           // bits needed for hi - lo  (>= 1)
    const int shift = width > 8 ? width - 8 : 0;      // (ob - lo) >> shift is in [0, 255]
    for (int b = tid; b < kSelBins; b += kSelThreads) hist[b] = 0;
    __syncthreads();
    for_each_key<CACHED, Row>(cache, row, P, tid, [&](uint32_t ob, int) {
      if (ob >= lo && ob <= hi) atomicAdd(&hist[(ob - lo) >> shift], 1);
    });
    __syncthreads();
    if (warp == 0) {
      // lane owns bins [8*lane, 8*lane+8); suffix sums over lanes locate the threshold bin
      int c[8], tot = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) { c[e] = hist[8 * lane + e]; tot += c[e]; }
      int suf = tot;                                   // inclusive suffix: lanes >= this one
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += t;
      }
      const int above_lanes = suf - tot;
      if (above_lanes < need && need <= suf) {
        int run = above_lanes;
#pragma unroll
        for (int e = 7; e >= 0; --e) {
          if (run < need && need <= run + c[e]) { s_bstar = 8 * lane + e; s_above = run; s_thr = c[e]; }
          run += c[e];
        }
      }
    }
    __syncthreads();
    const int bstar = s_bstar, cnt_above = s_above, cnt_thr = s_thr;
    const bool finish = s_ncand + cnt_above + cnt_thr <= kSelCap;
    __syncthreads();                                   // everyone has read s_ncand before it moves
    // take the keys above the threshold bin (and, when finishing, the threshold bin itself); the
    // order inside cand does not matter: it is sorted below
    for_each_key<CACHED, Row>(cache, row, P, tid, [&](uint32_t ob, int p) {
      if (ob >= lo && ob <= hi) {
        const int bin = static_cast<int>((ob - lo) >> shift);
        if (bin > bstar || (finish && bin == bstar)) cand[atomicAdd(&s_ncand, 1)] = make_key(ob, p);
      }
    });
    if (finish) break;
    need -= cnt_above;
    const uint32_t nlo = lo + (static_cast<uint32_t>(bstar) << shift);
    const unsigned long long top = static_cast<unsigned long long>(nlo) + ((1ull << shift) - 1ull);
    hi = top < hi ? static_cast<uint32_t>(top) : hi;
    lo = nlo;
    __syncthreads();
  }
  __syncthreads();
  // sort the candidates (descending) and emit the first kk
  const int ncand = s_ncand;
  int n2 = 2;
  while (n2 < ncand) n2 <<= 1;
  for (int i = ncand + tid; i < n2; i += kSelThreads) cand[i] = 0ull;
  __syncthreads();
  for (int k2 = 2; k2 <= n2; k2 <<= 1) {
    for (int j = k2 >> 1; j > 0; j >>= 1) {
      for (int t = tid; t < (n2 >> 1); t += kSelThreads) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int x = i | j;
        const unsigned long long ka = cand[i], kb = cand[x];
        if ((ka < kb) == ((i & k2) == 0)) { cand[i] = kb; cand[x] = ka; }
      }
      __syncthreads();
    }
  }
  for (int gi = 0; gi < n_out; ++gi) {               // pooled: the list goes to every head of the group
    for (int j = tid; j < k; j += kSelThreads) {
      if (j < kk) {
        const unsigned long long key = cand[j];
        out_pages[gi * k + j] = static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(key));
        if (out_scores) out_scores[gi * k + j] = unorder_bits(static_cast<uint32_t>(key >> 32));
      } else {
        out_pages[gi * k + j] = -1;
      }
    }
  }
}


// ---- bf16 fast path: candidates from tensor-core bounds, exact scores for the candidates only ----
// The page score in the order the interface fixes, by four lanes (u = lane % 4; qs: [q+ (D) | q- (D)]
// fp32 in shared memory): lane u runs the chains of runs u, u + 4(, u + 8, u + 12) - 16 fused
// multiply-adds per run of 8 dimensions - and the butterfly c[i] += c[i ^ off], off = D/16 .. 1, is
// taken inside the lane while off >= 4 and with two shuffles below that.  All four lanes return it.
template <int D>
__device__ __forceinline__ float exact_score4(const float* __restrict__ qs, const __nv_bfloat16* __restrict__ lo_p,
                                              const __nv_bfloat16* __restrict__ hi_p, int u) {
  constexpr int RPL = D / 32;      // runs per lane
  uint4 lo_raw[RPL], hi_raw[RPL];  // requested together, converted run by run
#pragma unroll
  for (int w = 0; w < RPL; ++w) {
    lo_raw[w] = __ldg(reinterpret_cast<const uint4*>(lo_p + 8 * (u + 4 * w)));
    hi_raw[w] = __ldg(reinterpret_cast<const uint4*>(hi_p + 8 * (u + 4 * w)));
  }
  float c[RPL];
#pragma unroll
  for (int w = 0; w < RPL; ++w) {
    const int t = u + 4 * w;
    const uint32_t lw[4] = {lo_raw[w].x, lo_raw[w].y, lo_raw[w].z, lo_raw[w].w};
    const uint32_t hw[4] = {hi_raw[w].x, hi_raw[w].y, hi_raw[w].z, hi_raw[w].w};
    float acc = 0.f;
#pragma unroll
    for (int j4 = 0; j4 < 2; ++j4) {
      const float4 qp = *reinterpret_cast<const float4*>(qs + 8 * t + 4 * j4);
      const float4 qn = *reinterpret_cast<const float4*>(qs + D + 8 * t + 4 * j4);
      acc = __fmaf_rn(qp.x, __uint_as_float(hw[2 * j4] << 16), acc);
      acc = __fmaf_rn(qn.x, __uint_as_float(lw[2 * j4] << 16), acc);
      acc = __fmaf_rn(qp.y, __uint_as_float(hw[2 * j4] & 0xffff0000u), acc);
      acc = __fmaf_rn(qn.y, __uint_as_float(lw[2 * j4] & 0xffff0000u), acc);
      acc = __fmaf_rn(qp.z, __uint_as_float(hw[2 * j4 + 1] << 16), acc);
      acc = __fmaf_rn(qn.z, __uint_as_float(lw[2 * j4 + 1] << 16), acc);
      acc = __fmaf_rn(qp.w, __uint_as_float(hw[2 * j4 + 1] & 0xffff0000u), acc);
      acc = __fmaf_rn(qn.w, __uint_as_float(lw[2 * j4 + 1] & 0xffff0000u), acc);
    }
    c[w] = acc;
  }
  float v;
  if constexpr (RPL == 4) v = __fadd_rn(__fadd_rn(c[0], c[2]), __fadd_rn(c[1], c[3]));   // off = 8, then off = 4
  else v = __fadd_rn(c[0], c[1]);                                                         // off = 4
  v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, 2));
  v = __fadd_rn(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return __fadd_rn(v, 0.0f);
}

struct RefineParams {
  float2* bounds;                 // (A - delta, A + delta) per (row, page); reused as fp32 score rows by the fallback
  const __nv_bfloat16* q;
  const __nv_bfloat16* kmin;
  const __nv_bfloat16* kmax;
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* active_idx;
  const int32_t* n_active;
  const int32_t* step;
  int32_t* topk_pages;
  float* topk_scores;
  int32_t* status;
  int N, B, Hq, Hkv, g, k, score_stride, Pmax, n_phys;
  // stage 3 inside this kernel (whole-step call): the lists are ORed into one bitmap per (sequence, KV
  // head) as they are emitted, and the last CTA of a (sequence, KV head) to finish writes the union.
  // union_bits == nullptr: lists only.
  uint32_t* union_bits;           // [N][Hkv][W] words, all zero between launches
  unsigned int* union_tickets;    // [N][Hkv] arrival counters, self-resetting
  int32_t* union_pages;
  int32_t* union_count;
  int W;                          // words per bitmap, ceil(Pmax / 32) <= kSelBins
};

// The set bits of a bitmap in shared memory, ascending, then -1 up to Pmax; the count.  All NT threads
// of the CTA call it; s_warp: NT / 32 ints of shared memory.
template <int NT>
__device__ __forceinline__ void union_emit(const uint32_t* bitmap, int W, int Pmax, int32_t* __restrict__ out,
                                           int32_t* __restrict__ count, int* s_warp) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // each thread owns a contiguous run of words; exclusive scan of the per-thread popcounts
  const int per = (W + NT - 1) / NT;
  const int w0 = tid * per, w1 = min(W, w0 + per);
  int cnt = 0;
  for (int w = w0; w < w1; ++w) cnt += __popc(bitmap[w]);
  int inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += t;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  int base = 0, total = 0;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) {
    if (w < warp) base += s_warp[w];
    total += s_warp[w];
  }
  int pos = base + inc - cnt;
  for (int w = w0; w < w1; ++w) {
    uint32_t v = bitmap[w];
    while (v) {
      const int b = __ffs(v) - 1;
      v &= v - 1;
      out[pos++] = w * 32 + b;
    }
  }
  for (int t = total + tid; t < Pmax; t += NT) out[t] = -1;
  if (tid == 0) *count = total;
}

__device__ __forceinline__ uint32_t prefix_word(int w, int P) {   // word w of the bitmap "pages 0 .. P-1"
  const int lo = w * 32;
  return (P >= lo + 32) ? 0xffffffffu : (P > lo ? ((1u << (P - lo)) - 1u) : 0u);
}

// One CTA of kSelThreads per (sequence, head, 1/8 of the active slots).  Per query: tau = lower edge
// of the histogram bin that holds the k-th largest LOWER bound; every page whose UPPER bound reaches
// tau is a candidate (a superset of the exact top-k, ties included: the exact score lies between the
// bounds); exact scores in the fixed order for the candidates (four lanes each), sort, emit.  More
// than kSelCap candidates (possible only when most pages nearly tie): exact scores for every page
// into the score row, then the plain threshold search.
// POOLED (one list per KV head, Section 4.2's selector with the group's maximum as the page score):
// a CTA serves the G heads of a KV head at once.  max over the heads of the lower (upper) bounds is
// a lower (upper) bound of the pooled score, so the same search applies to those; a candidate's
// exact score is the largest of its G exact scores; the list goes to every head of the group.
constexpr int kMaxPool = 16;     // heads per KV head the interface admits

template <int D, bool POOLED>
__global__ void __launch_bounds__(kSelThreads, POOLED ? 4 : 6)
topk_refine_kernel(RefineParams p) {
  const int qid = blockIdx.x;
  const int pool = POOLED ? p.Hq / p.Hkv : 1, Hl = p.Hq / pool;
  const int h = (qid % Hl) * pool, s = (qid / Hl) % p.N, j0 = qid / (Hl * p.N);   // pooled: h = the group's first head
  // With stage 3 inside (whole-step call) the next kernel is stage 4, and the chain of launches
  // guarantees that the step counters are final before any CTA of this kernel runs.  On a first step
  // stage 4 is not released early: its CTAs then take the SMs in launch order once this grid has
  // drained, which its dense pass is measurably faster with (one sequence: 38 against 46 us).
  bool first_step;
  if (p.union_bits) {
    first_step = p.step && __ldcg(p.step + s) == 0;
    if (!first_step) grid_dep_trigger();
  } else {
    grid_dep_trigger();
  }
  grid_dep_wait();
  if (!p.union_bits) first_step = p.step && p.step[s] == 0;
  __shared__ __align__(16) float qs[(POOLED ? kMaxPool : 1) * 2 * D];
  __shared__ __align__(16) unsigned long long ckey[kSelCap];
  __shared__ int cpage[kSelCap];
  __shared__ int hist[kSelBins];
  __shared__ uint32_t s_red[2][kSelThreads / 32];
  __shared__ int s_ncand, s_bstar;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kh = h / (p.Hq / p.Hkv);
  int na = first_step ? 0 : p.n_active[s];
  na = na > p.B ? p.B : na;
  if (na <= 0) {
    // no lists for this sequence: on the first step of a block the union is the whole prefix, with
    // no active token it is empty; written by the first CTA of the (sequence, KV head)
    if (!p.union_bits || j0 != 0 || h != kh * (p.Hq / p.Hkv)) return;
    const int P0 = first_step ? min(pages_of(p.kv_len[s], p.g), p.Pmax) : 0;
    uint32_t* bm = reinterpret_cast<uint32_t*>(hist);
    for (int w = tid; w < p.W; w += kSelThreads) bm[w] = prefix_word(w, P0);
    __syncthreads();
    union_emit<kSelThreads>(bm, p.W, p.Pmax, p.union_pages + (static_cast<size_t>(s) * p.Hkv + kh) * p.Pmax,
                            p.union_count + s * p.Hkv + kh, reinterpret_cast<int*>(s_red[0]));
    return;
  }
  if (j0 >= na) return;                                  // no slot for this CTA
  int P = pages_of(p.kv_len[s], p.g);
  if (P > p.Pmax) { if (tid == 0) set_status(p.status, LOSA_ERR_BOUNDS); P = p.Pmax; }
  const int kk = min(p.k, P);
  uint32_t* bits = p.union_bits ? p.union_bits + (static_cast<size_t>(s) * p.Hkv + kh) * p.W : nullptr;
  auto mark = [&](int pg) { if (bits) atomicOr(&bits[pg >> 5], 1u << (pg & 31)); };
  const __nv_bfloat16* lo_base = p.kmin + static_cast<size_t>(kh) * D;
  const __nv_bfloat16* hi_base = p.kmax + static_cast<size_t>(kh) * D;
  const int u = lane & 3;
  for (int a = j0; a < na; a += kSelSlots) {
    const int tok = p.active_idx[s * p.B + a];
    if (tok < 0 || tok >= p.B) { if (tid == 0) set_status(p.status, LOSA_ERR_BOUNDS); continue; }
    float2* row2 = p.bounds + ((static_cast<size_t>(s) * p.B + a) * p.Hq + h) * p.score_stride;
    const size_t o = ((static_cast<size_t>(s) * p.B + tok) * p.Hq + h) * p.k;
    int32_t* out_pages = p.topk_pages + o;
    float* out_scores = p.topk_scores ? p.topk_scores + o : nullptr;
    // the bounds of this thread's pages: one round trip, kept in registers when the prefix has at
    // most kSelThreads * kSelPerThread pages
    const bool cached = P <= kSelThreads * kSelPerThread;
    if constexpr (POOLED) {
      if (!cached) {
        // the passes below read the row several times: pool once, into the group's first row (the
        // rows are scratch, this CTA is their only reader, and a thread reads back only what it wrote)
        constexpr int U = 4;                                   // pages per thread whose loads are in flight together
        for (int p0 = tid; p0 < P; p0 += kSelThreads * U) {
          float2 v[U];
#pragma unroll
          for (int e = 0; e < U; ++e) v[e] = p0 + e * kSelThreads < P ? row2[p0 + e * kSelThreads] : make_float2(0.f, 0.f);
          for (int gi = 1; gi < pool; ++gi) {
            float2 w[U];
#pragma unroll
            for (int e = 0; e < U; ++e)
              w[e] = p0 + e * kSelThreads < P ? row2[static_cast<size_t>(gi) * p.score_stride + p0 + e * kSelThreads]
                                              : make_float2(0.f, 0.f);
#pragma unroll
            for (int e = 0; e < U; ++e) { v[e].x = fmaxf(v[e].x, w[e].x); v[e].y = fmaxf(v[e].y, w[e].y); }
          }
#pragma unroll
          for (int e = 0; e < U; ++e)
            if (p0 + e * kSelThreads < P) row2[p0 + e * kSelThreads] = v[e];
        }
      }
    }
    uint32_t lbc[kSelPerThread], ubc[kSelPerThread];
    if (cached) {
      float2 bv[kSelPerThread];
#pragma unroll
      for (int i = 0; i < kSelPerThread; ++i) {
        const int pg = tid + kSelThreads * i;
        bv[i] = pg < P ? row2[pg] : make_float2(0.f, 0.f);
      }
      if constexpr (POOLED) {
        for (int gi = 1; gi < pool; ++gi) {
          float2 bg[kSelPerThread];
#pragma unroll
          for (int i = 0; i < kSelPerThread; ++i) {
            const int pg = tid + kSelThreads * i;
            bg[i] = pg < P ? row2[static_cast<size_t>(gi) * p.score_stride + pg] : make_float2(0.f, 0.f);
          }
#pragma unroll
          for (int i = 0; i < kSelPerThread; ++i) {
            bv[i].x = fmaxf(bv[i].x, bg[i].x);
            bv[i].y = fmaxf(bv[i].y, bg[i].y);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < kSelPerThread; ++i) {
        lbc[i] = order_bits(bv[i].x);
        ubc[i] = order_bits(bv[i].y);
      }
    }
    auto for_each_page = [&](auto&& f) {        // f(lower bits, upper bits, page)
      if (cached) {
#pragma unroll
        for (int i = 0; i < kSelPerThread; ++i) {
          const int pg = tid + kSelThreads * i;
          if (pg < P) f(lbc[i], ubc[i], pg);
        }
      } else {
        for (int pg = tid; pg < P; pg += kSelThreads) {
          const float2 bv = row2[pg];                  // pooled: already the group's maximum
          f(order_bits(bv.x), order_bits(bv.y), pg);
        }
      }
    };
    // the query, split into its positive and negative parts
    for (int j = tid; j < pool * D; j += kSelThreads) {       // the group's heads are consecutive in q
      const float v = __bfloat162float(p.q[((static_cast<size_t>(s) * p.B + tok) * p.Hq + h) * D + j]);
      const int gi = j / D, d = j % D;
      qs[gi * 2 * D + d] = fmaxf(v, 0.f);
      qs[gi * 2 * D + D + d] = fminf(v, 0.f);
    }
    if (tid == 0) s_ncand = 0;
    for (int b = tid; b < kSelBins; b += kSelThreads) hist[b] = 0;
    // ---- tau
    uint32_t tau = 0u;
    if (kk < P) {
      uint32_t lo = 0xffffffffu, hi = 0u;
      for_each_page([&](uint32_t lb, uint32_t, int) { lo = min(lo, lb); hi = max(hi, lb); });
      lo = __reduce_min_sync(0xffffffffu, lo);
      hi = __reduce_max_sync(0xffffffffu, hi);
      if (lane == 0) { s_red[0][warp] = lo; s_red[1][warp] = hi; }
      __syncthreads();
#pragma unroll
      for (int w = 0; w < kSelThreads / 32; ++w) { lo = min(lo, s_red[0][w]); hi = max(hi, s_red[1][w]); }
      if (lo < hi) {
        const int width = 32 - __clz(hi - lo);
        const int shift = width > 8 ? width - 8 : 0;
        for_each_page([&](uint32_t lb, uint32_t, int) { atomicAdd(&hist[(lb - lo) >> shift], 1); });
        __syncthreads();
        if (warp == 0) {
          int c[8], tot = 0;
#pragma unroll
          for (int e = 0; e < 8; ++e) { c[e] = hist[8 * lane + e]; tot += c[e]; }
          int suf = tot;
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_down_sync(0xffffffffu, suf, off);
            if (lane + off < 32) suf += t;
          }
          const int above_lanes = suf - tot;
          if (above_lanes < kk && kk <= suf) {
            int run = above_lanes;
#pragma unroll
            for (int e = 7; e >= 0; --e) {
              if (run < kk && kk <= run + c[e]) s_bstar = 8 * lane + e;
              run += c[e];
            }
          }
        }
        __syncthreads();
        tau = lo + (static_cast<uint32_t>(s_bstar) << shift);
      } else {
        tau = lo;
      }
    } else {
      __syncthreads();
    }
    // ---- candidates: pages whose upper bound reaches tau
    for_each_page([&](uint32_t, uint32_t ub, int pg) {
      if (ub >= tau) {
        const int i = atomicAdd(&s_ncand, 1);
        if (i < kSelCap) cpage[i] = pg;
      }
    });
    __syncthreads();
    const int ncand = s_ncand;
    auto phys_of = [&](int pg) {
      int ph = __ldg(p.page_table + static_cast<size_t>(s) * p.Pmax + pg);
      if (ph < 0 || ph >= p.n_phys) { set_status(p.status, LOSA_ERR_BOUNDS); ph = 0; }
      return ph;
    };
    auto exact_at = [&](int ph) {                 // called by the four lanes of a group with the same page
      const size_t so = static_cast<size_t>(ph) * p.Hkv * D;
      float e = exact_score4<D>(qs, lo_base + so, hi_base + so, u);
      if constexpr (POOLED)
        for (int gi = 1; gi < pool; ++gi) e = fmaxf(e, exact_score4<D>(qs + gi * 2 * D, lo_base + so, hi_base + so, u));
      return e;
    };
    if (ncand > kSelCap) {
      float* row = reinterpret_cast<float*>(row2);             // the bounds are not needed any more
      for (int p0 = 0; p0 < P; p0 += kSelThreads / 4) {          // whole warps: the shuffles need all lanes
        const int pg = min(p0 + tid / 4, P - 1);
        const float e = exact_at(phys_of(pg));
        if (u == 0 && p0 + tid / 4 < P) row[pg] = e;
      }
      __syncthreads();
      const RowView<false> rv{row, 1, p.score_stride};
      topk_select_body<false>(rv, P, kk, p.k, out_pages, out_scores, pool);
      __syncthreads();
      if (bits)
        for (int j = tid; j < kk; j += kSelThreads) mark(out_pages[j]);     // this CTA's own stores
      continue;
    }
    // a group of four lanes per candidate, 32 candidates per round; the physical page ids of four
    // rounds are requested together (one round trip instead of four)
    constexpr int kPer = kSelThreads / 4, kAhead = 4;
    for (int i0 = 0; i0 < ncand; i0 += kPer * kAhead) {
      int pgs[kAhead], phs[kAhead];
#pragma unroll
      for (int r = 0; r < kAhead; ++r) {
        pgs[r] = cpage[min(i0 + r * kPer + tid / 4, ncand - 1)];
        phs[r] = phys_of(pgs[r]);
      }
#pragma unroll
      for (int r = 0; r < kAhead; ++r) {
        if (i0 + r * kPer < ncand) {                     // uniform over the CTA
          const float e = exact_at(phs[r]);
          const int i = i0 + r * kPer + tid / 4;
          if (u == 0 && i < ncand) ckey[i] = make_key(order_bits(e), pgs[r]);
        }
      }
    }
    // ---- order the candidates (descending) and emit the first kk
    __syncthreads();
    if (ncand <= kSelThreads) {
      // few candidates (the usual case): a candidate's position is the number of larger keys (all
      // keys differ); one candidate per thread, the keys are read as broadcasts, four at a time
      if ((tid & ~31) < ncand) {                       // whole warps without a candidate skip the count
        const unsigned long long mine = tid < ncand ? ckey[tid] : ~0ull;
        int rank = 0;
        const int n4 = ncand & ~3;
        for (int i = 0; i < n4; i += 4) {
          const ulonglong2 k01 = *reinterpret_cast<const ulonglong2*>(&ckey[i]);
          const ulonglong2 k23 = *reinterpret_cast<const ulonglong2*>(&ckey[i + 2]);
          rank += (k01.x > mine ? 1 : 0) + (k01.y > mine ? 1 : 0) + (k23.x > mine ? 1 : 0) + (k23.y > mine ? 1 : 0);
        }
        for (int i = n4; i < ncand; ++i) rank += ckey[i] > mine ? 1 : 0;
        if (tid < ncand && rank < kk) {
          const int pg = static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(mine));
          for (int gi = 0; gi < pool; ++gi) {
            out_pages[gi * p.k + rank] = pg;
            if (out_scores) out_scores[gi * p.k + rank] = unorder_bits(static_cast<uint32_t>(mine >> 32));
          }
          mark(pg);
        }
      }
      for (int gi = 0; gi < pool; ++gi)
        for (int j = kk + tid; j < p.k; j += kSelThreads) out_pages[gi * p.k + j] = -1;
    } else {
      int n2 = 2;
      while (n2 < ncand) n2 <<= 1;
      for (int i = ncand + tid; i < n2; i += kSelThreads) ckey[i] = 0ull;
      __syncthreads();
      for (int k2 = 2; k2 <= n2; k2 <<= 1) {
        for (int j = k2 >> 1; j > 0; j >>= 1) {
          for (int t = tid; t < (n2 >> 1); t += kSelThreads) {
            const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
            const int x = i | j;
            const unsigned long long ka = ckey[i], kb = ckey[x];
            if ((ka < kb) == ((i & k2) == 0)) { ckey[i] = kb; ckey[x] = ka; }
          }
          __syncthreads();
        }
      }
      for (int gi = 0; gi < pool; ++gi) {
        for (int j = tid; j < p.k; j += kSelThreads) {
          if (j < kk) {
            const unsigned long long key = ckey[j];
            out_pages[gi * p.k + j] = static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(key));
            if (out_scores) out_scores[gi * p.k + j] = unorder_bits(static_cast<uint32_t>(key >> 32));
            if (gi == 0) mark(static_cast<int32_t>(0xffffffffu - static_cast<uint32_t>(key)));
          } else {
            out_pages[gi * p.k + j] = -1;
          }
        }
      }
    }
    __syncthreads();                               // the shared state is reused by the next slot
  }
  if (!bits) return;
  // ---- stage 3: the last CTA of this (sequence, KV head) writes the union
  __syncthreads();                                 // every thread's marks precede ...
  if (tid == 0) {
    __threadfence();                               // ... this fence (cumulative), which precedes the ticket
    // CTAs of this (sequence, KV head) that hold a slot: all of them arrive here
    const unsigned int n_grp = static_cast<unsigned int>((p.Hq / p.Hkv / pool) * min(na, static_cast<int>(gridDim.x) / (Hl * p.N)));
    s_bstar = atomicInc(&p.union_tickets[s * p.Hkv + kh], n_grp - 1) == n_grp - 1 ? 1 : 0;
  }
  __syncthreads();
  if (!s_bstar) return;
  __threadfence();
  uint32_t* bm = reinterpret_cast<uint32_t*>(hist);
  for (int w = tid; w < p.W; w += kSelThreads) {
    bm[w] = atomicExch(bits + w, 0u);              // the marks were made in L2; all zero again for the next launch
  }
  __syncthreads();
  union_emit<kSelThreads>(bm, p.W, p.Pmax, p.union_pages + (static_cast<size_t>(s) * p.Hkv + kh) * p.Pmax,
                          p.union_count + s * p.Hkv + kh, reinterpret_cast<int*>(s_red[0]));
}

template <bool POOLED>
__global__ void __launch_bounds__(kSelThreads)
topk_select_kernel(float* __restrict__ scores, const int32_t* __restrict__ kv_len,
                   const int32_t* __restrict__ active_idx, const int32_t* __restrict__ n_active,
                   const int32_t* __restrict__ step, int32_t* __restrict__ topk_pages,
                   float* __restrict__ topk_scores, int N, int B, int Hq, int g, int k, int Pmax, int score_stride, int pool,
                   int32_t* __restrict__ status) {
  grid_dep_trigger();
  grid_dep_wait();
  // A CTA serves the active slots a = j, j + kSelSlots, ... of one (sequence, head): launching a CTA
  // costs about as much as an idle CTA's whole life, and most of the B slots are idle on most steps.
  // pool > 1 (pooled selector): one list per KV head from the maximum of its `pool` heads' rows
  const int qid = blockIdx.x, Hl = Hq / pool;
  const int h = (qid % Hl) * pool, s = (qid / Hl) % N, j = qid / (Hl * N);
  if (step && step[s] == 0) return;
  int na = n_active[s];
  na = na > B ? B : na;
  int P = pages_of(kv_len[s], g);
  if (P > Pmax) { if (threadIdx.x == 0) set_status(status, LOSA_ERR_BOUNDS); P = Pmax; }
  const int kk = min(k, P);
  for (int a = j; a < na; a += kSelSlots) {
    const int tok = active_idx[s * B + a];
    if (tok < 0 || tok >= B) { if (threadIdx.x == 0) set_status(status, LOSA_ERR_BOUNDS); continue; }
    RowView<POOLED> row{scores + ((static_cast<size_t>(s) * B + a) * Hq + h) * score_stride, pool, score_stride};
    const size_t o = ((static_cast<size_t>(s) * B + tok) * Hq + h) * k;
    if (P <= kSelThreads * kSelPerThread) {
      topk_select_body<true>(row, P, kk, k, topk_pages + o, topk_scores ? topk_scores + o : nullptr, pool);
    } else {
      if (POOLED && pool > 1) {
        // the selection reads the row several times: pool once, into the group's first row (the
        // score rows are scratch and this CTA is the only reader of these)
        float* first = scores + ((static_cast<size_t>(s) * B + a) * Hq + h) * score_stride;
        constexpr int U = 4;                                   // pages per thread whose loads are in flight together
        for (int p0 = threadIdx.x; p0 < P; p0 += kSelThreads * U) {
          float v[U];
#pragma unroll
          for (int u = 0; u < U; ++u) v[u] = p0 + u * kSelThreads < P ? row[p0 + u * kSelThreads] : 0.f;
#pragma unroll
          for (int u = 0; u < U; ++u)
            if (p0 + u * kSelThreads < P) first[p0 + u * kSelThreads] = v[u];
        }
        __syncthreads();
        row.g = 1;
      }
      topk_select_body<false>(row, P, kk, k, topk_pages + o, topk_scores ? topk_scores + o : nullptr, pool);
    }
    __syncthreads();                                 // the shared state is reused by the next slot
  }
}

__global__ void __launch_bounds__(kThreads)
union_kernel(const int32_t* __restrict__ topk_pages, const int32_t* __restrict__ active_idx,
             const int32_t* __restrict__ n_active, const int32_t* __restrict__ kv_len,
             const int32_t* __restrict__ step, int32_t* __restrict__ union_pages,
             int32_t* __restrict__ union_count, int B, int Hq, int Hkv, int g, int k, int Pmax,
             int32_t* __restrict__ status) {
  grid_dep_trigger();                              // the stage-4 kernel sets up its barriers and tensor memory meanwhile
  grid_dep_wait();
  extern __shared__ uint32_t bitmap[];
  __shared__ int s_warp[kThreads / 32];
  const int kh = blockIdx.x, s = blockIdx.y, tid = threadIdx.x;
  const int P = min(pages_of(kv_len[s], g), Pmax);
  const int W = (Pmax + 31) / 32;
  const int G = Hq / Hkv;
  const bool all = step && step[s] == 0;
  for (int w = tid; w < W; w += kThreads) {
    bitmap[w] = all ? prefix_word(w, P) : 0u;
  }
  __syncthreads();
  if (!all) {
    int na = n_active[s];
    na = na < 0 ? 0 : (na > B ? B : na);
    const int per_tok = G * k;
    // two dependent reads per entry (block position of the active slot, then the list entry): the
    // positions are staged once, and the list entries are requested four at a time
    __shared__ int s_tok[LOSA_MAX_BLOCK];
    for (int a = tid; a < na; a += kThreads) s_tok[a] = active_idx[s * B + a];
    __syncthreads();
    constexpr int U = 4;
    const int total = na * per_tok;
    for (int base = tid; base < total; base += kThreads * U) {
      int pv[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int idx = base + u * kThreads;
        pv[u] = -1;
        if (idx < total) {
          const int a = idx / per_tok, rem = idx % per_tok, gi = rem / k, j = rem % k;
          const int tok = s_tok[a];
          if (tok < 0 || tok >= B) { set_status(status, LOSA_ERR_BOUNDS); continue; }
          pv[u] = topk_pages[((static_cast<size_t>(s) * B + tok) * Hq + kh * G + gi) * k + j];
        }
      }
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int p = pv[u];
        if (p < 0) continue;
        if (p >= P) { set_status(status, LOSA_ERR_BOUNDS); continue; }
        atomicOr(&bitmap[p >> 5], 1u << (p & 31));
      }
    }
    __syncthreads();
  }
  union_emit<kThreads>(bitmap, W, Pmax, union_pages + (static_cast<size_t>(s) * Hkv + kh) * Pmax,
                       union_count + s * Hkv + kh, s_warp);
}

int pow2_at_least(int x) {
  int n = 2;
  while (n < x) n <<= 1;
  return n;
}

}  // namespace

int32_t topk_max_sortable(const losa_ctx* c) {
  int n = 2;
  while (static_cast<size_t>(n) * 2 * sizeof(unsigned long long) <= static_cast<size_t>(c->max_smem_optin)) n <<= 1;
  return n;
}

int32_t launch_page_scores_topk(losa_ctx* c, const void* q, const losa_kv_t* kv,
                                const int32_t* active_idx, const int32_t* n_active,
                                const int32_t* step, int32_t k, int32_t* topk_pages,
                                float* topk_scores_opt, cudaStream_t st, int selector, bool after_stage1,
                                int32_t* union_pages, int32_t* union_count, bool* union_done) {
  if (union_done) *union_done = false;
  const losa_shape_t& sh = c->shape;
  if (sh.max_pages_per_seq == 0) return LOSA_OK;
  const bool pooled = selector == kSelectorPooled;
  const int pool = pooled ? sh.n_q_heads / sh.n_kv_heads : 1;
  const bool bf = sh.dtype == LOSA_BF16;
  if (bf && (selector == kSelectorExact || pooled) && k <= kSelCap) {
    // bf16, exact lists (per query head, or per KV head from the group's maximum): bounds from the
    // tensor cores, exact scores for the candidates only
    int32_t rc = launch_page_bounds(c, q, kv, active_idx, n_active, step, st, false, after_stage1);
    if (rc != LOSA_OK) return rc;
    RefineParams rp;
    rp.bounds = reinterpret_cast<float2*>(c->ws + c->lay.scores);
    rp.q = static_cast<const __nv_bfloat16*>(q);
    rp.kmin = static_cast<const __nv_bfloat16*>(kv->kmin);
    rp.kmax = static_cast<const __nv_bfloat16*>(kv->kmax);
    rp.page_table = kv->page_table;
    rp.kv_len = kv->kv_len;
    rp.active_idx = active_idx;
    rp.n_active = n_active;
    rp.step = step;
    rp.topk_pages = topk_pages;
    rp.topk_scores = topk_scores_opt;
    rp.status = status_ptr(c);
    rp.N = sh.batch; rp.B = sh.block_size; rp.Hq = sh.n_q_heads; rp.Hkv = sh.n_kv_heads; rp.g = sh.page_size;
    rp.k = k; rp.score_stride = c->lay.score_stride; rp.Pmax = sh.max_pages_per_seq; rp.n_phys = kv->n_phys_pages;
    rp.W = (sh.max_pages_per_seq + 31) / 32;
    const bool with_union = union_pages && union_count && union_done && rp.W <= kSelBins;
    rp.union_bits = with_union ? reinterpret_cast<uint32_t*>(c->ws + c->lay.union_bits) : nullptr;
    rp.union_tickets = reinterpret_cast<unsigned int*>(c->ws + c->lay.union_tickets);
    rp.union_pages = union_pages;
    rp.union_count = union_count;
    if (with_union) *union_done = true;
    const int queries = sh.batch * std::min<int>(sh.block_size, kSelSlots) * (sh.n_q_heads / pool);
    if (pool > 1) {
      if (sh.head_dim == 128) launch_k(topk_refine_kernel<128, true>, queries, kSelThreads, 0, st, rp);
      else launch_k(topk_refine_kernel<64, true>, queries, kSelThreads, 0, st, rp);
    } else {
      if (sh.head_dim == 128) launch_k(topk_refine_kernel<128, false>, queries, kSelThreads, 0, st, rp);
      else launch_k(topk_refine_kernel<64, false>, queries, kSelThreads, 0, st, rp);
    }
    return after_launch(c);
  }
  int32_t rc = selector == kSelectorMma ? launch_page_bounds(c, q, kv, active_idx, n_active, step, st, true, after_stage1)
                                        : launch_page_scores(c, q, kv, active_idx, n_active, step, st);
  if (rc != LOSA_OK) return rc;

  float* sc = reinterpret_cast<float*>(c->ws + c->lay.scores);
  if (k <= kSelCap) {
    const int queries = sh.batch * std::min<int>(sh.block_size, kSelSlots) * (sh.n_q_heads / pool);
    if (pool > 1)
      launch_k(topk_select_kernel<true>, queries, kSelThreads, 0, st,
          sc, kv->kv_len, active_idx, n_active, step, topk_pages, topk_scores_opt, sh.batch, sh.block_size,
          sh.n_q_heads, sh.page_size, k, sh.max_pages_per_seq, c->lay.score_stride, pool, status_ptr(c));
    else
      launch_k(topk_select_kernel<false>, queries, kSelThreads, 0, st,
          sc, kv->kv_len, active_idx, n_active, step, topk_pages, topk_scores_opt, sh.batch, sh.block_size,
          sh.n_q_heads, sh.page_size, k, sh.max_pages_per_seq, c->lay.score_stride, 1, status_ptr(c));
    return after_launch(c);
  }
  // budgets beyond what one warp can sort: whole-list bitonic sort, one CTA per query
  const size_t smem = static_cast<size_t>(pow2_at_least(sh.max_pages_per_seq)) * sizeof(unsigned long long);
  if (smem > 48 * 1024)
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(topk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  dim3 grid(sh.n_q_heads / pool, sh.block_size, sh.batch);
  launch_k(topk_kernel, grid, kThreads, smem, st, sc, kv->kv_len, active_idx, n_active, step, topk_pages,
                                            topk_scores_opt, sh.block_size, sh.n_q_heads, sh.page_size,
                                            k, sh.max_pages_per_seq, c->lay.score_stride, pool, status_ptr(c));
  return after_launch(c);
}

int32_t launch_page_union(losa_ctx* c, const int32_t* topk_pages, const int32_t* active_idx,
                          const int32_t* n_active, int32_t k, const int32_t* kv_len,
                          const int32_t* step, int32_t* union_pages, int32_t* union_count,
                          cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  const size_t smem = static_cast<size_t>((sh.max_pages_per_seq + 31) / 32 + 1) * sizeof(uint32_t);
  dim3 grid(sh.n_kv_heads, sh.batch);
  launch_k(union_kernel, grid, kThreads, smem, st, topk_pages, active_idx, n_active, kv_len, step, union_pages,
                                             union_count, sh.block_size, sh.n_q_heads, sh.n_kv_heads,
                                             sh.page_size, k, sh.max_pages_per_seq, status_ptr(c));
  return after_launch(c);
}

}  // namespace losa
