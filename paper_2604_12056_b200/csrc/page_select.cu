// Stages 2 and 3 — QUEST page scores, top-k per active query, union per KV head
// (Section 2.3, Section 4.2, Section 4.4).
//
//   page_scores_kernel : each CTA reads the min/max keys of 64 pages of one (sequence, KV head)
//                        once and scores them against every active query of that KV head.  A page
//                        is handled by d/8 lanes: one 16-byte vector of kmin and kmax per lane
//                        (four pages per lane), a chain of 16 fused multiply-adds per lane and
//                        page (q+ kmax, q- kmin), then the butterfly over the lanes as a
//                        reduce-scatter over two query rows at a time: exactly the additions and
//                        the order the interface fixes, so the fp32 result is reproducible bit for bit.
//   topk_select_kernel : one 128-thread CTA per (sequence, active token, head); threshold search over
//                        64-bit keys (order-preserving score bits, inverted page id), see below.
//   topk_kernel        : budgets above 512 pages: one CTA per query sorts all keys with a
//                        shared-memory bitonic network.
//   union_kernel       : one CTA per (sequence, KV head) ORs the selected ids into a bitmap and
//                        emits the set bits in ascending order with a popcount scan.
#include <algorithm>

#include "kernels.h"

namespace losa {
namespace {

constexpr int kThreads = 256;
constexpr int kPagesPerCta = 64;
constexpr int kRowTile = 32;

// Eight consecutive elements as loaded, converted to fp32 later: lets several dependent-free loads
// be in flight before any of them is used.
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 u;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { u = *reinterpret_cast<const uint4*>(p); }
  __device__ __forceinline__ void zero() { u = make_uint4(0u, 0u, 0u, 0u); }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};
template <> struct Raw8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = *reinterpret_cast<const float4*>(p);
    b = *reinterpret_cast<const float4*>(p + 4);
  }
  __device__ __forceinline__ void zero() { a = make_float4(0.f, 0.f, 0.f, 0.f); b = a; }
  __device__ __forceinline__ void unpack(float (&v)[8]) const {
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
};

// A load whose issue point stays where it is written (it is requested ahead of the branch that
// decides whether it is needed).
__device__ __forceinline__ int ld_keep_s32(const int32_t* ptr) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(ptr));
  return v;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
page_scores_kernel(const T* __restrict__ q, const T* __restrict__ kmin, const T* __restrict__ kmax,
                   const int32_t* __restrict__ page_table, const int32_t* __restrict__ kv_len,
                   const int32_t* __restrict__ active_idx, const int32_t* __restrict__ n_active,
                   const int32_t* __restrict__ step, float* __restrict__ scores, int B, int Hq, int Hkv,
                   int g, int Pmax, int n_phys, int score_stride, int32_t* __restrict__ status) {
  grid_dep_wait();
  constexpr int LPP = D / 8;            // lanes per page
  constexpr int GROUPS = kThreads / LPP;
  constexpr int ITER = kPagesPerCta / GROUPS;
  constexpr int STG = (kRowTile * (D / 8) + kThreads - 1) / kThreads;   // staging items per thread and row tile
  const int s = blockIdx.z, kh = blockIdx.y, p0 = blockIdx.x * kPagesPerCta;
  const int tid = threadIdx.x;
  const int grp = tid / LPP, sub = tid % LPP;
  const int G = Hq / Hkv;
  // First round trip: the scalars, and with them - their addresses depend on nothing else - this
  // lane's page-table entries and the block positions of the query rows it may have to stage
  // (entries the scalars later rule out are read and dropped).
  int phys[ITER], tok0[STG];
#pragma unroll
  for (int it = 0; it < ITER; ++it) {
    const int p = p0 + grp * ITER + it;
    phys[it] = p < Pmax ? ld_keep_s32(page_table + static_cast<size_t>(s) * Pmax + p) : -1;
  }
#pragma unroll
  for (int i = 0; i < STG; ++i) {
    const int a = ((tid + i * kThreads) / (D / 8)) / G;
    tok0[i] = a < B ? ld_keep_s32(active_idx + s * B + a) : 0;
  }
  if (step && step[s] == 0) return;
  int P = pages_of(kv_len[s], g);
  if (P > Pmax) { set_status(status, LOSA_ERR_BOUNDS); P = Pmax; }    // a length beyond the page-table row
  if (p0 >= P) return;
  int na = n_active[s];
  na = na < 0 ? 0 : (na > B ? B : na);
  const int rows = na * G;
  if (rows == 0) return;

  // positive and negative parts of the staged queries, fp32: U = sum q+ kmax + q- kmin.  A row is
  // stored as two halves [half][lane chunk][4 floats] so that the d/8 lanes of a page read
  // consecutive 16-byte words (no bank conflicts): element j = 8*c + e sits at (e/4)*(D/2) + 4*c + e%4.
  __shared__ __align__(16) float qpos[kRowTile * D];
  __shared__ __align__(16) float qneg[kRowTile * D];
  const int np = min(kPagesPerCta, P - p0);

  // Second round trip: this lane's share of the pages' kmin / kmax (kept in registers for every
  // query row) and the query rows themselves.  Everything of a trip is requested before anything
  // of it is used.
  const int nr_first = min(kRowTile, rows);
  Raw8<T> klo[ITER], khi[ITER], q0[STG];
#pragma unroll
  for (int it = 0; it < ITER; ++it) {
    klo[it].zero();
    khi[it].zero();
    if (grp * ITER + it < np) {
      int ph = phys[it];
      if (ph < 0 || ph >= n_phys) { set_status(status, LOSA_ERR_BOUNDS); ph = 0; }
      const size_t so = (static_cast<size_t>(ph) * Hkv + kh) * D + sub * 8;
      klo[it].load(kmin + so);
      khi[it].load(kmax + so);
    }
  }
#pragma unroll
  for (int i = 0; i < STG; ++i) {
    const int idx = tid + i * kThreads;
    q0[i].zero();
    if (idx < nr_first * (D / 8)) {
      const int r = idx / (D / 8), ch = idx % (D / 8), gi = r % G;
      int tok = tok0[i];
      if (tok < 0 || tok >= B) { set_status(status, LOSA_ERR_BOUNDS); tok = 0; }
      q0[i].load(q + ((static_cast<size_t>(s) * B + tok) * Hq + kh * G + gi) * D + ch * 8);
    }
  }
  auto stage = [&](int r, int ch, const float (&v)[8]) {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int at = r * D + (e >> 2) * (D / 2) + ch * 4 + (e & 3);
      qpos[at] = fmaxf(v[e], 0.f);
      qneg[at] = fminf(v[e], 0.f);
    }
  };
  float lo[ITER][8], hi[ITER][8];
  for (int r0 = 0; r0 < rows; r0 += kRowTile) {
    const int nr = min(kRowTile, rows - r0);
    if (r0 == 0) {
#pragma unroll
      for (int i = 0; i < STG; ++i) {
        const int idx = tid + i * kThreads;
        if (idx < nr * (D / 8)) {
          float v[8];
          q0[i].unpack(v);
          stage(idx / (D / 8), idx % (D / 8), v);
        }
      }
#pragma unroll
      for (int it = 0; it < ITER; ++it) {
        klo[it].unpack(lo[it]);
        khi[it].unpack(hi[it]);
      }
    } else {
      for (int idx = tid; idx < nr * (D / 8); idx += kThreads) {
        const int r = idx / (D / 8), ch = idx % (D / 8);
        const int row = r0 + r, a = row / G, gi = row % G;
        int tok = active_idx[s * B + a];
        if (tok < 0 || tok >= B) { set_status(status, LOSA_ERR_BOUNDS); tok = 0; }
        float v[8];
        load8(q + ((static_cast<size_t>(s) * B + tok) * Hq + kh * G + gi) * D + ch * 8, v);
        stage(r, ch, v);
      }
    }
    __syncthreads();
    // Two query rows at a time: one load of a row's run feeds the chains of the ITER pages held in
    // registers.  A lane then has NV = 2 * ITER run sums, one per (page, row) pair; every pair needs
    // the butterfly c[i] += c[i ^ off] (off = LPP/2 .. 1) over the LPP lanes of its group.  Taken as
    // a reduce-scatter it costs NV shuffles per lane instead of NV * log2(LPP): at each level the
    // lane keeps the half of its values chosen by its own bit `off` and sends the other half; the
    // additions, and their order, are those of the plain butterfly (fp32 addition commutes), so the
    // result is the same bit for bit.  Lanes 2i and 2i+1 end with pair i = (page it = i / 2, row i % 2).
    constexpr int NV = 2 * ITER;
    static_assert(NV == LPP / 2, "one result per pair of lanes");
    int a = r0 / G, gi = r0 % G;          // row r0 + r = (active token a, head gi of the KV head), gi fastest
    for (int r = 0; r < nr; r += 2) {
      float v[NV];
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int rs = min(r + rr, nr - 1);         // an odd tail computes its last row twice and stores it once
        float qp[8], qn[8];
        *reinterpret_cast<float4*>(&qp[0]) = *reinterpret_cast<const float4*>(&qpos[rs * D + sub * 4]);
        *reinterpret_cast<float4*>(&qp[4]) = *reinterpret_cast<const float4*>(&qpos[rs * D + D / 2 + sub * 4]);
        *reinterpret_cast<float4*>(&qn[0]) = *reinterpret_cast<const float4*>(&qneg[rs * D + sub * 4]);
        *reinterpret_cast<float4*>(&qn[4]) = *reinterpret_cast<const float4*>(&qneg[rs * D + D / 2 + sub * 4]);
        float acc[ITER];
#pragma unroll
        for (int it = 0; it < ITER; ++it) acc[it] = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
          for (int it = 0; it < ITER; ++it) {
            acc[it] = __fmaf_rn(qp[j], hi[it][j], acc[it]);
            acc[it] = __fmaf_rn(qn[j], lo[it][j], acc[it]);
          }
        }
#pragma unroll
        for (int it = 0; it < ITER; ++it) v[it * 2 + rr] = acc[it];
      }
      {
        int n = NV;
#pragma unroll
        for (int off = LPP / 2; off >= 2; off >>= 1) {
          n >>= 1;
          const bool up = (sub & off) != 0;
#pragma unroll
          for (int k = 0; k < NV / 2; ++k) {
            if (k < n) {
              const float send = up ? v[k] : v[k + n];
              const float keep = up ? v[k + n] : v[k];
              v[k] = __fadd_rn(keep, __shfl_xor_sync(0xffffffffu, send, off));
            }
          }
        }
        v[0] = __fadd_rn(v[0], __shfl_xor_sync(0xffffffffu, v[0], 1));
      }
      const int i = sub >> 1, it = i >> 1, rr = i & 1, pl = grp * ITER + it;
      if ((sub & 1) == 0 && pl < np && r + rr < nr) {
        int a2 = a, g2 = gi + rr;
        if (g2 >= G) { g2 -= G; ++a2; }
        scores[((static_cast<size_t>(s) * B + a2) * Hq + kh * G + g2) * score_stride + p0 + pl] = __fadd_rn(v[0], 0.0f);
      }
      gi += 2;
      while (gi >= G) { gi -= G; ++a; }
    }
    __syncthreads();
  }
}

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
  const int kh = blockIdx.x, s = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = min(pages_of(kv_len[s], g), Pmax);
  const int W = (Pmax + 31) / 32;
  const int G = Hq / Hkv;
  const bool all = step && step[s] == 0;
  for (int w = tid; w < W; w += kThreads) {
    uint32_t v = 0;
    if (all) {
      const int lo = w * 32;
      v = (P >= lo + 32) ? 0xffffffffu : (P > lo ? ((1u << (P - lo)) - 1u) : 0u);
    }
    bitmap[w] = v;
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
  // each thread owns a contiguous run of words; exclusive scan of the per-thread popcounts
  const int per = (W + kThreads - 1) / kThreads;
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
  for (int w = 0; w < kThreads / 32; ++w) {
    if (w < warp) base += s_warp[w];
    total += s_warp[w];
  }
  int pos = base + inc - cnt;
  int32_t* out = union_pages + (static_cast<size_t>(s) * Hkv + kh) * Pmax;
  for (int w = w0; w < w1; ++w) {
    uint32_t v = bitmap[w];
    while (v) {
      const int b = __ffs(v) - 1;
      v &= v - 1;
      out[pos++] = w * 32 + b;
    }
  }
  for (int t = total + tid; t < Pmax; t += kThreads) out[t] = -1;
  if (tid == 0) union_count[s * Hkv + kh] = total;
}

template <typename T, int D>
void launch_scores(losa_ctx* c, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                   const int32_t* n_active, const int32_t* step, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  dim3 grid((sh.max_pages_per_seq + kPagesPerCta - 1) / kPagesPerCta, sh.n_kv_heads, sh.batch);
  launch_k(page_scores_kernel<T, D>, grid, kThreads, 0, st, 
      static_cast<const T*>(q), static_cast<const T*>(kv->kmin), static_cast<const T*>(kv->kmax),
      kv->page_table, kv->kv_len, active_idx, n_active, step,
      reinterpret_cast<float*>(c->ws + c->lay.scores), sh.block_size, sh.n_q_heads, sh.n_kv_heads,
      sh.page_size, sh.max_pages_per_seq, kv->n_phys_pages, c->lay.score_stride, status_ptr(c));
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
                                float* topk_scores_opt, cudaStream_t st, bool pooled) {
  const losa_shape_t& sh = c->shape;
  if (sh.max_pages_per_seq == 0) return LOSA_OK;
  const int pool = pooled ? sh.n_q_heads / sh.n_kv_heads : 1;
  const bool bf = sh.dtype == LOSA_BF16;
  if (bf && sh.head_dim == 128) launch_scores<__nv_bfloat16, 128>(c, q, kv, active_idx, n_active, step, st);
  else if (bf) launch_scores<__nv_bfloat16, 64>(c, q, kv, active_idx, n_active, step, st);
  else if (sh.head_dim == 128) launch_scores<float, 128>(c, q, kv, active_idx, n_active, step, st);
  else launch_scores<float, 64>(c, q, kv, active_idx, n_active, step, st);
  int32_t rc = after_launch(c);
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
