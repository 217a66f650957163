// Stage 2, first half — QUEST page scores for the active queries (Section 2.3, Section 4.2).
//
// U(p) = sum_j max(q_j,0) kmax[p,j] + min(q_j,0) kmin[p,j] decides integer page ids, so it is
// evaluated in fp32 in the one order the interface fixes: per run of 8 consecutive j a chain of 16
// fused multiply-adds (q+ kmax, then q- kmin, j ascending) from +0; the d/8 run sums combined by the
// butterfly c[i] += c[i ^ off], off = d/16 .. 1; finally + 0.0f.
//
// Persistent kernel, one CTA of eight warps per SM.  The pages of all (sequence, KV head) pairs form
// one flat list that is cut into equal contiguous ranges, one per CTA; a CTA walks its range in
// tiles of TP pages of one (sequence, KV head), warp w taking pages [w WP, (w+1) WP) of every tile.
//   loading : each warp copies its own pages' kmax / kmin into its slice of a ring of shared-memory
//             stages with asynchronous 16-byte copies (cp.async; d elements of one summary are
//             consecutive lanes, so every copy instruction is coalesced), NS - 1 tiles ahead, the
//             page-table entries one tile further ahead.  A warp only ever reads what it copied
//             itself, so completion is the warp's own cp.async group count: no producer warp, no
//             barrier, no spinning.
//   compute : a lane owns the runs u and u + d/16 of PG pages (two runs whose sums the butterfly's
//             first level adds) and keeps them in registers as pairs, so the two chains advance
//             together in one packed instruction (fma.rn.f32x2): half the issue slots of the scalar
//             form, the same roundings.  Query rows are staged once per (sequence, KV head) as
//             positive / negative parts in the same pair layout (bf16 inputs stay bf16 in shared
//             memory, two to a word: max(q, 0) and min(q, 0) of a bf16 are bf16; the shared-memory
//             pipe, which also carries the shuffles, is what bounds this kernel).  The first level
//             of the butterfly is the add of a pair's halves; the other levels run over the d/16
//             lanes of a page as a reduce-scatter over the 2 PG (page, row) pairs a lane works on:
//             same additions, same order, 2 PG - 1 shuffles per pass instead of 2 PG log2(d/16).
#include "kernels.h"

namespace losa {
namespace {

constexpr int kPsWarps = 8;
constexpr int kPsThreads = kPsWarps * 32;
constexpr int kPsRowTile = 32;                      // query rows staged at a time
constexpr int kPsSeqStage = 4;                      // sequences whose active lists are cached in shared memory
constexpr int kPsMaxStages = 4;
constexpr int kPsSmemBudget = 232448;               // 227 KB opt-in limit per CTA

template <typename T, int D, int PG>
struct PsCfg {
  static constexpr int LPP = D / 16;                      // lanes per page
  static constexpr int GPW = 32 / LPP;                    // page groups per warp
  static constexpr int WP = GPW * PG;                     // pages per warp and tile
  static constexpr int TP = kPsWarps * WP;                // pages per tile
  static constexpr int HALF_BYTES = D * static_cast<int>(sizeof(T));   // kmax (or kmin) of one page and KV head
  static constexpr int PAGE_BYTES = 2 * HALF_BYTES;
  static constexpr int STAGE_BYTES = TP * PAGE_BYTES;
  static constexpr int QBUF_BYTES = 2 * kPsRowTile * D * static_cast<int>(sizeof(T));   // q+ and q- of one row tile
  static constexpr int NP = 2 * PG;                       // (page, row) pairs a lane works on per pass
  static constexpr int CH = HALF_BYTES / 16;              // 16-byte chunks of one summary
  static constexpr int RPI = 32 / CH;                     // summaries one warp-wide copy instruction covers
  static constexpr int NI = 2 * WP / RPI;                 // copy instructions per warp and tile
  static_assert(WP <= 32 && NP >= LPP / 2 && CH <= 32, "tile / reduce-scatter shape");
};

constexpr int ps_tail_bytes(int n_seq) {
  // prefix [n_seq + 1] | active counts [n_seq] | cached active lists
  return 16 + 4 * (n_seq + 1) + 4 * n_seq + 4 * kPsSeqStage * LOSA_MAX_BLOCK + 4 * n_seq;   // ... | pages per sequence
}

struct PsParams {
  const void* q;
  const void* kmin;
  const void* kmax;
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* active_idx;
  const int32_t* n_active;
  const int32_t* step;
  float* scores;
  int32_t* status;
  int N, B, Hq, Hkv, G, g, Pmax, n_phys, score_stride, n_ctas, n_stages;
  int early;   // the kernel before this one in the stream is stage 1 of the same step: the list and the first copies may be taken before it ends
  int tile_pages;   // tensor-core bounds kernel: pages per tile of this launch (16 .. 128, chosen on the host)
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most `pending` of this thread's newest copy groups are still in flight
__device__ __forceinline__ void cp_async_wait_pending(int pending) {
  switch (pending) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
  }
}

// 8 consecutive elements from shared memory as fp32
__device__ __forceinline__ void ld8(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 a = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void ld8(const float* p, float (&v)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// Walk of a CTA's item range [lo, hi) in tiles: item = (sequence s, KV head kh, logical page p),
// sequence-major, then KV head, then page; a tile never leaves its (s, kh) nor exceeds TP pages.
struct TileWalk {
  const int* pre;     // shared: exclusive prefix of the sequences' page counts, pre[N] = total
  int Hkv, TP, hi;
  int cur, s;
  int kh, p0, np;     // the current tile
  bool first_of_pair; // the tile is the CTA's first of this (s, kh)
  int last_pair;
  __device__ __forceinline__ void init(const int* pre_, int Hkv_, int TP_, int lo, int hi_) {
    pre = pre_; Hkv = Hkv_; TP = TP_; hi = hi_; cur = lo; s = 0; last_pair = -1; np = 0;
  }
  __device__ __forceinline__ bool next() {
    cur += np;
    if (cur >= hi) return false;
    while (static_cast<long long>(Hkv) * pre[s + 1] <= cur) ++s;
    const int Ps = pre[s + 1] - pre[s];
    const int off = cur - Hkv * pre[s];
    kh = off / Ps;
    p0 = off % Ps;
    np = min(min(TP, Ps - p0), hi - cur);
    const int pair = s * Hkv + kh;
    first_of_pair = pair != last_pair;
    last_pair = pair;
    return true;
  }
};

// The same walk over a list that counts TILES: a (sequence, KV head) with P pages has nt = ceil(P / TP)
// tiles of ceil(P / nt) pages each (the last one shorter), so every CTA gets whole tiles and the
// CTAs differ by at most one tile - a tile costs about the same whatever it holds (a chain of
// dependent latencies), and a range cut in the middle of tiles has one or two more of them.
struct TileWalkEven {
  const int* pre;     // shared: exclusive prefix of the sequences' tile counts per KV head
  const int* pages;   // shared: pages per sequence
  int Hkv, TP, hi;
  int cur, s;
  int kh, p0, np;     // the current tile
  __device__ __forceinline__ void init(const int* pre_, const int* pages_, int Hkv_, int TP_, int lo, int hi_) {
    pre = pre_; pages = pages_; Hkv = Hkv_; TP = TP_; hi = hi_; cur = lo - 1; s = 0; np = 0;
  }
  __device__ __forceinline__ bool next() {
    if (++cur >= hi) return false;
    while (static_cast<long long>(Hkv) * pre[s + 1] <= cur) ++s;
    const int nt = pre[s + 1] - pre[s], off = cur - Hkv * pre[s], P = pages[s];
    kh = off / nt;
    const int ts = (P + nt - 1) / nt;
    p0 = (off % nt) * ts;
    np = min(ts, P - p0);
    return true;
  }
};

// Common prologue of the page-score kernels (all threads of the CTA): the number of pages to score
// per sequence (none on a first step, none without active tokens) and its exclusive prefix into
// pre[0 .. N], the clamped active counts into na_s, this CTA's range [lo, hi) of the flat
// (sequence, KV head, page) list, and the active lists of the first kPsSeqStage sequences of that
// range into tok_s.  Returns false when the range is empty.  The caller synchronises the CTA before
// reading tok_s.
// The work list: pages of every sequence that is past its first step, whatever its number of
// active tokens (a sequence without any is walked without arithmetic), so that the list - and the
// first copies - depend on nothing stage 1 writes.  Reads bypass L1 (they may run beside the
// previous kernel).
// tile_pages > 0: the list counts tiles of at most that many pages (TileWalkEven) and pages_s
// receives the page count of every sequence.
__device__ __forceinline__ bool ps_list(const PsParams& p, int* pre, int& lo, int& hi, int& s_lo, int tile_pages = 0,
                                        int* pages_s = nullptr) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (warp == 0) {
    int run = 0;
    for (int b0 = 0; b0 < p.N; b0 += 32) {
      const int s = b0 + lane;
      int c = 0;
      if (s < p.N) {
        const bool first_step = p.step && __ldcg(p.step + s) == 0;
        int P = pages_of(__ldcg(p.kv_len + s), p.g);
        if (P > p.Pmax) { set_status(p.status, LOSA_ERR_BOUNDS); P = p.Pmax; }   // a length beyond the page-table row
        c = (first_step || P < 0) ? 0 : P;
        if (pages_s) pages_s[s] = c;
        if (tile_pages > 0) c = (c + tile_pages - 1) / tile_pages;
      }
      int inc = c;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      if (s < p.N) pre[s] = run + inc - c;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (lane == 0) pre[p.N] = run;
  }
  __syncthreads();
  const long long T_all = static_cast<long long>(p.Hkv) * pre[p.N];
  lo = static_cast<int>(cta_lo(T_all, blockIdx.x, p.n_ctas));
  hi = static_cast<int>(cta_lo(T_all, blockIdx.x + 1, p.n_ctas));
  if (lo >= hi) return false;
  s_lo = 0;
  while (static_cast<long long>(p.Hkv) * pre[s_lo + 1] <= lo) ++s_lo;
  return true;
}
// What stage 1 wrote: the clamped numbers of active tokens, and the active lists of the first few
// sequences of this CTA's range (the caller synchronises the CTA afterwards).
__device__ __forceinline__ void ps_active(const PsParams& p, int* na_s, int* tok_s, int s_lo) {
  for (int s = threadIdx.x; s < p.N; s += blockDim.x) {
    const int na = p.n_active[s];
    na_s[s] = na < 0 ? 0 : (na > p.B ? p.B : na);
  }
  for (int i = threadIdx.x; i < kPsSeqStage * p.B; i += blockDim.x) {
    const int s = s_lo + i / p.B;
    tok_s[i] = s < p.N ? p.active_idx[s * p.B + i % p.B] : -1;
  }
}

template <typename T, int D, int PG>
__global__ void __launch_bounds__(kPsThreads, 1) page_scores_stream_kernel(PsParams p) {
  using C = PsCfg<T, D, PG>;
  constexpr int LPP = C::LPP, TP = C::TP, NP = C::NP, WP = C::WP;
  extern __shared__ uint8_t ps_smem[];
  const uint32_t raw = smem_u32(ps_smem);
  const uint32_t base = (raw + 127u) & ~127u;
  uint8_t* gen = ps_smem + (base - raw);
  const int NS = p.n_stages;
  T* qpos = reinterpret_cast<T*>(gen + static_cast<size_t>(NS) * C::STAGE_BYTES);
  T* qneg = qpos + kPsRowTile * D;
  int* pre = reinterpret_cast<int*>(qneg + kPsRowTile * D);
  int* na_s = pre + p.N + 1;
  int* tok_s = na_s + p.N;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  grid_dep_trigger();
  grid_dep_wait();
  int lo, hi, s_lo;
  if (!ps_list(p, pre, lo, hi, s_lo)) return;                        // whole CTA: nothing in its range
  ps_active(p, na_s, tok_s, s_lo);
  // block position of active slot a of sequence s
  auto token_of = [&](int s, int a) {
    int tok = (s >= s_lo && s < s_lo + kPsSeqStage) ? tok_s[(s - s_lo) * p.B + a] : p.active_idx[s * p.B + a];
    if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); tok = 0; }
    return tok;
  };
  const T* qg = static_cast<const T*>(p.q);
  const T* kmaxg = static_cast<const T*>(p.kmax);
  const T* kming = static_cast<const T*>(p.kmin);
  const int u = lane % LPP, grp = lane / LPP;
  const uint32_t warp_off = static_cast<uint32_t>(warp) * WP * C::PAGE_BYTES;   // this warp's slice of a stage

  // ---- loading pipeline of this warp: page-table entry of lane j's page (j < WP) one tile ahead of
  //      the copies, the copies NS - 1 tiles ahead of the arithmetic
  TileWalk w_ids, w_copy, w;
  w_ids.init(pre, p.Hkv, TP, lo, hi);
  w_copy.init(pre, p.Hkv, TP, lo, hi);
  w.init(pre, p.Hkv, TP, lo, hi);
  auto request_id = [&]() {                          // entry of this lane's page in the next tile of w_ids (0 when there is none)
    int id = 0;
    if (w_ids.next()) {
      const int pl = warp * WP + lane;
      if (lane < WP && pl < w_ids.np) {
        id = __ldg(p.page_table + static_cast<size_t>(w_ids.s) * p.Pmax + w_ids.p0 + pl);
        if (id < 0 || id >= p.n_phys) { set_status(p.status, LOSA_ERR_BOUNDS); id = 0; }
      }
    }
    return id;
  };
  auto copy_tile = [&](int id, int stage) {          // the next tile of w_copy into `stage` (nothing when there is none); always one group
    if (w_copy.next()) {
      const uint32_t dst = base + static_cast<uint32_t>(stage) * C::STAGE_BYTES + warp_off;
      const int c = lane % C::CH, sub = lane / C::CH;
      constexpr int EPC = 16 / static_cast<int>(sizeof(T));
#pragma unroll
      for (int i = 0; i < C::NI; ++i) {
        const int row = i * C::RPI + sub, pl = row >> 1, a = row & 1;     // page of the warp's slice, 0 = kmax / 1 = kmin
        const int ph = __shfl_sync(0xffffffffu, id, pl);
        if (warp * WP + pl < w_copy.np) {
          const T* src = (a ? kming : kmaxg) + (static_cast<size_t>(ph) * p.Hkv + w_copy.kh) * D + c * EPC;
          cp_async16(dst + pl * C::PAGE_BYTES + a * C::HALF_BYTES + c * 16, src);
        }
      }
    }
    cp_async_commit();
  };
  int id_next = request_id();
  for (int i = 0; i < NS - 1; ++i) {
    const int id = id_next;
    id_next = request_id();
    copy_tile(id, i);
  }
  __syncthreads();                                   // the cached active lists are in place

  // q+ / q- of one run (8 elements j = 8 rho .. 8 rho + 7) of row r into the pair layout.  Lane
  // u = rho % LPP works on the pair {run u, run u + LPP}; h = rho / LPP says which half this run is.
  //   bf16: a row is D/2 words, word (jj / 4) * (4 LPP) + 4 u + jj % 4 holds element jj of both runs
  //         (low half: run u), so a lane's four words of a chunk are one 16-byte read and the LPP
  //         lanes of a page read consecutive 16-byte words;
  //   fp32: a row is D floats, float (jj / 2) * (4 LPP) + 4 u + 2 (jj % 2) + h.
  auto put_run = [&](int r, int rho, const float (&v)[8]) {
    const int uu = rho % LPP, h = rho / LPP;
#pragma unroll
    for (int jj = 0; jj < 8; ++jj) {
      const float vp = fmaxf(v[jj], 0.f), vn = fminf(v[jj], 0.f);
      if constexpr (sizeof(T) == 2) {
        const int at = r * D + 2 * ((jj >> 2) * (4 * LPP) + 4 * uu + (jj & 3)) + h;
        qpos[at] = __float2bfloat16_rn(vp);          // exact: v is a bf16 value
        qneg[at] = __float2bfloat16_rn(vn);
      } else {
        const int at = r * D + (jj >> 1) * (4 * LPP) + 4 * uu + 2 * (jj & 1) + h;
        qpos[at] = vp;
        qneg[at] = vn;
      }
    }
  };
  // rows r0 .. r0 + nr - 1 of (sequence s, KV head kh) from global memory into the staging buffers (all threads)
  auto stage_rows = [&](int s, int kh, int r0, int nr) {
    for (int idx = tid; idx < nr * (D / 8); idx += kPsThreads) {
      const int r = idx / (D / 8), rho = idx % (D / 8), row = r0 + r;
      const int tok = token_of(s, row / p.G);
      float v[8];
      load8(qg + ((static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + row % p.G) * D + rho * 8, v);
      put_run(r, rho, v);
    }
  };
  // Staging on demand (all threads, same arguments): a new (sequence, KV head), or another row tile
  // when a pair has more rows than one staging holds (every token active).  The first tile's rows
  // are staged before the loop, while the first copies are still in flight.
  int staged_pair = -1, staged_r0 = -1;
  auto ensure_rows = [&](int s, int kh, int r0, int nr) {
    const int pair = s * p.Hkv + kh;
    if (pair == staged_pair && r0 == staged_r0) return;
    __syncthreads();
    stage_rows(s, kh, r0, nr);
    __syncthreads();
    staged_pair = pair;
    staged_r0 = r0;
  };
  {
    TileWalk first;
    first.init(pre, p.Hkv, TP, lo, hi);
    if (first.next()) ensure_rows(first.s, first.kh, 0, min(kPsRowTile, na_s[first.s] * p.G));
  }

  // ---- reduce-scatter set-up.  After the add of a pair's halves (butterfly offset d/16) a lane
  // holds one partial sum for each of its NP = 2 PG (page, row) pairs; the remaining offsets
  // d/32 .. 1 pair the lanes u ^ LPP/2, u ^ LPP/4, .., u ^ 1.  As a reduce-scatter a lane keeps half
  // of its values at every level and sends the other half, so a pass costs NP - 1 shuffles; once a
  // single value is left the level is the plain exchange (both lanes end with the same sum).  Which
  // half is kept is a matter of naming: a lane whose bit is set holds its pages in an order with
  // the level's page bit flipped, or takes the pass's two rows the other way round, so that
  // everyone keeps the low half of the array.  The additions and their order are those of the
  // plain butterfly (fp32 addition commutes).
  constexpr int LV = LPP == 8 ? 3 : 2;                // levels over lanes (LPP = 2^LV)
  constexpr int LOGNP = NP == 8 ? 3 : 2;              // NP = 2^LOGNP
  constexpr int NF = (NP >> LV) > 0 ? (NP >> LV) : 1; // complete sums a lane ends up with
  int xperm = 0;                                      // page-order flip of this lane
  bool rowswap = false, stores = true;                // the lane takes the rows the other way round / is not a duplicate
#pragma unroll
  for (int l = 0; l < LV; ++l) {
    const int mask = (LPP / 2) >> l;
    const bool set = (u & mask) != 0;
    if (l < LOGNP) {
      const int b = LOGNP - 1 - l;                    // bit of the pair index 2 i + rr this level splits on
      if (b >= 1) { if (set) xperm ^= 1 << (b - 1); }
      else rowswap = set;
    } else if (set) {
      stores = false;
    }
  }
  const int slot0 = grp * PG;                        // this lane's first page within the warp's slice

  for (int t = 0; w.next(); ++t) {
    const int stage = t % NS;
    const int rows = na_s[w.s] * p.G;
    // ---- the tile's summaries have landed (this warp's copies of it are the oldest but NS - 2 groups)
    cp_async_wait_pending(NS - 2);
    __syncwarp();
    float2 kx[PG][8], kn[PG][8];                     // {run u, run u + LPP} of kmax / kmin, element jj
    {
      const uint8_t* st = gen + static_cast<size_t>(stage) * C::STAGE_BYTES + warp_off;
#pragma unroll
      for (int i = 0; i < PG; ++i) {
        float a0[8], a1[8], b0[8], b1[8];
        const T* src = reinterpret_cast<const T*>(st + static_cast<size_t>(slot0 + (i ^ xperm)) * C::PAGE_BYTES) + u * 8;
        ld8(src, a0);
        ld8(src + 8 * LPP, a1);
        ld8(src + D, b0);
        ld8(src + D + 8 * LPP, b1);
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
          kx[i][jj] = make_float2(a0[jj], a1[jj]);
          kn[i][jj] = make_float2(b0[jj], b1[jj]);
        }
      }
    }
    __syncwarp();                                    // the slice that tile t - 1 used is free: refill it
    {
      const int id = id_next;
      id_next = request_id();
      copy_tile(id, (t + NS - 1) % NS);
    }
    const bool warp_has_pages = warp * WP < w.np;
    float* tile_base = p.scores + (static_cast<size_t>(w.s) * p.B * p.Hq + w.kh * p.G) * p.score_stride + w.p0 + warp * WP + slot0;
    const int np_lane = w.np - warp * WP - slot0;    // page slot i of this lane is valid iff i < np_lane

    // the chains of one pass: rows ra and rb (of the staged tile) against the PG pages in registers
    auto fma_pass = [&](int ra, int rb, float2 (&acc)[PG][2]) {
#pragma unroll
      for (int i = 0; i < PG; ++i) acc[i][0] = acc[i][1] = make_float2(0.f, 0.f);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {               // elements jj = 4 hf .. 4 hf + 3 of both runs
        float2 qp0[4], qn0[4], qp1[4], qn1[4];
        if constexpr (sizeof(T) == 2) {
          const uint32_t* bp = reinterpret_cast<const uint32_t*>(qpos) + hf * (4 * LPP) + 4 * u;
          const uint32_t* bn = reinterpret_cast<const uint32_t*>(qneg) + hf * (4 * LPP) + 4 * u;
          const uint4 wp0 = *reinterpret_cast<const uint4*>(bp + ra * (D / 2)), wn0 = *reinterpret_cast<const uint4*>(bn + ra * (D / 2));
          const uint4 wp1 = *reinterpret_cast<const uint4*>(bp + rb * (D / 2)), wn1 = *reinterpret_cast<const uint4*>(bn + rb * (D / 2));
          const uint32_t a[4] = {wp0.x, wp0.y, wp0.z, wp0.w}, b[4] = {wn0.x, wn0.y, wn0.z, wn0.w};
          const uint32_t c[4] = {wp1.x, wp1.y, wp1.z, wp1.w}, d[4] = {wn1.x, wn1.y, wn1.z, wn1.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            qp0[e] = make_float2(__uint_as_float(a[e] << 16), __uint_as_float(a[e] & 0xffff0000u));
            qn0[e] = make_float2(__uint_as_float(b[e] << 16), __uint_as_float(b[e] & 0xffff0000u));
            qp1[e] = make_float2(__uint_as_float(c[e] << 16), __uint_as_float(c[e] & 0xffff0000u));
            qn1[e] = make_float2(__uint_as_float(d[e] << 16), __uint_as_float(d[e] & 0xffff0000u));
          }
        } else {
#pragma unroll
          for (int c2 = 0; c2 < 2; ++c2) {
            const int off = (2 * hf + c2) * (4 * LPP) + 4 * u;
            const float4 p0 = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(qpos) + ra * D + off);
            const float4 n0 = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(qneg) + ra * D + off);
            const float4 p1 = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(qpos) + rb * D + off);
            const float4 n1 = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(qneg) + rb * D + off);
            qp0[2 * c2] = make_float2(p0.x, p0.y); qp0[2 * c2 + 1] = make_float2(p0.z, p0.w);
            qn0[2 * c2] = make_float2(n0.x, n0.y); qn0[2 * c2 + 1] = make_float2(n0.z, n0.w);
            qp1[2 * c2] = make_float2(p1.x, p1.y); qp1[2 * c2 + 1] = make_float2(p1.z, p1.w);
            qn1[2 * c2] = make_float2(n1.x, n1.y); qn1[2 * c2 + 1] = make_float2(n1.z, n1.w);
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int jj = 4 * hf + e;
          // 2 PG independent chains advance by the q+ term, then all of them by the q- term:
          // dependent instructions stay 2 PG issue slots apart
#pragma unroll
          for (int i = 0; i < PG; ++i) {
            acc[i][0] = __ffma2_rn(qp0[e], kx[i][jj], acc[i][0]);
            acc[i][1] = __ffma2_rn(qp1[e], kx[i][jj], acc[i][1]);
          }
#pragma unroll
          for (int i = 0; i < PG; ++i) {
            acc[i][0] = __ffma2_rn(qn0[e], kn[i][jj], acc[i][0]);
            acc[i][1] = __ffma2_rn(qn1[e], kn[i][jj], acc[i][1]);
          }
        }
      }
    };
    // the butterfly of one pass and its stores; offa / offb: offsets of the score rows of this lane's
    // first and second row; has_b: the second row exists
    auto reduce_store = [&](const float2 (&acc)[PG][2], size_t offa, size_t offb, bool has_a, bool has_b) {
      float v[NP];
#pragma unroll
      for (int i = 0; i < PG; ++i)
#pragma unroll
        for (int rr = 0; rr < 2; ++rr) v[2 * i + rr] = __fadd_rn(acc[i][rr].x, acc[i][rr].y);      // offset d/16
      int n = NP;
#pragma unroll
      for (int l = 0; l < LV; ++l) {
        const int mask = (LPP / 2) >> l;
        if (l < LOGNP) {
          n >>= 1;
#pragma unroll
          for (int k = 0; k < NP / 2; ++k)
            if (k < n) v[k] = __fadd_rn(v[k], __shfl_xor_sync(0xffffffffu, v[k + n], mask));
        } else {
          v[0] = __fadd_rn(v[0], __shfl_xor_sync(0xffffffffu, v[0], mask));
        }
      }
#pragma unroll
      for (int k = 0; k < NF; ++k) {
        const int i = (k >> 1) ^ xperm;
        const bool second = (k & 1) != 0;              // of this lane's two rows (only when both are left: NF >= 2)
        if (stores && i < np_lane && (second ? has_b : has_a))
          tile_base[(second ? offb : offa) + i] = __fadd_rn(v[k], 0.0f);
      }
    };

    for (int r0 = 0; r0 < rows; r0 += kPsRowTile) {
      const int nr = min(kPsRowTile, rows - r0);
      ensure_rows(w.s, w.kh, r0, nr);
      if (!warp_has_pages) continue;
      int a_row = r0 / p.G, g_row = r0 % p.G;        // row r0 + r = (active slot a_row, head g_row of the KV head)
      // offsets of the score rows of rows r and r + 1 as this lane sees them (its first row is r + 1
      // when it takes the rows the other way round); then steps two rows on
      auto row_offsets = [&](size_t& offa, size_t& offb) {
        const size_t o0 = (static_cast<size_t>(a_row) * p.Hq + g_row) * p.score_stride;
        int a1 = a_row, g1 = g_row + 1;
        if (g1 >= p.G) { g1 = 0; ++a1; }
        const size_t o1 = (static_cast<size_t>(a1) * p.Hq + g1) * p.score_stride;
        offa = rowswap ? o1 : o0;
        offb = rowswap ? o0 : o1;
        g_row += 2;
        while (g_row >= p.G) { g_row -= p.G; ++a_row; }
      };
      // rows of a pass as this lane takes them; an odd tail computes its last row twice and stores it once
      auto pass_rows = [&](int r, int& ra, int& rb) {
        const int r1 = min(r + 1, nr - 1);
        ra = rowswap ? r1 : r;
        rb = rowswap ? r : r1;
      };
      auto finish_pass = [&](const float2 (&acc)[PG][2], int r) {
        size_t offa, offb;
        row_offsets(offa, offb);
        const bool two = r + 1 < nr;
        reduce_store(acc, offa, offb, rowswap ? two : true, rowswap ? true : two);
      };
      // software pipeline over the passes: the chains of pass i + 1 are issued in the same straight
      // line of code as the butterfly of pass i, whose shuffle latencies they hide (two passes per
      // trip, the two accumulator sets trading places, so that nothing is copied)
      float2 acc[PG][2], nxt[PG][2];
      int ra, rb;
      pass_rows(0, ra, rb);
      fma_pass(ra, rb, acc);
      int r = 0;
      while (r + 4 < nr) {
        pass_rows(r + 2, ra, rb);
        fma_pass(ra, rb, nxt);
        finish_pass(acc, r);
        pass_rows(r + 4, ra, rb);
        fma_pass(ra, rb, acc);
        finish_pass(nxt, r + 2);
        r += 4;
      }
      if (r + 2 < nr) {
        pass_rows(r + 2, ra, rb);
        fma_pass(ra, rb, nxt);
        finish_pass(acc, r);
        finish_pass(nxt, r + 2);
      } else {
        finish_pass(acc, r);
      }
    }
  }
  cp_async_wait_pending(0);
}


// =============================================================================================
// Tensor-core page bounds (bf16).  U(p) is the product of [q+ | q-] (rows) with [kmax | kmin]
// (pages): a GEMM whose bf16 operands are exact (q+ and q- are q or 0).  The tensor cores accumulate
// in an order and rounding of their own, so their result A(p) is not the fp32 value the interface
// fixes; but |A(p) - U(p)| <= delta(p) = kMmaErrCoef * S(p), S(p) = sum_j |q+_j kmax_j| + |q-_j kmin_j|
// (the same MMAs on the operands with their sign bits cleared): every product is exact, each of the
// <= 2 d additions of either summation errs by at most 2^-23 of a running magnitude that never
// exceeds S(p); 2 * 2 d * 2^-23 <= 2^-13 for d <= 128 once more, and kMmaErrCoef = 2^-13 leaves a
// factor of four (which also covers the rounding of S and of A -+ delta themselves).  The kernel
// writes the pair (A - delta, A + delta) per (query row, page).  The selection that follows keeps
// every page whose upper bound reaches the k-th largest lower bound - a superset of the exact
// top-k, ties included - and evaluates U in the fixed order for those few pages only.
//
// Same persistent streaming structure as the kernel above (one CTA per SM, per-warp cp.async ring),
// but its work list counts whole tiles: a (sequence, KV head) with P pages is cut into
// ceil(P / tile) tiles of equal size, tile <= 128 pages chosen per launch (see launch_page_bounds),
// because a tile costs this kernel about the same whatever it holds.
// A warp's slice of a tile is 16 pages = two 8-page MMA tiles; query rows are staged per
// (sequence, KV head) as bf16 rows [q+ | q-].  The contraction index is free to permute: lane
// (g = lane / 4, t = lane % 4) reads one 16-byte chunk (8 elements) per operand row and uses its
// halves as the lane's k-columns of two consecutive m16n8k16 steps, for A and B alike, so every
// fragment load is one 16-byte shared-memory read; chunk positions are XOR-swizzled by the row's
// parity so that the two rows a quarter-warp touches fall into different banks.
constexpr float kMmaErrCoef = 1.0f / 8192.0f;
constexpr int kMmaWP = 16;                          // pages per warp and tile
constexpr int kMmaTP = kPsWarps * kMmaWP;           // pages per tile
constexpr int kMmaStages = 2;                       // tiles in shared memory: two leave room for the CTAs of the in-block attention, which runs beside

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// positive / negative part of two packed bf16 values (sign bit set <=> negative; -0 maps to +0 / -0)
__device__ __forceinline__ uint32_t bf2_pos(uint32_t w) { return w & ~(((w >> 15) & 0x00010001u) * 0xffffu); }
__device__ __forceinline__ uint32_t bf2_neg(uint32_t w) { return w & (((w >> 15) & 0x00010001u) * 0xffffu); }

template <int D>
struct MmaCfg {
  static constexpr int ROW_BYTES = 4 * D;                 // [kmax | kmin] of a page, or [q+ | q-] of a query row
  static constexpr int CPR = ROW_BYTES / 16;              // 16-byte chunks per row
  static constexpr int CH = CPR / 2;                      // chunks of one summary
  static constexpr int RPI = 32 / CH;                     // summaries one warp-wide copy instruction covers
  static constexpr int NI = 2 * kMmaWP / RPI;             // copy instructions per warp and tile
  static constexpr int STAGE_BYTES = kMmaTP * ROW_BYTES;
  static constexpr int QBUF_BYTES = kPsRowTile * ROW_BYTES;
};
// byte offset of chunk c of row r in a tile of rows of `row_bytes`, with the parity swizzle
__device__ __forceinline__ uint32_t mma_off(int r, int c, int row_bytes) {
  return static_cast<uint32_t>(r * row_bytes + ((c ^ ((r & 1) << 2)) << 4));
}

// APPROX: write the tensor-core score A itself as an fp32 score row (no magnitudes, no radius).
template <int D, bool APPROX>
__global__ void __launch_bounds__(kPsThreads, 1) page_bounds_mma_kernel(PsParams p) {
  using C = MmaCfg<D>;
  using T = __nv_bfloat16;
  constexpr int WP = kMmaWP;                         // (a tile holds p.tile_pages <= kMmaTP pages)
  extern __shared__ uint8_t ps_smem[];
  const uint32_t raw = smem_u32(ps_smem);
  const uint32_t base = (raw + 127u) & ~127u;
  uint8_t* gen = ps_smem + (base - raw);
  const int NS = p.n_stages;
  uint8_t* qbuf = gen + static_cast<size_t>(NS) * C::STAGE_BYTES;            // [kPsRowTile][q+ | q-], swizzled chunks
  int* pre = reinterpret_cast<int*>(qbuf + C::QBUF_BYTES);
  int* na_s = pre + p.N + 1;
  int* tok_s = na_s + p.N;
  int* pages_s = tok_s + kPsSeqStage * LOSA_MAX_BLOCK;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  grid_dep_trigger();
  // When the previous kernel of the stream is known to be stage 1 of this step (whole-step path), the
  // work list, the page-table entries and the first tiles of summaries are taken while it still
  // runs: none of them is written by it, and it released this kernel only after everything before
  // it had completed.  Otherwise wait first.
  if (!p.early) grid_dep_wait();
  int lo = 0, hi = 0, s_lo = 0;
  const int tile = p.tile_pages;                     // at most TP
  const bool any = ps_list(p, pre, lo, hi, s_lo, tile, pages_s);
  auto token_of = [&](int s, int a) {
    int tok = (s >= s_lo && s < s_lo + kPsSeqStage) ? tok_s[(s - s_lo) * p.B + a] : p.active_idx[s * p.B + a];
    if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); tok = 0; }
    return tok;
  };
  const T* qg = static_cast<const T*>(p.q);
  const T* kmaxg = static_cast<const T*>(p.kmax);
  const T* kming = static_cast<const T*>(p.kmin);
  float2* bounds = reinterpret_cast<float2*>(p.scores);
  const uint32_t warp_off = static_cast<uint32_t>(warp) * WP * C::ROW_BYTES;

  TileWalkEven w_ids, w_copy, w;
  w_ids.init(pre, pages_s, p.Hkv, tile, lo, hi);
  w_copy.init(pre, pages_s, p.Hkv, tile, lo, hi);
  w.init(pre, pages_s, p.Hkv, tile, lo, hi);
  auto request_id = [&]() {
    int id = 0;
    if (w_ids.next()) {
      const int pl = warp * WP + lane;
      if (lane < WP && pl < w_ids.np) {
        id = __ldcg(p.page_table + static_cast<size_t>(w_ids.s) * p.Pmax + w_ids.p0 + pl);
        if (id < 0 || id >= p.n_phys) { set_status(p.status, LOSA_ERR_BOUNDS); id = 0; }
      }
    }
    return id;
  };
  auto copy_tile = [&](int id, int stage) {          // always one group, empty when the walk is over
    if (w_copy.next()) {
      const uint32_t dst = base + static_cast<uint32_t>(stage) * C::STAGE_BYTES + warp_off;
      const int c = lane % C::CH, sub = lane / C::CH;
#pragma unroll
      for (int i = 0; i < C::NI; ++i) {
        const int row = i * C::RPI + sub, pl = row >> 1, a = row & 1;     // page of the slice, 0 = kmax / 1 = kmin
        const int ph = __shfl_sync(0xffffffffu, id, pl);
        if (warp * WP + pl < w_copy.np) {
          const T* src = (a ? kming : kmaxg) + (static_cast<size_t>(ph) * p.Hkv + w_copy.kh) * D + c * 8;
          cp_async16(dst + mma_off(pl, a * C::CH + c, C::ROW_BYTES), src);
        } else {
          // pages past the tile's end take part in the MMAs (their columns are not stored): keep them finite
          *reinterpret_cast<uint4*>(gen + static_cast<size_t>(stage) * C::STAGE_BYTES + warp_off + mma_off(pl, a * C::CH + c, C::ROW_BYTES)) =
              make_uint4(0u, 0u, 0u, 0u);
        }
      }
    }
    cp_async_commit();
  };
  int id_next = 0;
  if (any) {
    id_next = request_id();
    for (int i = 0; i < NS - 1; ++i) {
      const int id = id_next;
      id_next = request_id();
      copy_tile(id, i);
    }
  }
  if (p.early) grid_dep_wait();                      // every CTA, also one without work: the next kernel counts on it
  if (!any) return;
  ps_active(p, na_s, tok_s, s_lo);
  __syncthreads();                                   // the cached active lists are in place

  // rows r0 .. r0 + nr - 1 of (sequence s, KV head kh) as [q+ | q-] into the staging tile; the rows
  // up to the next multiple of 16 are cleared (they take part in the last 16-row MMA tile)
  auto stage_rows = [&](int s, int kh, int r0, int nr) {
    const int nr16 = (nr + 15) & ~15;
    for (int idx = tid; idx < nr16 * C::CH; idx += kPsThreads) {
      const int r = idx / C::CH, c = idx % C::CH, row = r0 + r;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < nr) {
        const int tok = token_of(s, row / p.G);
        v = *reinterpret_cast<const uint4*>(qg + ((static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + row % p.G) * D + c * 8);
      }
      *reinterpret_cast<uint4*>(qbuf + mma_off(r, c, C::ROW_BYTES)) = make_uint4(bf2_pos(v.x), bf2_pos(v.y), bf2_pos(v.z), bf2_pos(v.w));
      *reinterpret_cast<uint4*>(qbuf + mma_off(r, c + C::CH, C::ROW_BYTES)) = make_uint4(bf2_neg(v.x), bf2_neg(v.y), bf2_neg(v.z), bf2_neg(v.w));
    }
  };
  // Staging on demand (all threads, same arguments): a new (sequence, KV head), or another row tile
  // when a pair has more rows than one staging holds (every token active).  The first tile's rows
  // are staged before the loop, while the first copies are still in flight.
  int staged_pair = -1, staged_r0 = -1;
  auto ensure_rows = [&](int s, int kh, int r0, int nr) {
    const int pair = s * p.Hkv + kh;
    if (pair == staged_pair && r0 == staged_r0) return;
    __syncthreads();
    stage_rows(s, kh, r0, nr);
    __syncthreads();
    staged_pair = pair;
    staged_r0 = r0;
  };
  {
    TileWalkEven first;
    first.init(pre, pages_s, p.Hkv, tile, lo, hi);
    if (first.next()) ensure_rows(first.s, first.kh, 0, min(kPsRowTile, na_s[first.s] * p.G));
  }

  const int g = lane >> 2, t4 = lane & 3;
  for (int t = 0; w.next(); ++t) {
    const int stage = t % NS;
    const int rows = na_s[w.s] * p.G;
    cp_async_wait_pending(NS - 2);
    __syncwarp();
    {                                                // the slice that tile t - 1 used is free: refill it
      const int id = id_next;
      id_next = request_id();
      copy_tile(id, (t + NS - 1) % NS);
    }
    const uint8_t* st = gen + static_cast<size_t>(stage) * C::STAGE_BYTES + warp_off;
    const bool warp_has_pages = warp * WP < w.np;
    for (int r0 = 0; r0 < rows; r0 += kPsRowTile) {
      const int nr = min(kPsRowTile, rows - r0);
      ensure_rows(w.s, w.kh, r0, nr);
      if (!warp_has_pages) continue;
      for (int mt = 0; mt * 16 < nr; ++mt) {
        float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};     // pages 0..7 / 8..15 of the slice
        float m0[4] = {0.f, 0.f, 0.f, 0.f}, m1[4] = {0.f, 0.f, 0.f, 0.f};     // the same on the magnitudes
        // chunk 4 sg + t4 of a row of parity b sits at position 4 (sg ^ b) + t4: with d = 64 b bytes,
        // at base + d + 64 sg for even sg and base - d + 64 sg for odd sg (all four rows this lane
        // reads have the parity of g), so every address below is a lane constant plus an immediate
        const int dsw = (g & 1) * 64;
        const uint8_t* a_lo_p = qbuf + (16 * mt + g) * C::ROW_BYTES + t4 * 16;
        const uint8_t* a_hi_p = a_lo_p + 8 * C::ROW_BYTES;
        const uint8_t* b_0_p = st + g * C::ROW_BYTES + t4 * 16;
        const uint8_t* b_1_p = b_0_p + 8 * C::ROW_BYTES;
#pragma unroll
        for (int sg = 0; sg < C::CPR / 4; ++sg) {
          const int off = 64 * sg + ((sg & 1) ? -dsw : dsw);
          uint4 a_lo = *reinterpret_cast<const uint4*>(a_lo_p + off);
          uint4 a_hi = *reinterpret_cast<const uint4*>(a_hi_p + off);
          uint4 b_0 = *reinterpret_cast<const uint4*>(b_0_p + off);
          uint4 b_1 = *reinterpret_cast<const uint4*>(b_1_p + off);
          mma_bf16_16816(c0, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b_0.x, b_0.y);
          mma_bf16_16816(c1, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b_1.x, b_1.y);
          mma_bf16_16816(c0, a_lo.z, a_hi.z, a_lo.w, a_hi.w, b_0.z, b_0.w);
          mma_bf16_16816(c1, a_lo.z, a_hi.z, a_lo.w, a_hi.w, b_1.z, b_1.w);
          if (APPROX) continue;                          // no error radius wanted
          constexpr uint32_t kAbs = 0x7fff7fffu;
          a_lo.x &= kAbs; a_lo.y &= kAbs; a_lo.z &= kAbs; a_lo.w &= kAbs;
          a_hi.x &= kAbs; a_hi.y &= kAbs; a_hi.z &= kAbs; a_hi.w &= kAbs;
          b_0.x &= kAbs; b_0.y &= kAbs; b_0.z &= kAbs; b_0.w &= kAbs;
          b_1.x &= kAbs; b_1.y &= kAbs; b_1.z &= kAbs; b_1.w &= kAbs;
          mma_bf16_16816(m0, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b_0.x, b_0.y);
          mma_bf16_16816(m1, a_lo.x, a_hi.x, a_lo.y, a_hi.y, b_1.x, b_1.y);
          mma_bf16_16816(m0, a_lo.z, a_hi.z, a_lo.w, a_hi.w, b_0.z, b_0.w);
          mma_bf16_16816(m1, a_lo.z, a_hi.z, a_lo.w, a_hi.w, b_1.z, b_1.w);
        }
        // c[0], c[1]: row g, pages 2 t4, 2 t4 + 1 of the 8-page tile; c[2], c[3]: row g + 8
#pragma unroll
        for (int hr = 0; hr < 2; ++hr) {
          const int r = 16 * mt + g + 8 * hr;
          if (r < nr) {
            const int row = r0 + r, a = row / p.G, gi = row % p.G;
            const size_t at = ((static_cast<size_t>(w.s) * p.B + a) * p.Hq + w.kh * p.G + gi) * p.score_stride + w.p0 + warp * WP + 2 * t4;
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int col = warp * WP + 2 * t4 + e;
              if (APPROX) {
                if (col < w.np) p.scores[at + e] = c0[2 * hr + e];
                if (col + 8 < w.np) p.scores[at + e + 8] = c1[2 * hr + e];
              } else {
                const float d0 = kMmaErrCoef * m0[2 * hr + e], d1 = kMmaErrCoef * m1[2 * hr + e];
                if (col < w.np) bounds[at + e] = make_float2(c0[2 * hr + e] - d0, c0[2 * hr + e] + d0);
                if (col + 8 < w.np) bounds[at + e + 8] = make_float2(c1[2 * hr + e] - d1, c1[2 * hr + e] + d1);
              }
            }
          }
        }
      }
    }
  }
  cp_async_wait_pending(0);
}

template <typename T, int D, int PG>
int32_t launch_stream(losa_ctx* c, const PsParams& pp, cudaStream_t st) {
  using C = PsCfg<T, D, PG>;
  PsParams p = pp;
  const int tail = ps_tail_bytes(p.N);
  int ns = (kPsSmemBudget - C::QBUF_BYTES - tail - 128) / C::STAGE_BYTES;
  ns = ns > kPsMaxStages ? kPsMaxStages : ns;
  if (ns < 2) return LOSA_ERR_UNSUPPORTED;
  p.n_stages = ns;
  const int smem = 128 + ns * C::STAGE_BYTES + C::QBUF_BYTES + tail;
  if (!c->scores_attr_set) {
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(page_scores_stream_kernel<T, D, PG>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    c->scores_attr_set = 1;
  }
  launch_k(page_scores_stream_kernel<T, D, PG>, p.n_ctas, kPsThreads, smem, st, p);
  return after_launch(c);
}

template <int D, bool APPROX>
int32_t launch_bounds_t(losa_ctx* c, const PsParams& pp, cudaStream_t st) {
  using C = MmaCfg<D>;
  PsParams p = pp;
  const int tail = ps_tail_bytes(p.N);
  int ns = (kPsSmemBudget - C::QBUF_BYTES - tail - 128) / C::STAGE_BYTES;
  ns = ns > kMmaStages ? kMmaStages : ns;
  if (ns < 2) return LOSA_ERR_UNSUPPORTED;
  p.n_stages = ns;
  const int smem = 128 + ns * C::STAGE_BYTES + C::QBUF_BYTES + tail;
  int32_t& attr_set = APPROX ? c->approx_attr_set : c->bounds_attr_set;
  if (!attr_set) {
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(page_bounds_mma_kernel<D, APPROX>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_set = 1;
  }
  launch_k(page_bounds_mma_kernel<D, APPROX>, p.n_ctas, kPsThreads, smem, st, p);
  return after_launch(c);
}

PsParams make_params(losa_ctx* c, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                     const int32_t* n_active, const int32_t* step) {
  const losa_shape_t& sh = c->shape;
  PsParams p;
  p.q = q;
  p.kmin = kv->kmin;
  p.kmax = kv->kmax;
  p.page_table = kv->page_table;
  p.kv_len = kv->kv_len;
  p.active_idx = active_idx;
  p.n_active = n_active;
  p.step = step;
  p.scores = reinterpret_cast<float*>(c->ws + c->lay.scores);
  p.status = status_ptr(c);
  p.N = sh.batch;
  p.B = sh.block_size;
  p.Hq = sh.n_q_heads;
  p.Hkv = sh.n_kv_heads;
  p.G = sh.n_q_heads / sh.n_kv_heads;
  p.g = sh.page_size;
  p.Pmax = sh.max_pages_per_seq;
  p.n_phys = kv->n_phys_pages;
  p.score_stride = c->lay.score_stride;
  p.n_ctas = c->n_sms;
  p.n_stages = 0;
  p.early = 0;
  p.tile_pages = 0;
  return p;
}

}  // namespace

// bf16 only: (lower, upper) bound pairs of the page scores into the workspace's score rows (as float2)
int32_t launch_page_bounds(losa_ctx* c, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                           const int32_t* n_active, const int32_t* step, cudaStream_t st, bool approx_only, bool after_stage1) {
  PsParams p = make_params(c, q, kv, active_idx, n_active, step);
  p.early = after_stage1 ? 1 : 0;
  // Pages per tile: a tile costs a fixed part plus a part per page (about 0.8 us + 2 us per 128 pages),
  // and the kernel lasts as many tiles as its busiest CTA gets; of the sizes 16, 32 .. 128 the one that
  // makes (rounds) x (cost of a tile) least, on the assumption that every prefix has its longest
  // length (the real lengths live on the device): short prefixes get small tiles so that every CTA has one.
  {
    const losa_shape_t& sh = c->shape;
    float best = 3.0e38f;
    for (int tp = kMmaTP; tp >= 16; tp -= 16) {
      const long long tiles = static_cast<long long>(sh.batch) * sh.n_kv_heads * ((sh.max_pages_per_seq + tp - 1) / tp);
      const long long rounds = (tiles + p.n_ctas - 1) / p.n_ctas;
      const float cost = static_cast<float>(rounds) * (0.8f + 2.0f * static_cast<float>(tp) / 128.f);
      if (cost < best) { best = cost; p.tile_pages = tp; }
    }
  }
  if (approx_only) return c->shape.head_dim == 128 ? launch_bounds_t<128, true>(c, p, st) : launch_bounds_t<64, true>(c, p, st);
  return c->shape.head_dim == 128 ? launch_bounds_t<128, false>(c, p, st) : launch_bounds_t<64, false>(c, p, st);
}

int32_t launch_page_scores(losa_ctx* c, const void* q, const losa_kv_t* kv, const int32_t* active_idx,
                           const int32_t* n_active, const int32_t* step, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  const PsParams p = make_params(c, q, kv, active_idx, n_active, step);
  const bool bf = sh.dtype == LOSA_BF16;
  if (bf && sh.head_dim == 128) return launch_stream<__nv_bfloat16, 128, 4>(c, p, st);
  if (bf) return launch_stream<__nv_bfloat16, 64, 4>(c, p, st);
  if (sh.head_dim == 128) return launch_stream<float, 128, 2>(c, p, st);
  return launch_stream<float, 64, 2>(c, p, st);
}

}  // namespace losa
