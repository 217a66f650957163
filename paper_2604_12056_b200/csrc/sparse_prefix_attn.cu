// Stage 4 — paged sparse prefix attention for the active tokens (Section 2.2, Section 4.2).
//
// Work decomposition (both element types).  The pages to read form a flat list of items
// (segment = (sequence, KV head, row group), position in that segment's union list).  The list is
// cut into one contiguous, equally long range per CTA (one CTA per SM), so ragged unions never
// leave an SM idle.  A CTA produces, for every segment its range touches, an un-normalised partial
// (row max, row sum, sum p*v) in the workspace; a small combine kernel merges the partials of a
// segment by log-sum-exp — the same merge Section 2.2 uses between prefix and block — and writes
// (o_p, L_p) of the ACTIVE tokens only, which is what keeps the reuse rule exact for the others.
//
// bf16 kernel (sparse_prefix_attn_tc5.cuh): TMA streams the pages of K and V into rings of shared
//   memory; Q K^T and P V run on the tcgen05 tensor cores with Q, S, P and O in tensor memory; the
//   softmax warps own one query row per thread.  Query rows are the GQA-grouped (active token,
//   head) pairs of the KV head, up to 128 per row group.
// fp32 kernel: CUDA cores, fp32 FMA (bf16 tensor cores cannot meet the 1e-5 fp32 tolerance).
//
// Every wait on an mbarrier is bounded; when a bound runs out the CTA records LOSA_ERR_TIMEOUT,
// raises its abort flag (which ends every other wait of the CTA) and leaves through the common exit.
#include <cuda.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <algorithm>

#include "kernels.h"

namespace losa {
namespace {

struct AttnParams {
  const void* q;
  const void* k_pages;
  const void* v_pages;
  int64_t stride_page, stride_head, stride_tok;
  const int32_t* page_table;
  const int32_t* kv_len;
  const int32_t* active_idx;
  const int32_t* n_active;
  const int32_t* union_pages;
  const int32_t* union_count;
  float* partials;
  int32_t* seg_prefix;  // workspace copy of the segment prefix (written by the bf16 main kernel, read by its combine kernel)
  void* o_p;                // cached prefix output, fp32 or bf16 (o_p_bf16)
  int o_p_bf16;
  float* lse_p;
  int32_t* status;
  const float* k_scale;   // FP8 pages: [n_phys, H_kv] power-of-two scales (else null)
  const float* v_scale;
  int N, B, Hq, Hkv, G, Pmax, n_phys, n_rg, n_seg, n_ctas;
  float sm_scale;
  long long wait_cycles;  // bound of every mbarrier wait of the bf16 main kernel, in SM clock cycles
};


// Partial results.  A slot (CTA b, segment seg -> b + seg) holds eight records, record t for the
// rows 16t .. 16t+15 of the row group: m[16], l[16], o[16][D] (un-normalised, relative to m).
constexpr int kTileRows = 16;
__device__ __forceinline__ float* record_base(float* partials, int slot, int w, int D) {
  return partials + (static_cast<size_t>(slot) * 8 + w) * kTileRows * (D + 2);
}

__device__ __forceinline__ int clamp_active(int na, int B) { return na < 0 ? 0 : (na > B ? B : na); }

// C (2 or 4) consecutive elements as one vector access; a lane of the row-wise kernels below owns
// columns lane * C .. lane * C + C - 1 of a row of D = 32 C elements.
template <int C> __device__ __forceinline__ void ldv(const float* p, float (&v)[C]) {
  if constexpr (C == 4) { const float4 t = *reinterpret_cast<const float4*>(p); v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w; }
  else { const float2 t = *reinterpret_cast<const float2*>(p); v[0] = t.x; v[1] = t.y; }
}
template <int C> __device__ __forceinline__ void stv(float* p, const float (&v)[C]) {
  if constexpr (C == 4) *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  else *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]);
}
template <int C> struct RawRow;                      // C elements of the I/O type, moved as they are
template <> struct RawRow<4> { uint2 bits; };
template <> struct RawRow<2> { uint32_t bits; };
template <int C> __device__ __forceinline__ RawRow<C> ld_raw(const __nv_bfloat16* p) { return *reinterpret_cast<const RawRow<C>*>(p); }
template <int C> __device__ __forceinline__ void st_raw(__nv_bfloat16* p, const RawRow<C>& r) { *reinterpret_cast<RawRow<C>*>(p) = r; }
template <int C> __device__ __forceinline__ void st_bf16(__nv_bfloat16* p, const float (&v)[C]) {
  RawRow<C> r;
  if constexpr (C == 4) {
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]), b = __floats2bfloat162_rn(v[2], v[3]);
    r.bits = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
  } else {
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
    r.bits = *reinterpret_cast<uint32_t*>(&a);
  }
  st_raw<C>(p, r);
}

// C elements of the cached prefix output (fp32 or bf16 storage) at element offset i
template <int C> __device__ __forceinline__ void ld_state(const void* base, int bf16, size_t i, float (&v)[C]) {
  if (bf16) {
    const RawRow<C> r = ld_raw<C>(static_cast<const __nv_bfloat16*>(base) + i);
    if constexpr (C == 4) {
      v[0] = __uint_as_float(r.bits.x << 16); v[1] = __uint_as_float(r.bits.x & 0xffff0000u);
      v[2] = __uint_as_float(r.bits.y << 16); v[3] = __uint_as_float(r.bits.y & 0xffff0000u);
    } else {
      v[0] = __uint_as_float(r.bits << 16); v[1] = __uint_as_float(r.bits & 0xffff0000u);
    }
  } else {
    ldv<C>(static_cast<const float*>(base) + i, v);
  }
}
// ... stored; with bf16 storage v comes back holding the stored (rounded) values, which is what every
// later use must see
template <int C> __device__ __forceinline__ void st_state(void* base, int bf16, size_t i, float (&v)[C]) {
  if (bf16) {
#pragma unroll
    for (int c = 0; c < C; ++c) v[c] = __bfloat162float(__float2bfloat16_rn(v[c]));
    st_bf16<C>(static_cast<__nv_bfloat16*>(base) + i, v);
  } else {
    stv<C>(static_cast<float*>(base) + i, v);
  }
}

// ===================================================================== fp32 / CUDA-core kernel
template <typename T, int D, int GP>
__global__ void __launch_bounds__(256, 1) attn_simt_kernel(AttnParams p) {
  grid_dep_wait();
  extern __shared__ __align__(16) float sm[];
  float* Ks = sm;                         // [GP][D]
  float* Vs = Ks + GP * D;                // [GP][D]
  float* Qs = Vs + GP * D;                // [128][D]
  float* Os = Qs + kRowsPerGroup * D;     // [128][D]
  float* Ms = Os + kRowsPerGroup * D;     // [128]
  float* Ls = Ms + kRowsPerGroup;         // [128]
  int* pre = reinterpret_cast<int*>(Ls + kRowsPerGroup);   // [n_seg + 1]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (warp == 0) segment_prefix(pre, p.n_seg, p.n_rg, p.Hkv, p.G, p.n_active, p.union_count, p.B, lane);
  __syncthreads();
  const long long T_all = pre[p.n_seg];
  const int lo = static_cast<int>(cta_lo(T_all, blockIdx.x, p.n_ctas));
  const int hi = static_cast<int>(cta_lo(T_all, blockIdx.x + 1, p.n_ctas));
  if (lo >= hi) return;
  int sg = 0;
  while (pre[sg + 1] <= lo) ++sg;
  const T* q = static_cast<const T*>(p.q);
  const T* kp = static_cast<const T*>(p.k_pages);
  const T* vp = static_cast<const T*>(p.v_pages);
  int item = lo;
  while (item < hi) {
    const int seg_end = min(hi, pre[sg + 1]);
    const int n_sk = p.n_seg / p.n_rg, rg = sg / n_sk, sk = sg % n_sk, s = sk / p.Hkv, kh = sk % p.Hkv;
    const int rows = rows_in_group(clamp_active(p.n_active[s], p.B), p.G, rg);
    const int len = p.kv_len[s];
    __syncthreads();
    for (int idx = tid * 8; idx < rows * D; idx += 256 * 8) {
      const int r = idx / D, j = idx % D;
      const int row = rg * kRowsPerGroup + r, a = row / p.G, gi = row % p.G;
      int tok = p.active_idx[s * p.B + a];
      if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); tok = 0; }
      float v[8];
      load8(q + ((static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + gi) * D + j, v);
#pragma unroll
      for (int e = 0; e < 8; ++e) { Qs[idx + e] = v[e]; Os[idx + e] = 0.f; }
    }
    for (int r = tid; r < rows; r += 256) { Ms[r] = -INFINITY; Ls[r] = 0.f; }
    for (int u = item - pre[sg]; u < seg_end - pre[sg]; ++u) {
      int page = p.union_pages[static_cast<size_t>(sk) * p.Pmax + u];
      bool ok = page >= 0 && page < p.Pmax;
      int phys = ok ? p.page_table[static_cast<size_t>(s) * p.Pmax + page] : 0;
      ok = ok && phys >= 0 && phys < p.n_phys;
      const int valid = ok ? min(GP, len - page * GP) : 0;
      if (!ok || valid <= 0) { set_status(p.status, LOSA_ERR_BOUNDS); continue; }
      __syncthreads();
      const size_t off = static_cast<size_t>(phys) * p.stride_page + static_cast<size_t>(kh) * p.stride_head;
      for (int idx = tid * 8; idx < GP * D; idx += 256 * 8) {
        const int t = idx / D, j = idx % D;
        float a[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, b[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        if (t < valid) {
          load8(kp + off + static_cast<size_t>(t) * p.stride_tok + j, a);
          load8(vp + off + static_cast<size_t>(t) * p.stride_tok + j, b);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) { Ks[idx + e] = a[e]; Vs[idx + e] = b[e]; }
      }
      __syncthreads();
      for (int r = warp; r < rows; r += 8) {
        constexpr int TPL = (GP + 31) / 32;
        float sc[TPL];
#pragma unroll
        for (int w = 0; w < TPL; ++w) {
          const int t = lane + 32 * w;
          float dot = 0.f;
          if (t < valid) {
            const float* kr = Ks + t * D;
            const float* qr = Qs + r * D;
#pragma unroll 8
            for (int j = 0; j < D; ++j) {
              const int jj = (j + lane) & (D - 1);
              dot = fmaf(qr[jj], kr[jj], dot);
            }
          }
          sc[w] = (t < valid) ? dot * p.sm_scale : -INFINITY;
        }
        float mx = sc[0];
#pragma unroll
        for (int w = 1; w < TPL; ++w) mx = fmaxf(mx, sc[w]);
        mx = warp_max(mx);
        const float m_old = Ms[r], m_new = fmaxf(m_old, mx);
        const float corr = expf(m_old - m_new);
        float pw[TPL], ps = 0.f;
#pragma unroll
        for (int w = 0; w < TPL; ++w) { pw[w] = expf(sc[w] - m_new); ps += pw[w]; }
        ps = warp_sum(ps);
        float acc[D / 32];
#pragma unroll
        for (int c = 0; c < D / 32; ++c) acc[c] = Os[r * D + lane + 32 * c] * corr;
        for (int t = 0; t < valid; ++t) {
          float pt = pw[0];
#pragma unroll
          for (int w = 1; w < TPL; ++w) pt = (t >= 32 * w) ? pw[w] : pt;
          pt = __shfl_sync(0xffffffffu, pt, t & 31);
#pragma unroll
          for (int c = 0; c < D / 32; ++c) acc[c] = fmaf(pt, Vs[t * D + lane + 32 * c], acc[c]);
        }
#pragma unroll
        for (int c = 0; c < D / 32; ++c) Os[r * D + lane + 32 * c] = acc[c];
        __syncwarp();
        if (lane == 0) { Ms[r] = m_new; Ls[r] = Ls[r] * corr + ps; }
        __syncwarp();
      }
    }
    __syncthreads();
    for (int r = tid; r < rows; r += 256) {
      float* rec = record_base(p.partials, blockIdx.x + sg, r / kTileRows, D);
      rec[r % kTileRows] = Ms[r];
      rec[kTileRows + r % kTileRows] = Ls[r];
    }
    for (int idx = tid; idx < rows * D; idx += 256) {
      const int r = idx / D;
      record_base(p.partials, blockIdx.x + sg, r / kTileRows, D)[2 * kTileRows + (r % kTileRows) * D + idx % D] = Os[idx];
    }
    item = seg_end;
    ++sg;
    while (item < hi && pre[sg + 1] <= item) ++sg;
  }
}

// ===================================================================== combine kernel
// grid (n_seg, 8): warp = one query row of the segment's row group at a time.  The CTAs whose item range
// meets the segment are consecutive; each of them left one record for the row's 16-row tile.  Lanes
// take one piece each for the row maxima and sums, then the warp walks the pieces with the loads of
// eight records issued together.  LOG2: partial maxima in base-2 units (tensor-core kernel) or
// natural units (fp32 kernel).
// Merge of the partial records of row r of segment sg by one warp: returns the un-normalised
// output columns lane * C + c in acc, the reference maximum M and the sum of weights Lsum.
template <int D, bool LOG2>
__device__ __forceinline__ void merge_records(const AttnParams& p, int sg, int r, int start, int end, long long T_all,
                                              int lane, float (&acc)[D / 32], float& M, float& Lsum) {
  constexpr int C = D / 32;
  const int tile = r / kTileRows, rr = r % kTileRows;
#pragma unroll
  for (int c = 0; c < C; ++c) acc[c] = 0.f;
  M = -INFINITY;
  Lsum = 0.f;
  if (end <= start) return;
  int b0 = static_cast<int>((static_cast<long long>(start) * p.n_ctas) / T_all);
  while (b0 + 1 < p.n_ctas && cta_lo(T_all, b0 + 1, p.n_ctas) <= start) ++b0;
  int b1 = static_cast<int>((static_cast<long long>(end - 1) * p.n_ctas) / T_all);   // last CTA that can meet it
  while (b1 + 1 < p.n_ctas && cta_lo(T_all, b1 + 1, p.n_ctas) < end) ++b1;
  const int n_pairs = b1 - b0 + 1;
  // record of piece x, or null when CTA b0 + x has no page of this segment
  auto record_of = [&](int x) -> const float* {
    if (x >= n_pairs) return nullptr;
    const int b = b0 + x;
    const long long lo = max(cta_lo(T_all, b, p.n_ctas), static_cast<long long>(start));
    const long long hi = min(cta_lo(T_all, b + 1, p.n_ctas), static_cast<long long>(end));
    if (hi <= lo) return nullptr;
    return record_base(p.partials, b + sg, tile, D);
  };
  for (int base = 0; base < n_pairs; base += 32) {
    const float* rec = record_of(base + lane);
    M = fmaxf(M, warp_max(rec ? rec[rr] : -INFINITY));
  }
  for (int base = 0; base < n_pairs; base += 32) {
    const float* rec = record_of(base + lane);
    float wj = 0.f, lj = 0.f;
    if (rec) {
      const float mj = rec[rr];
      wj = (mj == -INFINITY) ? 0.f : (LOG2 ? exp2f(mj - M) : expf(mj - M));
      lj = rec[kTileRows + rr];
    }
    Lsum += warp_sum(lj * wj);
    const int n = min(32, n_pairs - base);
    constexpr int U = 4;                            // records whose loads are in flight together
    for (int i0 = 0; i0 < n; i0 += U) {
      float w[U], v[U][C];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int i = i0 + u;
        w[u] = (i < n) ? __shfl_sync(0xffffffffu, wj, i & 31) : 0.f;
        const unsigned long long addr = __shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(rec), i & 31);
        const float* src = reinterpret_cast<const float*>(addr) + 2 * kTileRows + rr * D + lane * C;
#pragma unroll
        for (int c = 0; c < C; ++c) v[u][c] = 0.f;
        if (w[u] != 0.f) ldv<C>(src, v[u]);
      }
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int c = 0; c < C; ++c) acc[c] = fmaf(v[u][c], w[u], acc[c]);
    }
  }
}

template <int D, bool LOG2, bool PRE>
__global__ void __launch_bounds__(256) attn_combine_kernel(AttnParams p) {
  grid_dep_wait();
  __shared__ int pre[kMaxSegments + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sg = blockIdx.x;
  const int n_sk = p.n_seg / p.n_rg, rg = sg / n_sk, sk = sg % n_sk, s = sk / p.Hkv, kh = sk % p.Hkv;
  const int rows = rows_in_group(clamp_active(p.n_active[s], p.B), p.G, rg);
  if (blockIdx.y * 8 >= rows) return;                 // whole CTA idle: skip the prefix as well
  if (PRE) {                                          // the main kernel left the prefix in the workspace
    if (tid == 0) { pre[sg] = p.seg_prefix[sg]; pre[sg + 1] = p.seg_prefix[sg + 1]; pre[p.n_seg] = p.seg_prefix[p.n_seg]; }
  } else if (warp == 0) {
    segment_prefix(pre, p.n_seg, p.n_rg, p.Hkv, p.G, p.n_active, p.union_count, p.B, lane);
  }
  __syncthreads();
  constexpr int C = D / 32;
  for (int r = blockIdx.y * 8 + warp; r < rows; r += gridDim.y * 8) {   // few CTAs per segment: most row blocks are empty on most steps
    const int row = rg * kRowsPerGroup + r, a = row / p.G, gi = row % p.G;
    const int tok = p.active_idx[s * p.B + a];
    if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); continue; }
    const size_t orow = (static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + gi;
    float acc[C], M, Lsum;
    // (PRE: the prefix left by the tensor-core kernel is that of the charged list; a segment's pages follow its pad)
    const int pad = (PRE && pre[sg + 1] > pre[sg]) ? segment_pad(rows) : 0;
    merge_records<D, LOG2>(p, sg, r, pre[sg] + pad, pre[sg + 1], pre[p.n_seg], lane, acc, M, Lsum);
    const bool empty = !(Lsum > 0.f);
    const float inv = empty ? 0.f : 1.f / Lsum;
#pragma unroll
    for (int c = 0; c < C; ++c) acc[c] *= inv;
    st_state<C>(p.o_p, p.o_p_bf16, orow * D + lane * C, acc);
    if (lane == 0) p.lse_p[orow] = empty ? -INFINITY : (LOG2 ? (M + log2f(Lsum)) * kLn2 : M + logf(Lsum));
  }
}

// Whole-step path, last kernel (bf16 main kernel): one warp per (sequence, block token, head) row.
// An active row merges its partial records (as the combine kernel does) and stores the new prefix
// statistics; a stable row reads its cached ones (reuse rule, Section 4.2).  Either way the row is
// then merged with the in-block part by log-sum-exp (Section 2.2 / 4.3), the output is written and
// the row's query kept for the next step's Eq. 1; block 0 also bumps the step counters.
struct FinishParams {
  const void* q;
  void* q_prev;
  const float* o_b;
  const float* lse_b;
  void* out;
  float* lse_out;
  int32_t* step;
  const int32_t* slot_map;   // [N*B] slot of a block token in the active list, -1 = stable (null: look it up)
  size_t n_rows;
};

constexpr int kFinishThreads = 128;

template <typename T, int D>
__global__ void __launch_bounds__(kFinishThreads) attn_finish_kernel(AttnParams p, FinishParams f) {
  grid_dep_trigger();
  grid_dep_wait();
  constexpr int C = D / 32;
  const int lane = threadIdx.x & 31;
  const size_t row = static_cast<size_t>(blockIdx.x) * (kFinishThreads / 32) + (threadIdx.x >> 5);
  if (blockIdx.x == 0)
    for (int s = threadIdx.x; s < p.N; s += kFinishThreads) f.step[s] += 1;
  if (row >= f.n_rows) return;
  const int hq = static_cast<int>(row % p.Hq), tok = static_cast<int>((row / p.Hq) % p.B);
  const int s = static_cast<int>(row / (static_cast<size_t>(p.Hq) * p.B));
  const int kh = hq / p.G, gi = hq % p.G;
  // operands that do not depend on the row being active: requested first (one vector access each)
  const T* q = static_cast<const T*>(f.q);
  float b[C];
  ldv<C>(f.o_b + row * D + lane * C, b);
  const RawRow<C> qv = ld_raw<C>(q + row * D + lane * C);
  const float Lb = f.lse_b[row];
  // the cached prefix statistics as well: nine rows in ten are stable, and asking now saves them
  // a second round trip (an active row overwrites these below)
  float a[C], Lp;
  ld_state<C>(p.o_p, p.o_p_bf16, row * D + lane * C, a);
  Lp = p.lse_p[row];
  // the row's slot in the active list, if any (the list has at most B <= 64 entries)
  int slot = -1;
  if (f.slot_map) {
    slot = f.slot_map[s * p.B + tok];
    if (slot >= p.B) slot = -1;
  } else {
    const int na = clamp_active(p.n_active[s], p.B);
    for (int base = 0; base < na && slot < 0; base += 32) {
      const int i = base + lane;
      const unsigned hit = __ballot_sync(0xffffffffu, i < na && p.active_idx[s * p.B + i] == tok);
      if (hit) slot = base + __ffs(hit) - 1;
    }
  }
  if (slot >= 0) {
    const int rowk = slot * p.G + gi, rg = rowk / kRowsPerGroup, r = rowk % kRowsPerGroup;
    const int sg = rg * (p.n_seg / p.n_rg) + s * p.Hkv + kh;
    float acc[C], M, Lsum;
    const int v0 = p.seg_prefix[sg], v1 = p.seg_prefix[sg + 1];      // of the charged list: the segment's pages follow its pad
    const int pad = v1 > v0 ? segment_pad(rows_in_group(clamp_active(p.n_active[s], p.B), p.G, rg)) : 0;
    merge_records<D, true>(p, sg, r, v0 + pad, v1, p.seg_prefix[p.n_seg], lane, acc, M, Lsum);
    const bool empty = !(Lsum > 0.f);
    const float inv = empty ? 0.f : 1.f / Lsum;
    Lp = empty ? -INFINITY : (M + log2f(Lsum)) * kLn2;
#pragma unroll
    for (int c = 0; c < C; ++c) a[c] = acc[c] * inv;
    st_state<C>(p.o_p, p.o_p_bf16, row * D + lane * C, a);
    if (lane == 0) p.lse_p[row] = Lp;
  }
  const float Mx = fmaxf(Lp, Lb);
  const float L = Mx + logf(expf(Lp - Mx) + expf(Lb - Mx));
  const float wp = expf(Lp - L), wb = expf(Lb - L);
  T* out = static_cast<T*>(f.out);
  T* q_prev = static_cast<T*>(f.q_prev);
  float o[C];
#pragma unroll
  for (int c = 0; c < C; ++c) o[c] = (wp > 0.f ? wp * a[c] : 0.f) + wb * b[c];
  st_bf16<C>(out + row * D + lane * C, o);
  st_raw<C>(q_prev + row * D + lane * C, qv);
  if (f.lse_out && lane == 0) f.lse_out[row] = L;
}

// ===================================================================== bf16 TMA + tensor-core kernel: shared pieces
constexpr int kSmemBudget = 232448;                // 227 KB opt-in limit per CTA

constexpr int kStageIdx = 1024;     // active_idx entries (N * B) cached in shared memory when they fit
constexpr int kStageSeq = 64;       // ... together with n_active and kv_len of up to this many sequences
constexpr int kTailBytes = 512 + (kMaxSegments + 1) * 4 + 4 + kStageIdx * 4 + 2 * kStageSeq * 4;   // barriers, meta, prefix, index cache
// The K / V pages are read once per launch: they are marked evict-first in L2, so that the stream
// does not push out the small arrays the following kernels read (partial records, in-block output).
__device__ __forceinline__ unsigned long long l2_evict_first_policy() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3, unsigned long long policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "l"(policy) : "memory");
}
// Loads whose issue point must stay where it is written (they are prefetches): volatile asm.
__device__ __forceinline__ int ld_nc_s32(const int32_t* ptr) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(ptr));
  return v;
}
// 2^x, one MUFU instruction (ex2.approx: 2 ulp; -inf -> 0); the bf16 rounding of P dwarfs its error
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  const __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}


#include "sparse_prefix_attn_tc5.cuh"

// ===================================================================== host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

int32_t encode_pool_map(losa_ctx* c, unsigned char* blob, const void* pool, const losa_kv_t* kv) {
  const losa_shape_t& sh = c->shape;
  if (!c->encode_fn) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    LOSA_CUDA_TRY(c, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess) return cuda_fail(c, cudaErrorSymbolNotFound);
    c->encode_fn = fn;
  }
  const cuuint64_t dims[4] = {static_cast<cuuint64_t>(sh.head_dim), static_cast<cuuint64_t>(sh.page_size),
                              static_cast<cuuint64_t>(sh.n_kv_heads), static_cast<cuuint64_t>(kv->n_phys_pages)};
  // bf16 pages: 64-element (128-byte) boxes with the 128-byte swizzle, as the MMA descriptors expect them;
  // FP8 pages: whole rows of d bytes, unswizzled, into the staging slots (the kernel converts them)
  const bool fp8 = kv->kv_format == LOSA_KV_FP8_E4M3;
  const cuuint64_t es = fp8 ? 1 : 2;
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(kv->stride_tok) * es, static_cast<cuuint64_t>(kv->stride_head) * es,
                                 static_cast<cuuint64_t>(kv->stride_page) * es};
  const cuuint32_t box[4] = {fp8 ? static_cast<cuuint32_t>(sh.head_dim) : 64u, static_cast<cuuint32_t>(sh.page_size), 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_fn)(
      reinterpret_cast<CUtensorMap*>(blob), fp8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
      const_cast<void*>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      fp8 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    c->last_cuda_error = static_cast<int32_t>(r);
    return LOSA_ERR_CUDA;
  }
  return LOSA_OK;
}

int32_t ensure_tensor_maps(losa_ctx* c, const losa_kv_t* kv) {
  const bool same = c->tmap_key_k == kv->k_pages && c->tmap_key_v == kv->v_pages &&
                    c->tmap_strides[0] == kv->stride_page && c->tmap_strides[1] == kv->stride_head &&
                    c->tmap_strides[2] == kv->stride_tok && c->tmap_n_phys == kv->n_phys_pages &&
                    c->tmap_format == kv->kv_format;
  if (same) return LOSA_OK;
  int32_t rc = encode_pool_map(c, c->tmap_k, kv->k_pages, kv);
  if (rc != LOSA_OK) return rc;
  rc = encode_pool_map(c, c->tmap_v, kv->v_pages, kv);
  if (rc != LOSA_OK) return rc;
  c->tmap_key_k = kv->k_pages;
  c->tmap_key_v = kv->v_pages;
  c->tmap_strides[0] = kv->stride_page;
  c->tmap_strides[1] = kv->stride_head;
  c->tmap_strides[2] = kv->stride_tok;
  c->tmap_n_phys = kv->n_phys_pages;
  c->tmap_format = kv->kv_format;
  return LOSA_OK;
}

template <int D, int GP, bool FP8>
int32_t launch_tc5(losa_ctx* c, const AttnParams& ap, cudaStream_t st, bool with_combine) {
  constexpr int smem = tc5_smem_bytes<D, FP8>();
  static_assert(smem <= kSmemBudget, "shared memory of the stage-4 kernel");
  constexpr int bit = FP8 ? 2 : 1;  // a context has one shape on one device: one instantiation per cache format
  if (!(c->attn_attr_set & bit)) {
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(attn_tc5_kernel<D, GP, FP8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    c->attn_attr_set |= bit;
  }
  CUtensorMap mk, mv;
  memcpy(&mk, c->tmap_k, sizeof(mk));
  memcpy(&mv, c->tmap_v, sizeof(mv));
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_begin, st));
  launch_k(attn_tc5_kernel<D, GP, FP8>, ap.n_ctas, kTc5Threads, smem, st, mk, mv, ap);
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_end, st));
  int32_t rc = after_launch(c);
  if (rc != LOSA_OK || !with_combine) return rc;
  launch_k(attn_combine_kernel<D, true, true>, dim3(ap.n_seg, 8), 256, 0, st, ap);
  return after_launch(c);
}

template <typename T, int D, int GP>
int32_t launch_simt(losa_ctx* c, const AttnParams& ap, cudaStream_t st) {
  const size_t smem = (static_cast<size_t>(2) * GP * D + 2 * kRowsPerGroup * D + 2 * kRowsPerGroup) * sizeof(float) +
                      (ap.n_seg + 1) * sizeof(int);
  if (!(c->attn_attr_set & 1)) {
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(attn_simt_kernel<T, D, GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    c->attn_attr_set |= 1;
  }
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_begin, st));
  launch_k(attn_simt_kernel<T, D, GP>, ap.n_ctas, 256, smem, st, ap);
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_end, st));
  int32_t rc = after_launch(c);
  if (rc != LOSA_OK) return rc;
  launch_k(attn_combine_kernel<D, false, false>, dim3(ap.n_seg, 8), 256, 0, st, ap);
  return after_launch(c);
}

template <int D>
int32_t dispatch_page(losa_ctx* c, const AttnParams& ap, cudaStream_t st, bool with_combine) {
  const bool bf = c->shape.dtype == LOSA_BF16;
  if (ap.k_scale) {                 // FP8 pages (bf16 contexts only, checked by the C-ABI layer)
    switch (c->shape.page_size) {
      case 16: return launch_tc5<D, 16, true>(c, ap, st, with_combine);
      case 32: return launch_tc5<D, 32, true>(c, ap, st, with_combine);
      default: return launch_tc5<D, 64, true>(c, ap, st, with_combine);
    }
  }
  switch (c->shape.page_size) {
    case 16: return bf ? launch_tc5<D, 16, false>(c, ap, st, with_combine) : launch_simt<float, D, 16>(c, ap, st);
    case 32: return bf ? launch_tc5<D, 32, false>(c, ap, st, with_combine) : launch_simt<float, D, 32>(c, ap, st);
    default: return bf ? launch_tc5<D, 64, false>(c, ap, st, with_combine) : launch_simt<float, D, 64>(c, ap, st);
  }
}

}  // namespace


int32_t launch_sparse_prefix_attn(losa_ctx* c, const void* q, const losa_kv_t* kv,
                                  const int32_t* active_idx, const int32_t* n_active,
                                  const int32_t* union_pages, const int32_t* union_count,
                                  losa_state_t* state, cudaStream_t st, bool defer_combine) {
  const losa_shape_t& sh = c->shape;
  if (sh.dtype == LOSA_BF16) {
    int32_t rc = ensure_tensor_maps(c, kv);
    if (rc != LOSA_OK) return rc;
  }
  AttnParams ap;
  ap.q = q;
  ap.k_pages = kv->k_pages;
  ap.v_pages = kv->v_pages;
  ap.stride_page = kv->stride_page;
  ap.stride_head = kv->stride_head;
  ap.stride_tok = kv->stride_tok;
  ap.page_table = kv->page_table;
  ap.kv_len = kv->kv_len;
  ap.active_idx = active_idx;
  ap.n_active = n_active;
  ap.union_pages = union_pages;
  ap.union_count = union_count;
  ap.partials = reinterpret_cast<float*>(c->ws + c->lay.partials);
  ap.seg_prefix = reinterpret_cast<int32_t*>(c->ws + c->lay.seg_prefix);
  ap.o_p = state->o_p;
  ap.o_p_bf16 = state->o_p_format == LOSA_STATE_BF16 ? 1 : 0;
  ap.lse_p = state->lse_p;
  ap.status = status_ptr(c);
  const bool fp8 = kv->kv_format == LOSA_KV_FP8_E4M3;
  ap.k_scale = fp8 ? kv->k_scale : nullptr;
  ap.v_scale = fp8 ? kv->v_scale : nullptr;
  ap.N = sh.batch;
  ap.B = sh.block_size;
  ap.Hq = sh.n_q_heads;
  ap.Hkv = sh.n_kv_heads;
  ap.G = sh.n_q_heads / sh.n_kv_heads;
  ap.Pmax = sh.max_pages_per_seq;
  ap.n_phys = kv->n_phys_pages;
  ap.n_rg = c->lay.n_row_groups;
  ap.n_seg = c->lay.n_segments;
  ap.n_ctas = c->lay.n_ctas;
  ap.sm_scale = sh.sm_scale;
  ap.wait_cycles = c->wait_cycles > 0 ? c->wait_cycles : kWaitCycles;
  const bool with_combine = !(defer_combine && finish_fuses_combine(c));
  return sh.head_dim == 128 ? dispatch_page<128>(c, ap, st, with_combine) : dispatch_page<64>(c, ap, st, with_combine);
}

bool finish_fuses_combine(const losa_ctx* c) { return c->shape.dtype == LOSA_BF16; }

int32_t launch_attn_finish(losa_ctx* c, const void* q, const int32_t* active_idx, const int32_t* n_active,
                           const int32_t* slot_map,
                           losa_state_t* state, void* out, float* lse_out_opt, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  AttnParams ap = {};
  ap.active_idx = active_idx;
  ap.n_active = n_active;
  ap.partials = reinterpret_cast<float*>(c->ws + c->lay.partials);
  ap.seg_prefix = reinterpret_cast<int32_t*>(c->ws + c->lay.seg_prefix);
  ap.o_p = state->o_p;
  ap.o_p_bf16 = state->o_p_format == LOSA_STATE_BF16 ? 1 : 0;
  ap.lse_p = state->lse_p;
  ap.status = status_ptr(c);
  ap.N = sh.batch;
  ap.B = sh.block_size;
  ap.Hq = sh.n_q_heads;
  ap.Hkv = sh.n_kv_heads;
  ap.G = sh.n_q_heads / sh.n_kv_heads;
  ap.n_rg = c->lay.n_row_groups;
  ap.n_seg = c->lay.n_segments;
  ap.n_ctas = c->lay.n_ctas;
  FinishParams fp;
  fp.q = q;
  fp.slot_map = slot_map;
  fp.q_prev = state->q_prev;
  fp.o_b = reinterpret_cast<const float*>(c->ws + c->lay.block_o);
  fp.lse_b = reinterpret_cast<const float*>(c->ws + c->lay.block_lse);
  fp.out = out;
  fp.lse_out = lse_out_opt;
  fp.step = state->step;
  fp.n_rows = static_cast<size_t>(sh.batch) * sh.block_size * sh.n_q_heads;
  const int blocks = static_cast<int>((fp.n_rows + kFinishThreads / 32 - 1) / (kFinishThreads / 32));
  if (sh.head_dim == 128) launch_k(attn_finish_kernel<__nv_bfloat16, 128>, blocks, kFinishThreads, 0, st, ap, fp);
  else launch_k(attn_finish_kernel<__nv_bfloat16, 64>, blocks, kFinishThreads, 0, st, ap, fp);
  return after_launch(c);
}

}  // namespace losa
