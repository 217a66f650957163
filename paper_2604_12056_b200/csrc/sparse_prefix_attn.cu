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
// bf16 kernel: four producer warps resolve union position -> logical page -> physical page two
//   batches ahead and stream each page's K and V slice into a ring of shared-memory stages with
//   TMA tensor copies (128-byte swizzle, completion on an mbarrier); eight consumer warps run
//   Q K^T and P V on the tensor cores (bf16 m16n8k16, fp32 accumulate) straight from the swizzled
//   tiles with ldmatrix, with an online softmax in registers.  Query rows are the GQA-grouped
//   (active token, head) pairs of the KV head: 16-row tiles; with few rows the eight warps take
//   different pages of the ring, with many rows they take different row tiles of the same page.
//   Consumer warps never synchronise with each other: each keeps its own (m, l, o), reads its own
//   query fragments from global memory and writes its own 16-row record per (CTA, segment) piece.
// fp32 kernel: CUDA cores, fp32 FMA (bf16 tensor cores cannot meet the 1e-5 fp32 tolerance).
//
// Every wait on an mbarrier is bounded; when a bound runs out the CTA records LOSA_ERR_TIMEOUT,
// stops computing and still walks every barrier so that no thread is left behind.
#include <cuda.h>

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
  float* o_p;
  float* lse_p;
  int32_t* status;
  int N, B, Hq, Hkv, G, Pmax, n_phys, n_rg, n_seg, n_ctas;
  float sm_scale;
#ifdef LOSA_TRACE
  unsigned long long* trace;   // [n_ctas][8] timestamps, development builds only
#endif
};

#ifdef LOSA_TRACE
__device__ __forceinline__ unsigned long long gtime() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
#define LOSA_STAMP(slot) do { if (p.trace) p.trace[blockIdx.x * 8 + (slot)] = gtime(); } while (0)
#else
#define LOSA_STAMP(slot) do { } while (0)
#endif

// Partial results.  A slot (CTA b, segment seg -> b + seg) holds eight records of one 16-row tile
// each: m[16], l[16], o[16][D] (un-normalised, relative to m).  The tensor-core kernel writes one
// record per consumer warp; the fp32 kernel writes record t for rows 16t .. 16t+15.
constexpr int kTileRows = 16;
__device__ __forceinline__ float* record_base(float* partials, int slot, int w, int D) {
  return partials + (static_cast<size_t>(slot) * 8 + w) * kTileRows * (D + 2);
}
// How the eight consumer warps split a segment with `rows` query rows: nrtp row tiles (padded to a
// power of two) times ns = 8 / nrtp page slots.
__device__ __forceinline__ int row_tiles_padded(int rows) {
  const int nrt = (rows + kTileRows - 1) / kTileRows;
  return nrt <= 1 ? 1 : (nrt <= 2 ? 2 : (nrt <= 4 ? 4 : 8));
}

__device__ __forceinline__ int clamp_active(int na, int B) { return na < 0 ? 0 : (na > B ? B : na); }

// ===================================================================== fp32 / CUDA-core kernel
template <typename T, int D, int GP>
__global__ void __launch_bounds__(256, 1) attn_simt_kernel(AttnParams p) {
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
    const int rg = sg % p.n_rg, sk = sg / p.n_rg, s = sk / p.Hkv, kh = sk % p.Hkv;
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
// grid (n_seg, 16): warp = one query row of the segment's row group.  The CTAs whose item range
// meets the segment are consecutive; each of them left up to `ns` records for the row's tile (one
// per page slot).  Lanes take one (piece, slot) pair each for the row maxima and sums, then the
// warp walks the pairs with the loads of four records issued together.  LOG2: partial maxima in
// base-2 units (tensor-core kernel) or natural units (fp32 kernel, which writes one record per
// row tile: SIMT).
template <int D, bool LOG2, bool SIMT>
__global__ void __launch_bounds__(256) attn_combine_kernel(AttnParams p) {
  __shared__ int pre[kMaxSegments + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sg = blockIdx.x, r = blockIdx.y * 8 + warp;
  const int rg = sg % p.n_rg, sk = sg / p.n_rg, s = sk / p.Hkv, kh = sk % p.Hkv;
  const int rows = rows_in_group(clamp_active(p.n_active[s], p.B), p.G, rg);
  if (blockIdx.y * 8 >= rows) return;                 // whole CTA idle: skip the prefix as well
  if (warp == 0) segment_prefix(pre, p.n_seg, p.n_rg, p.Hkv, p.G, p.n_active, p.union_count, p.B, lane);
  __syncthreads();
  if (r >= rows) return;
  const int row = rg * kRowsPerGroup + r, a = row / p.G, gi = row % p.G;
  const int tok = p.active_idx[s * p.B + a];
  if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); return; }
  const size_t orow = (static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + gi;
  const int start = pre[sg], end = pre[sg + 1];
  const long long T_all = pre[p.n_seg];
  const int nrtp = SIMT ? 8 : row_tiles_padded(rows), ns = 8 / nrtp;
  const int tile = r / kTileRows, rr = r % kTileRows;
  constexpr int C = D / 32;
  float acc[C];
#pragma unroll
  for (int c = 0; c < C; ++c) acc[c] = 0.f;
  float M = -INFINITY, Lsum = 0.f;
  if (end > start) {
    int b0 = static_cast<int>((static_cast<long long>(start) * p.n_ctas) / T_all);
    while (b0 + 1 < p.n_ctas && cta_lo(T_all, b0 + 1, p.n_ctas) <= start) ++b0;
    int b1 = static_cast<int>((static_cast<long long>(end - 1) * p.n_ctas) / T_all);   // last CTA that can meet it
    while (b1 + 1 < p.n_ctas && cta_lo(T_all, b1 + 1, p.n_ctas) < end) ++b1;
    const int n_pairs = (b1 - b0 + 1) * ns;
    // record of pair x (piece x / ns, page slot x % ns), or null when that warp had no page
    auto record_of = [&](int x) -> const float* {
      if (x >= n_pairs) return nullptr;
      const int b = b0 + x / ns, sl = x % ns;
      const long long lo = max(cta_lo(T_all, b, p.n_ctas), static_cast<long long>(start));
      const long long hi = min(cta_lo(T_all, b + 1, p.n_ctas), static_cast<long long>(end));
      if (hi - lo <= sl) return nullptr;              // fewer pages in the piece than this slot index
      return record_base(p.partials, b + sg, tile + nrtp * sl, D);
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
      constexpr int U = 8;                            // records whose loads are in flight together
      for (int i0 = 0; i0 < n; i0 += U) {
        float w[U], v[U][C];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int i = i0 + u;
          w[u] = (i < n) ? __shfl_sync(0xffffffffu, wj, i & 31) : 0.f;
          const unsigned long long addr = __shfl_sync(0xffffffffu, reinterpret_cast<unsigned long long>(rec), i & 31);
          const float* src = reinterpret_cast<const float*>(addr) + 2 * kTileRows + rr * D + lane;
#pragma unroll
          for (int c = 0; c < C; ++c) v[u][c] = (w[u] != 0.f) ? src[32 * c] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
          for (int c = 0; c < C; ++c) acc[c] = fmaf(v[u][c], w[u], acc[c]);
      }
    }
  }
  const bool empty = !(Lsum > 0.f);
  const float inv = empty ? 0.f : 1.f / Lsum;
#pragma unroll
  for (int c = 0; c < C; ++c) p.o_p[orow * D + lane + 32 * c] = acc[c] * inv;
  if (lane == 0) p.lse_p[orow] = empty ? -INFINITY : (LOG2 ? (M + log2f(Lsum)) * kLn2 : M + logf(Lsum));
}

// ===================================================================== bf16 TMA + tensor-core kernel
constexpr int kConsumerWarps = 8;
constexpr int kProducerWarps = 4;    // registers are allocated per 4 warps: 9 warps would cost the same as 12
constexpr int kMmaThreads = (kConsumerWarps + kProducerWarps) * 32;
constexpr long long kWaitCycles = 2000000000ll;   // ~1 s: bound of every mbarrier wait
constexpr int kSmemBudget = 232448;                // 227 KB opt-in limit per CTA

template <int D, int GP> constexpr int stage_bytes() { return 2 * GP * D * 2; }
constexpr int kStageIdx = 1024;     // active_idx entries (N * B) cached in shared memory when they fit
constexpr int kStageSeq = 64;       // ... together with n_active and kv_len of up to this many sequences
constexpr int kTailBytes = 512 + (kMaxSegments + 1) * 4 + 4 + kStageIdx * 4 + 2 * kStageSeq * 4;   // barriers, meta, prefix, index cache
template <int D, int GP> constexpr int n_stages() {
  const int n = (kSmemBudget - 1024 - kTailBytes) / stage_bytes<D, GP>();
  return n > 16 ? 16 : n;
}
template <int D, int GP> constexpr int mma_smem_bytes() {
  return 1024 + n_stages<D, GP>() * stage_bytes<D, GP>() + kTailBytes;
}

__device__ __forceinline__ uint32_t smem_u32(const void* ptr) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(ptr));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) when the bound runs out or
// another warp has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      set_status(status, LOSA_ERR_TIMEOUT);
      return false;
    }
  }
}
// Bounded wait until the producer has tagged the stage with `round`.
__device__ __forceinline__ bool wait_round(volatile int* tag, int round, volatile int* abort_flag,
                                           int32_t* status) {
  if (*tag == round) return true;
  const long long t0 = clock64();
  while (*tag != round) {
    __nanosleep(64);                 // the producers share this SM's issue slots: do not spin hot
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitCycles) {
      *abort_flag = 1;
      set_status(status, LOSA_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}
// Loads whose issue point must stay where it is written (they are prefetches): volatile asm.
__device__ __forceinline__ int ld_nc_s32(const int32_t* ptr) {
  int v;
  asm volatile("ld.global.nc.s32 %0, [%1];" : "=r"(v) : "l"(ptr));
  return v;
}
__device__ __forceinline__ uint32_t ld_nc_u32(const uint32_t* ptr) {
  uint32_t v;
  asm volatile("ld.global.nc.b32 %0, [%1];" : "=r"(v) : "l"(ptr));
  return v;
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 2^x, one MUFU instruction (ex2.approx: 2 ulp; -inf -> 0); the bf16 rounding of P dwarfs its error
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Byte offset of 16-byte chunk `chunk` (0 .. D/8-1) of token row `t` inside a K or V tile that TMA
// wrote as D/64 boxes of [GP rows][64 bf16] with the 128-byte swizzle.
template <int GP>
__device__ __forceinline__ uint32_t tile_off(int t, int chunk) {
  return static_cast<uint32_t>((chunk >> 3) * (GP * 128) + t * 128 + (((chunk & 7) ^ (t & 7)) << 4));
}

template <int D, int GP>
__global__ void __launch_bounds__(kMmaThreads, 1)
attn_mma_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, AttnParams p) {
  constexpr int NSTAGE = n_stages<D, GP>();
  constexpr int STAGE = stage_bytes<D, GP>();
  constexpr int KBYTES = GP * D * 2;
  constexpr int NT = GP / 8;        // score n-tiles per page
  constexpr int KS = D / 16;        // k-steps of Q K^T
  constexpr int ND = D / 8;         // output n-tiles
  constexpr int OREGS = ND * 4;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - raw);                 // generic pointer to the same place
  const uint32_t stage0 = base;
  uint8_t* tail = gen + NSTAGE * STAGE;
  const uint32_t full0 = base + NSTAGE * STAGE;          // full[NSTAGE], then empty[NSTAGE]
  const uint32_t empty0 = full0 + 8 * NSTAGE;
  volatile int* meta = reinterpret_cast<volatile int*>(tail + 16 * NSTAGE);        // valid tokens per stage
  volatile int* stage_round = meta + NSTAGE;   // which pass over the ring the stage's current page belongs to
  volatile int* abort_flag = stage_round + NSTAGE;
  int* pre = reinterpret_cast<int*>(tail + 512);
  int* tok_s = pre + kMaxSegments + 2;          // [N][B] active_idx, when staged
  int* na_s = tok_s + kStageIdx;                // [N] clamped n_active
  int* len_s = na_s + kStageSeq;                // [N] kv_len
  const bool staged = p.N * p.B <= kStageIdx && p.N <= kStageSeq;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) LOSA_STAMP(0);
  if (tid == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      mbar_init(full0 + 8 * i, 1);
      mbar_init(empty0 + 8 * i, kConsumerWarps);
      stage_round[i] = -1;
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) {
    segment_prefix(pre, p.n_seg, p.n_rg, p.Hkv, p.G, p.n_active, p.union_count, p.B, lane);
  } else if (staged) {
    // The small index arrays are read now, while the memory system is idle: once the page stream
    // saturates it, every dependent global load costs microseconds of queueing.
    for (int i = tid - 32; i < p.N * p.B; i += kMmaThreads - 32) tok_s[i] = p.active_idx[i];
    for (int i = tid - 32; i < p.N; i += kMmaThreads - 32) {
      na_s[i] = clamp_active(p.n_active[i], p.B);
      len_s[i] = p.kv_len[i];
    }
  }
  __syncthreads();
  const long long T_all = pre[p.n_seg];
  const int lo = static_cast<int>(cta_lo(T_all, blockIdx.x, p.n_ctas));
  const int hi = static_cast<int>(cta_lo(T_all, blockIdx.x + 1, p.n_ctas));
  if (lo >= hi) return;
  int sg0 = 0;
  while (pre[sg0 + 1] <= lo) ++sg0;
  if (tid == 0) LOSA_STAMP(1);
  auto n_active_of = [&](int s) { return staged ? na_s[s] : clamp_active(p.n_active[s], p.B); };
  auto kv_len_of = [&](int s) { return staged ? len_s[s] : p.kv_len[s]; };
  auto token_of = [&](int s, int a) { return staged ? tok_s[s * p.B + a] : p.active_idx[s * p.B + a]; };

  if (warp >= kConsumerWarps) {
    // ------------------------------------------------------------------ producer warp
    // Issuing a page (four tensor copies plus barrier traffic) costs one thread ~0.3 us, more than
    // the 0.37 us the HBM needs to deliver it, so kProducerWarps warps share the work: producer w
    // takes the CTA's items w, w + kProducerWarps, ...  Lane j of a batch of 32 such items resolves
    // item -> logical page -> physical page.  The two loads depend on each other, so they run as a
    // pipeline over batches: while the copies of batch k are issued, the physical pages of batch
    // k+1 and the logical pages of batch k+2 are in flight.
    const int pw = warp - kConsumerWarps;
    constexpr int STEP = 32 * kProducerWarps;       // items covered by one batch of every producer
    int cursor = sg0;                               // segment cursor of the first pipeline stage
    int page_a = -1, sk_a = 0;                      // batch k+1: logical page (loaded) and its (sequence, KV head)
    int phys_b = 0, kh_b = 0, valid_b = 0;          // batch k  : ready to issue
    auto stage_a = [&](int i, int& page, int& sk) {
      page = -1; sk = 0;
      if (i < hi) {
        while (pre[cursor + 1] <= i) ++cursor;
        sk = cursor / p.n_rg;
        page = ld_nc_s32(p.union_pages + static_cast<size_t>(sk) * p.Pmax + (i - pre[cursor]));
      }
    };
    auto stage_b = [&](int i, int page, int sk, int& phys, int& kh, int& valid) {
      phys = 0; kh = 0; valid = 0;
      if (i < hi) {
        const int s = sk / p.Hkv;
        kh = sk % p.Hkv;
        const bool ok = page >= 0 && page < p.Pmax;
        phys = ok ? ld_nc_s32(p.page_table + static_cast<size_t>(s) * p.Pmax + page) : -1;
        valid = ok ? min(GP, kv_len_of(s) - page * GP) : 0;
      }
    };
    const int mine = lo + pw + kProducerWarps * lane;        // this lane's item in the first batch
    stage_a(mine, page_a, sk_a);
    stage_b(mine, page_a, sk_a, phys_b, kh_b, valid_b);
    stage_a(mine + STEP, page_a, sk_a);
    for (int b0 = lo; b0 + pw < hi; b0 += STEP) {
      int page_n, sk_n, phys_n, kh_n, valid_n;
      const int i_lane = b0 + pw + kProducerWarps * lane;
      stage_a(i_lane + 2 * STEP, page_n, sk_n);
      stage_b(i_lane + STEP, page_a, sk_a, phys_n, kh_n, valid_n);
      if (i_lane < hi && (phys_b < 0 || phys_b >= p.n_phys || valid_b <= 0)) {
        set_status(p.status, LOSA_ERR_BOUNDS);
        phys_b = 0;
        valid_b = 0;
      }
      const int nb = min(32, (hi - b0 - pw + kProducerWarps - 1) / kProducerWarps);
      for (int j = 0; j < nb; ++j) {
        const int ph = __shfl_sync(0xffffffffu, phys_b, j);
        const int khj = __shfl_sync(0xffffffffu, kh_b, j);
        const int vj = __shfl_sync(0xffffffffu, valid_b, j);
        if (lane == 0) {
          const int it = b0 + pw + kProducerWarps * j - lo, stage = it % NSTAGE, round = it / NSTAGE;
          // Another producer fills this stage in the previous pass over the ring; until it has
          // done so (tag == round - 1) the parity wait below would look at the wrong phase.
          const bool go = (round == 0 || wait_round(stage_round + stage, round - 1, abort_flag, p.status)) &&
                          mbar_wait(empty0 + 8 * stage, (round & 1) ^ 1, abort_flag, p.status);
          if (go) {
#ifdef LOSA_TRACE
            if (p.trace && it < 80) p.trace[p.n_ctas * 34 + (blockIdx.x * 80 + it) * 2] = gtime();
#endif
            if (it == 0) LOSA_STAMP(7);                  // about to issue the first copy
            if (it == NSTAGE - 1) LOSA_STAMP(2);         // ring filled once without waiting
            meta[stage] = vj;
            stage_round[stage] = round;
            const uint32_t fb = full0 + 8 * stage, dst = stage0 + stage * STAGE;
            mbar_expect_tx(fb, STAGE);
#pragma unroll
            for (int hf = 0; hf < D / 64; ++hf) {
              tma_load_4d(dst + hf * (GP * 128), &tmK, fb, hf * 64, 0, khj, ph);
              tma_load_4d(dst + KBYTES + hf * (GP * 128), &tmV, fb, hf * 64, 0, khj, ph);
            }
          }
        }
      }
      page_a = page_n; sk_a = sk_n;
      phys_b = phys_n; kh_b = kh_n; valid_b = valid_n;
    }
    if (lane == 0 && pw == 0) LOSA_STAMP(3);         // producer 0 has issued all its copies
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  // Each warp is on its own: it reads its query fragments straight from global memory, keeps its own
  // running (m, l, o) and leaves its own 16-row record per piece; no barrier ties the warps of a
  // CTA together, so a change of segment stalls one warp for one memory latency, nothing else.
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q);
  const int g8 = lane >> 2, q4 = lane & 3;
  const float scale2 = p.sm_scale * kLog2e;
  int sg = sg0, item = lo;
#ifdef LOSA_TRACE
  long long trace_wait = 0, trace_busy = 0;
#endif
  // How this warp takes part in the piece of segment `g` that starts at item `first`.
  struct Piece { int seg_end, npg, rows, nrt, nrtp, ns, rt, slot, s, kh, rg; bool has_rows, works; };
  auto piece_of = [&](int g, int first) {
    Piece c;
    c.seg_end = min(hi, pre[g + 1]);
    c.npg = c.seg_end - first;
    c.rg = g % p.n_rg;
    const int sk = g / p.n_rg;
    c.s = sk / p.Hkv;
    c.kh = sk % p.Hkv;
    c.rows = rows_in_group(n_active_of(c.s), p.G, c.rg);
    c.nrt = (c.rows + kTileRows - 1) / kTileRows;
    c.nrtp = row_tiles_padded(c.rows);
    c.ns = kConsumerWarps / c.nrtp;
    c.rt = warp % c.nrtp;
    c.slot = warp / c.nrtp;
    c.has_rows = c.rt < c.nrt;
    c.works = c.has_rows && c.slot < c.npg;
    return c;
  };
  // Row pointers of this lane's two rows (rt*16 + g8, +8) of a piece, null for padding rows.
  auto row_ptrs = [&](const Piece& c, const uint32_t* (&rowp)[2]) {
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow) {
      const int r = c.rt * kTileRows + g8 + 8 * hrow;
      rowp[hrow] = nullptr;
      if (c.works && r < c.rows) {
        const int row = c.rg * kRowsPerGroup + r, a = row / p.G, gi = row % p.G;
        int tok = token_of(c.s, a);
        if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); tok = 0; }
        rowp[hrow] = reinterpret_cast<const uint32_t*>(q + ((static_cast<size_t>(c.s) * p.B + tok) * p.Hq + c.kh * p.G + gi) * D);
      }
    }
  };
  // Pulls the query rows of a later piece into L2 (no registers held).
  auto prefetch_q = [&](const Piece& c) {
    const uint32_t* rowp[2];
    row_ptrs(c, rowp);
#pragma unroll
    for (int hrow = 0; hrow < 2; ++hrow)
      if (rowp[hrow] && q4 < (D * 2 + 127) / 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(rowp[hrow]) + q4 * 128));
  };
  // A fragments: 4-byte loads of two adjacent bf16, zero for padding rows.
  auto load_q = [&](const Piece& c, uint32_t (&dst)[KS][4]) {
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) { dst[ks][0] = dst[ks][1] = dst[ks][2] = dst[ks][3] = 0u; }
    const uint32_t* rowp[2];
    row_ptrs(c, rowp);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int w0 = ks * 8 + q4;                     // 32-bit word index of columns ks*16 + q4*2
      if (rowp[0]) { dst[ks][0] = ld_nc_u32(rowp[0] + w0); dst[ks][2] = ld_nc_u32(rowp[0] + w0 + 4); }
      if (rowp[1]) { dst[ks][1] = ld_nc_u32(rowp[1] + w0); dst[ks][3] = ld_nc_u32(rowp[1] + w0 + 4); }
    }
  };
  Piece cur = piece_of(sg, item);
  uint32_t qf[KS][4];
  load_q(cur, qf);
  while (item < hi) {
    const int seg_end = cur.seg_end, npg = cur.npg, ns = cur.ns, slot = cur.slot;
    const bool has_rows = cur.has_rows, works = cur.works;
    // The next piece's query rows are pulled into L2 now and loaded after this piece's pages: a
    // miss then would cost microseconds, because the page stream keeps the memory queues full.
    int sg_next = sg + 1;
    while (seg_end < hi && pre[sg_next + 1] <= seg_end) ++sg_next;
    Piece nxt = cur;
    if (seg_end < hi) {
      nxt = piece_of(sg_next, seg_end);
      prefetch_q(nxt);
    }

    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float oacc[ND][4];
#pragma unroll
    for (int n = 0; n < ND; ++n) { oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f; }
    // Page j of the piece belongs to the warps of page slot j % ns (one warp per row tile).  Only
    // they wait for it and release it, each with weight ns, so that a stage always collects
    // kConsumerWarps arrivals and is refilled as soon as ITS readers are done with it.
    for (int j = slot; j < npg; j += ns) {
      const int it = item + j - lo, stage = it % NSTAGE, round = it / NSTAGE;
      // A parity wait is only meaningful once the stage is in this item's pass over the ring:
      // this warp may get here while the stage's previous page is still in flight.
#ifdef LOSA_TRACE
      const long long tw0 = clock64();
#endif
      const bool ready = wait_round(stage_round + stage, round, abort_flag, p.status) &&
                         mbar_wait(full0 + 8 * stage, round & 1, abort_flag, p.status);
#ifdef LOSA_TRACE
      const long long tw1 = clock64();
      trace_wait += tw1 - tw0;
      if (lane == 0 && p.trace && it < 80) p.trace[p.n_ctas * 34 + (blockIdx.x * 80 + it) * 2 + 1] = gtime();
#endif
      if (tid == 0 && it == 0) LOSA_STAMP(4);        // first page landed
      if (ready && has_rows) {
        const int valid = meta[stage];
        const uint32_t kt = stage0 + stage * STAGE, vt = kt + KBYTES;
        if (valid < GP) {
          // rows of V past the end of the prefix may hold anything (even NaN): clear them
          uint8_t* vg = gen + stage * STAGE + KBYTES;
          for (int idx = lane; idx < (GP - valid) * (D / 8); idx += 32) {
            const int t = valid + idx / (D / 8), ch = idx % (D / 8);
            *reinterpret_cast<uint4*>(vg + tile_off<GP>(t, ch)) = make_uint4(0u, 0u, 0u, 0u);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          __syncwarp();
        }
        // ---- S = Q K^T.  The K fragments of k-step ks+1 are requested before the MMAs of k-step
        // ks are issued, so shared-memory latency hides behind tensor-core work.
        float sacc[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) { sacc[n][0] = sacc[n][1] = sacc[n][2] = sacc[n][3] = 0.f; }
        const int mi = lane >> 3, l7 = lane & 7;
        {
          // row of the K tile this lane addresses for n-tile pair np is np*16 + krow; its chunk for
          // k-step ks is ks*2 + (mi & 1)
          const int krow = (mi >> 1) * 8 + l7;
          uint32_t kb[2][NT / 2][4];
#pragma unroll
          for (int np = 0; np < NT / 2; ++np) ldsm_x4(kt + tile_off<GP>(np * 16 + krow, (mi & 1)), kb[0][np]);
#pragma unroll
          for (int ks = 0; ks < KS; ++ks) {
            if (ks + 1 < KS) {
#pragma unroll
              for (int np = 0; np < NT / 2; ++np)
                ldsm_x4(kt + tile_off<GP>(np * 16 + krow, (ks + 1) * 2 + (mi & 1)), kb[(ks + 1) & 1][np]);
            }
#pragma unroll
            for (int np = 0; np < NT / 2; ++np) {
              mma_bf16(sacc[2 * np], qf[ks], kb[ks & 1][np][0], kb[ks & 1][np][1]);
              mma_bf16(sacc[2 * np + 1], qf[ks], kb[ks & 1][np][2], kb[ks & 1][np][3]);
            }
          }
        }
        // ---- online softmax (base-2 units), rows g8 and g8 + 8 of the tile.  Raw scores stay in
        // sacc; the scale is folded into the exponent: p = 2^(s * scale2 - m).
        if (valid < GP) {                                // only a sequence's last page can be partial
#pragma unroll
          for (int n = 0; n < NT; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e)
              if (n * 8 + q4 * 2 + (e & 1) >= valid) sacc[n][e] = -INFINITY;
        }
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          mx0 = fmaxf(mx0, fmaxf(sacc[n][0], sacc[n][1]));
          mx1 = fmaxf(mx1, fmaxf(sacc[n][2], sacc[n][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        // scale2 > 0, so the maximum of the scaled scores is the scaled maximum
        const float mn0 = fmaxf(m0, mx0 * scale2), mn1 = fmaxf(m1, mx1 * scale2);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float c0 = ex2(m0 - ms0), c1 = ex2(m1 - ms1);
        m0 = mn0; m1 = mn1;
        float s0 = 0.f, s1 = 0.f;
        uint32_t pa[GP / 16][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const float e0 = ex2(fmaf(sacc[n][0], scale2, -ms0)), e1 = ex2(fmaf(sacc[n][1], scale2, -ms0));
          const float e2 = ex2(fmaf(sacc[n][2], scale2, -ms1)), e3 = ex2(fmaf(sacc[n][3], scale2, -ms1));
          s0 += e0 + e1;
          s1 += e2 + e3;
          pa[n >> 1][(n & 1) * 2] = pack_bf16(e0, e1);
          pa[n >> 1][(n & 1) * 2 + 1] = pack_bf16(e2, e3);
        }
        l0 = l0 * c0 + s0;
        l1 = l1 * c1 + s1;
        if (__any_sync(0xffffffffu, c0 != 1.f || c1 != 1.f)) {      // rescale only when some row maximum moved
#pragma unroll
          for (int n = 0; n < ND; ++n) { oacc[n][0] *= c0; oacc[n][1] *= c0; oacc[n][2] *= c1; oacc[n][3] *= c1; }
        }
        // ---- O += P V, V fragments fetched two MMA pairs ahead
        {
          constexpr int NV = (GP / 16) * (ND / 2);       // ldmatrix.x4.trans loads per page
          const int vrow = (mi & 1) * 8 + l7;
          uint32_t vb[3][4];
          auto vload = [&](int i, uint32_t (&dst)[4]) {
            const int k2 = i / (ND / 2), np = i % (ND / 2);
            ldsm_x4_trans(vt + tile_off<GP>(k2 * 16 + vrow, np * 2 + (mi >> 1)), dst);
          };
          vload(0, vb[0]);
          if (NV > 1) vload(1, vb[1]);
#pragma unroll
          for (int i = 0; i < NV; ++i) {
            if (i + 2 < NV) vload(i + 2, vb[(i + 2) % 3]);
            const int k2 = i / (ND / 2), np = i % (ND / 2);
            mma_bf16(oacc[2 * np], pa[k2], vb[i % 3][0], vb[i % 3][1]);
            mma_bf16(oacc[2 * np + 1], pa[k2], vb[i % 3][2], vb[i % 3][3]);
          }
        }
      }
      __syncwarp();
#ifdef LOSA_TRACE
      trace_busy += clock64() - tw1;
#endif
      if (ready && lane == 0) mbar_arrive(empty0 + 8 * stage, static_cast<uint32_t>(ns));
    }

    if (tid == 0 && seg_end == hi) LOSA_STAMP(5);    // warp 0 done with its pages
#ifdef LOSA_TRACE
    const long long ts0 = clock64();
#endif
    // ---- this warp's un-normalised record for the piece
    if (works) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
      l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
      float* rec = record_base(p.partials, blockIdx.x + sg, warp, D);
      if (q4 == 0) {
        rec[g8] = m0; rec[g8 + 8] = m1;
        rec[kTileRows + g8] = l0; rec[kTileRows + g8 + 8] = l1;
      }
#pragma unroll
      for (int n = 0; n < ND; ++n) {
        *reinterpret_cast<float2*>(rec + 2 * kTileRows + g8 * D + n * 8 + q4 * 2) = make_float2(oacc[n][0], oacc[n][1]);
        *reinterpret_cast<float2*>(rec + 2 * kTileRows + (g8 + 8) * D + n * 8 + q4 * 2) = make_float2(oacc[n][2], oacc[n][3]);
      }
    }
    item = seg_end;
    sg = sg_next;
    if (item < hi) {
      cur = nxt;
      load_q(cur, qf);
#ifdef LOSA_TRACE
      if (lane == 0 && p.trace) p.trace[p.n_ctas * 26 + blockIdx.x * 8 + warp] = (clock64() - ts0) + ((long long)(qf[0][0] & 1) << 40);
#endif
    }
  }
  if (tid == 0) LOSA_STAMP(6);
#ifdef LOSA_TRACE
  if (lane == 0 && p.trace) { p.trace[p.n_ctas * 8 + (blockIdx.x * 8 + warp) * 2] = trace_wait; p.trace[p.n_ctas * 8 + (blockIdx.x * 8 + warp) * 2 + 1] = trace_busy; }
  if (tid == 0 && p.trace) { unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); p.trace[p.n_ctas * 24 + blockIdx.x * 2] = smid; p.trace[p.n_ctas * 24 + blockIdx.x * 2 + 1] = sg - sg0; }
#endif
}

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
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(kv->stride_tok) * 2, static_cast<cuuint64_t>(kv->stride_head) * 2,
                                 static_cast<cuuint64_t>(kv->stride_page) * 2};
  const cuuint32_t box[4] = {64, static_cast<cuuint32_t>(sh.page_size), 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = reinterpret_cast<EncodeTiledFn>(c->encode_fn)(
      reinterpret_cast<CUtensorMap*>(blob), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(pool), dims,
      strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
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
                    c->tmap_strides[2] == kv->stride_tok && c->tmap_n_phys == kv->n_phys_pages;
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
  return LOSA_OK;
}

template <int D, int GP>
int32_t launch_mma(losa_ctx* c, const AttnParams& ap, cudaStream_t st) {
  constexpr int smem = mma_smem_bytes<D, GP>();
  static_assert(n_stages<D, GP>() >= 3, "ring too shallow");
  static int attr_device = -1;   // the opt-in is per device and per kernel
  if (attr_device != c->device) {
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(attn_mma_kernel<D, GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    attr_device = c->device;
  }
  CUtensorMap mk, mv;
  memcpy(&mk, c->tmap_k, sizeof(mk));
  memcpy(&mv, c->tmap_v, sizeof(mv));
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_begin, st));
  attn_mma_kernel<D, GP><<<ap.n_ctas, kMmaThreads, smem, st>>>(mk, mv, ap);
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_end, st));
  int32_t rc = after_launch(c);
  if (rc != LOSA_OK) return rc;
  attn_combine_kernel<D, true, false><<<dim3(ap.n_seg, kRowsPerGroup / 8), 256, 0, st>>>(ap);
  return after_launch(c);
}

template <typename T, int D, int GP>
int32_t launch_simt(losa_ctx* c, const AttnParams& ap, cudaStream_t st) {
  const size_t smem = (static_cast<size_t>(2) * GP * D + 2 * kRowsPerGroup * D + 2 * kRowsPerGroup) * sizeof(float) +
                      (ap.n_seg + 1) * sizeof(int);
  LOSA_CUDA_TRY(c, cudaFuncSetAttribute(attn_simt_kernel<T, D, GP>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_begin, st));
  attn_simt_kernel<T, D, GP><<<ap.n_ctas, 256, smem, st>>>(ap);
  if (c->profile) LOSA_CUDA_TRY(c, cudaEventRecord(c->ev_end, st));
  int32_t rc = after_launch(c);
  if (rc != LOSA_OK) return rc;
  attn_combine_kernel<D, false, true><<<dim3(ap.n_seg, kRowsPerGroup / 8), 256, 0, st>>>(ap);
  return after_launch(c);
}

template <int D>
int32_t dispatch_page(losa_ctx* c, const AttnParams& ap, cudaStream_t st) {
  const bool bf = c->shape.dtype == LOSA_BF16;
  switch (c->shape.page_size) {
    case 16: return bf ? launch_mma<D, 16>(c, ap, st) : launch_simt<float, D, 16>(c, ap, st);
    case 32: return bf ? launch_mma<D, 32>(c, ap, st) : launch_simt<float, D, 32>(c, ap, st);
    default: return bf ? launch_mma<D, 64>(c, ap, st) : launch_simt<float, D, 64>(c, ap, st);
  }
}

}  // namespace

#ifdef LOSA_TRACE
unsigned long long* g_trace = nullptr;
extern "C" void losa_debug_set_trace(void* p) { g_trace = static_cast<unsigned long long*>(p); }
#endif

int32_t launch_sparse_prefix_attn(losa_ctx* c, const void* q, const losa_kv_t* kv,
                                  const int32_t* active_idx, const int32_t* n_active,
                                  const int32_t* union_pages, const int32_t* union_count,
                                  losa_state_t* state, cudaStream_t st) {
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
  ap.o_p = state->o_p;
  ap.lse_p = state->lse_p;
  ap.status = status_ptr(c);
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
#ifdef LOSA_TRACE
  ap.trace = g_trace;
#endif
  return sh.head_dim == 128 ? dispatch_page<128>(c, ap, st) : dispatch_page<64>(c, ap, st);
}

}  // namespace losa
