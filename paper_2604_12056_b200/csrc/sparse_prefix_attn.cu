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
// bf16 kernel: one producer warp resolves union position -> logical page -> physical page 32
//   items ahead and streams each page's K and V slice into a ring of shared-memory stages with
//   TMA tensor copies (128-byte swizzle, completion on an mbarrier); eight consumer warps run
//   Q K^T and P V on the tensor cores (bf16 m16n8k16, fp32 accumulate) straight from the swizzled
//   tiles with ldmatrix, with an online softmax in registers.  Query rows are the GQA-grouped
//   (active token, head) pairs of the KV head: 16-row tiles; with few rows the eight warps take
//   different pages of the ring, with many rows they take different row tiles of the same page.
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
  int B, Hq, Hkv, G, Pmax, n_phys, n_rg, n_seg, n_ctas;
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

__device__ __forceinline__ float* partial_base(float* partials, int slot, int D) {
  return partials + static_cast<size_t>(slot) * kRowsPerGroup * (D + 2);
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
    float* part = partial_base(p.partials, blockIdx.x + sg, D);
    for (int r = tid; r < rows; r += 256) { part[r] = Ms[r]; part[kRowsPerGroup + r] = Ls[r]; }
    for (int idx = tid; idx < rows * D; idx += 256) part[2 * kRowsPerGroup + idx] = Os[idx];
    item = seg_end;
    ++sg;
    while (item < hi && pre[sg + 1] <= item) ++sg;
  }
}

// ===================================================================== combine kernel
// grid (n_seg, 16): warp = one query row of the segment's row group.  The CTAs whose item range
// meets the segment are consecutive; lanes take one piece each for the row maxima and sums, then
// the warp walks the pieces with every load of a group of four issued together.  LOG2 says
// whether the partial maxima are in base-2 units (tensor-core kernel) or natural units (fp32).
template <int D, bool LOG2>
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
    // pass 1: the row maximum over the pieces
    for (int base = b0; base <= b1; base += 32) {
      const int b = base + lane;
      float mj = -INFINITY;
      if (b <= b1) {
        const long long lo = cta_lo(T_all, b, p.n_ctas), hi = cta_lo(T_all, b + 1, p.n_ctas);
        if (lo < end && hi > start && hi > lo) mj = partial_base(p.partials, b + sg, D)[r];
      }
      M = fmaxf(M, warp_max(mj));
    }
    // pass 2: weights, sum and output
    for (int base = b0; base <= b1; base += 32) {
      const int b = base + lane;
      float wj = 0.f, lj = 0.f;
      if (b <= b1) {
        const long long lo = cta_lo(T_all, b, p.n_ctas), hi = cta_lo(T_all, b + 1, p.n_ctas);
        if (lo < end && hi > start && hi > lo) {
          const float* part = partial_base(p.partials, b + sg, D);
          const float mj = part[r];
          wj = (mj == -INFINITY) ? 0.f : (LOG2 ? exp2f(mj - M) : expf(mj - M));
          lj = part[kRowsPerGroup + r];
        }
      }
      Lsum += warp_sum(lj * wj);
      const int n = min(32, b1 - base + 1);
      for (int i0 = 0; i0 < n; i0 += 4) {
        float w[4], v[4][C];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int i = i0 + u;
          w[u] = (i < n) ? __shfl_sync(0xffffffffu, wj, i & 31) : 0.f;
          const float* src = partial_base(p.partials, base + i + sg, D) + 2 * kRowsPerGroup + r * D + lane;
#pragma unroll
          for (int c = 0; c < C; ++c) v[u][c] = (w[u] != 0.f) ? src[32 * c] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
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
constexpr int kMmaThreads = (kConsumerWarps + 1) * 32;
constexpr long long kWaitCycles = 2000000000ll;   // ~1 s: bound of every mbarrier wait
constexpr int kSmemBudget = 232448;                // 227 KB opt-in limit per CTA

template <int D> constexpr int q_stride_bytes() { return D * 2 + 16; }
template <int D> constexpr int q_region_bytes() { return kRowsPerGroup * q_stride_bytes<D>(); }
template <int D, int GP> constexpr int stage_bytes() { return 2 * GP * D * 2; }
constexpr int kTailBytes = 512 + (kMaxSegments + 1) * 4;   // barriers, per-stage meta, flags, prefix
template <int D, int GP> constexpr int n_stages() {
  const int n = (kSmemBudget - 1024 - q_region_bytes<D>() - kTailBytes) / stage_bytes<D, GP>();
  return n > 16 ? 16 : n;
}
template <int D, int GP> constexpr int mma_smem_bytes() {
  return 1024 + n_stages<D, GP>() * stage_bytes<D, GP>() + q_region_bytes<D>() + kTailBytes;
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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

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
  constexpr int QSTR = q_stride_bytes<D>();
  constexpr int OREGS = ND * 4;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;          // swizzled tiles need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - raw);                 // generic pointer to the same place
  const uint32_t stage0 = base;
  const uint32_t qs = base + NSTAGE * STAGE;
  uint8_t* qs_gen = gen + NSTAGE * STAGE;
  uint8_t* tail = qs_gen + q_region_bytes<D>();
  const uint32_t full0 = qs + q_region_bytes<D>();       // full[NSTAGE], then empty[NSTAGE]
  const uint32_t empty0 = full0 + 8 * NSTAGE;
  volatile int* meta = reinterpret_cast<volatile int*>(tail + 16 * NSTAGE);        // valid tokens per stage
  volatile int* stage_round = meta + NSTAGE;   // which pass over the ring the stage's current page belongs to
  volatile int* abort_flag = stage_round + NSTAGE;
  int* pre = reinterpret_cast<int*>(tail + 512);

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
  if (warp == 0) segment_prefix(pre, p.n_seg, p.n_rg, p.Hkv, p.G, p.n_active, p.union_count, p.B, lane);
  __syncthreads();
  const long long T_all = pre[p.n_seg];
  const int lo = static_cast<int>(cta_lo(T_all, blockIdx.x, p.n_ctas));
  const int hi = static_cast<int>(cta_lo(T_all, blockIdx.x + 1, p.n_ctas));
  if (lo >= hi) return;
  int sg0 = 0;
  while (pre[sg0 + 1] <= lo) ++sg0;
  if (tid == 0) LOSA_STAMP(1);

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer warp
    int sg = sg0;
    for (int b0 = lo; b0 < hi; b0 += 32) {
      const int i = b0 + lane;
      int phys = 0, kh = 0, valid = 0;
      if (i < hi) {
        while (pre[sg + 1] <= i) ++sg;
        const int u = i - pre[sg], sk = sg / p.n_rg, s = sk / p.Hkv;
        kh = sk % p.Hkv;
        const int page = p.union_pages[static_cast<size_t>(sk) * p.Pmax + u];
        bool ok = page >= 0 && page < p.Pmax;
        phys = ok ? p.page_table[static_cast<size_t>(s) * p.Pmax + page] : 0;
        ok = ok && phys >= 0 && phys < p.n_phys;
        valid = ok ? min(GP, p.kv_len[s] - page * GP) : 0;
        if (!ok || valid <= 0) { set_status(p.status, LOSA_ERR_BOUNDS); phys = 0; valid = 0; }
      }
      const int nb = min(32, hi - b0);
      for (int j = 0; j < nb; ++j) {
        const int ph = __shfl_sync(0xffffffffu, phys, j);
        const int khj = __shfl_sync(0xffffffffu, kh, j);
        const int vj = __shfl_sync(0xffffffffu, valid, j);
        if (lane == 0) {
          const int it = b0 + j - lo, stage = it % NSTAGE, round = it / NSTAGE;
          const bool go = mbar_wait(empty0 + 8 * stage, (round & 1) ^ 1, abort_flag, p.status);
          if (go) {
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
      sg = __shfl_sync(0xffffffffu, sg, nb - 1);
    }
    if (lane == 0) LOSA_STAMP(3);                    // all copies issued
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(p.q);
  const int g8 = lane >> 2, q4 = lane & 3;
  const float scale2 = p.sm_scale * kLog2e;
  int sg = sg0, item = lo;
#ifdef LOSA_TRACE
  long long trace_wait = 0, trace_busy = 0;
#endif
  while (item < hi) {
    const int seg_end = min(hi, pre[sg + 1]);
    const int npg = seg_end - item;
    const int rg = sg % p.n_rg, sk = sg / p.n_rg, s = sk / p.Hkv, kh = sk % p.Hkv;
    const int rows = rows_in_group(clamp_active(p.n_active[s], p.B), p.G, rg);
    const int nrt = (rows + 15) >> 4;
    const int nrtp = nrt <= 1 ? 1 : (nrt <= 2 ? 2 : (nrt <= 4 ? 4 : 8));
    const int ns = kConsumerWarps / nrtp;
    const int rt = warp % nrtp, slot = warp / nrtp;
    const bool has_rows = rt < nrt;

    // ---- gather the query rows of this row group (16-byte chunks, padded row stride)
    consumer_bar();
    for (int idx = tid; idx < nrtp * 16 * (D / 8); idx += kConsumerWarps * 32) {
      const int r = idx / (D / 8), ch = idx % (D / 8);
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (r < rows) {
        const int row = rg * kRowsPerGroup + r, a = row / p.G, gi = row % p.G;
        int tok = p.active_idx[s * p.B + a];
        if (tok < 0 || tok >= p.B) { set_status(p.status, LOSA_ERR_BOUNDS); tok = 0; }
        v = *reinterpret_cast<const uint4*>(q + ((static_cast<size_t>(s) * p.B + tok) * p.Hq + kh * p.G + gi) * D + ch * 8);
      }
      *reinterpret_cast<uint4*>(qs_gen + r * QSTR + ch * 16) = v;
    }
    consumer_bar();
    uint32_t qf[KS][4];
    {
      const int mi = lane >> 3, r = rt * 16 + (mi & 1) * 8 + (lane & 7);
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) ldsm_x4(qs + r * QSTR + (ks * 2 + (mi >> 1)) * 16, qf[ks]);
    }
    consumer_bar();   // the Q region now doubles as scratch for the cross-warp merge

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
        // ---- online softmax (base-2 units), rows g8 and g8 + 8 of the tile
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int col = n * 8 + q4 * 2 + (e & 1);
            const float v = (col < valid) ? sacc[n][e] * scale2 : -INFINITY;
            sacc[n][e] = v;
            if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
          }
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float c0 = exp2f(m0 - ms0), c1 = exp2f(m1 - ms1);
        m0 = mn0; m1 = mn1;
        float s0 = 0.f, s1 = 0.f;
        uint32_t pa[GP / 16][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) {
          const float e0 = exp2f(sacc[n][0] - ms0), e1 = exp2f(sacc[n][1] - ms0);
          const float e2 = exp2f(sacc[n][2] - ms1), e3 = exp2f(sacc[n][3] - ms1);
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
    // ---- merge the page slots of each row tile through shared memory (tree), slot 0 keeps it
    float* scr = reinterpret_cast<float*>(qs_gen);
    for (int stride = ns >> 1; stride >= 1; stride >>= 1) {
      const int nw = stride * nrtp;                 // writers this round
      if (slot >= stride && slot < 2 * stride) {
        const int w = (slot - stride) * nrtp + rt;
        float* dst = scr + w * 32 + lane;
        dst[0 * nw * 32] = m0; dst[1 * nw * 32] = m1; dst[2 * nw * 32] = l0; dst[3 * nw * 32] = l1;
#pragma unroll
        for (int n = 0; n < ND; ++n)
#pragma unroll
          for (int e = 0; e < 4; ++e) dst[(4 + n * 4 + e) * nw * 32] = oacc[n][e];
      }
      consumer_bar();
      if (slot < stride) {
        const int w = slot * nrtp + rt;
        const float* src = scr + w * 32 + lane;
        const float pm0 = src[0 * nw * 32], pm1 = src[1 * nw * 32];
        const float pl0 = src[2 * nw * 32], pl1 = src[3 * nw * 32];
        const float mn0 = fmaxf(m0, pm0), mn1 = fmaxf(m1, pm1);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float a0 = exp2f(m0 - ms0), b0 = exp2f(pm0 - ms0);
        const float a1 = exp2f(m1 - ms1), b1 = exp2f(pm1 - ms1);
        m0 = mn0; m1 = mn1;
        l0 = l0 * a0 + pl0 * b0;
        l1 = l1 * a1 + pl1 * b1;
#pragma unroll
        for (int n = 0; n < ND; ++n) {
          oacc[n][0] = oacc[n][0] * a0 + src[(4 + n * 4 + 0) * nw * 32] * b0;
          oacc[n][1] = oacc[n][1] * a0 + src[(4 + n * 4 + 1) * nw * 32] * b0;
          oacc[n][2] = oacc[n][2] * a1 + src[(4 + n * 4 + 2) * nw * 32] * b1;
          oacc[n][3] = oacc[n][3] * a1 + src[(4 + n * 4 + 3) * nw * 32] * b1;
        }
      }
      consumer_bar();
    }
    static_assert((4 + OREGS) * 4 * 32 * 4 <= q_region_bytes<D>(), "merge scratch must fit the Q region");

    // ---- un-normalised partial of this (CTA, segment) piece
    if (slot == 0 && has_rows) {
      l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
      l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
      float* part = partial_base(p.partials, blockIdx.x + sg, D);
      const int r0 = rt * 16 + g8, r1 = r0 + 8;
      if (r0 < rows) {
        if (q4 == 0) { part[r0] = m0; part[kRowsPerGroup + r0] = l0; }
#pragma unroll
        for (int n = 0; n < ND; ++n)
          *reinterpret_cast<float2*>(part + 2 * kRowsPerGroup + r0 * D + n * 8 + q4 * 2) = make_float2(oacc[n][0], oacc[n][1]);
      }
      if (r1 < rows) {
        if (q4 == 0) { part[r1] = m1; part[kRowsPerGroup + r1] = l1; }
#pragma unroll
        for (int n = 0; n < ND; ++n)
          *reinterpret_cast<float2*>(part + 2 * kRowsPerGroup + r1 * D + n * 8 + q4 * 2) = make_float2(oacc[n][2], oacc[n][3]);
      }
    }
    item = seg_end;
    ++sg;
    while (item < hi && pre[sg + 1] <= item) ++sg;
  }
  if (tid == 0) LOSA_STAMP(6);
#ifdef LOSA_TRACE
  if (lane == 0 && p.trace) { p.trace[p.n_ctas * 8 + (blockIdx.x * 8 + warp) * 2] = trace_wait; p.trace[p.n_ctas * 8 + (blockIdx.x * 8 + warp) * 2 + 1] = trace_busy; }
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
  attn_combine_kernel<D, true><<<dim3(ap.n_seg, kRowsPerGroup / 8), 256, 0, st>>>(ap);
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
  attn_combine_kernel<D, false><<<dim3(ap.n_seg, kRowsPerGroup / 8), 256, 0, st>>>(ap);
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
