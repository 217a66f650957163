// Stage 5 — dense in-block attention and the online-softmax merge (Section 4.3, Section 2.2);
// stage 6 — cache maintenance (Section 4.3, Section 2.1) and the page summaries (Section 2.3).
//
// These stages touch O(B * H * d) data: they are latency-bound.  In bf16 mode the in-block attention
// runs on the tensor cores (block_attn_mma_kernel); the fp32 mode and the cache kernels are plain
// CUDA-core code laid out for coalesced global access and conflict-free shared-memory access.
#include "kernels.h"

namespace losa {
namespace {

constexpr int kThreads = 256;
constexpr int kTokTile = 4;        // block tokens per CTA of the in-block attention
constexpr int kBaThreads = 128;
constexpr int kBaRows = 4;         // query rows a warp works on together

// One CTA per (four block tokens, KV head, sequence): K_b, V_b of the KV head and the CTA's query
// rows staged in shared memory as fp32.  A warp takes four query rows at a time (with G = 4 the
// heads of one token), so every K_b / V_b element read from shared memory feeds four multiply-adds:
// the kernel is bound by shared-memory reads, and this is what keeps it short enough to hide beside
// stages 1-3.  Scores: lane = block key (rows of K_b padded by four floats: conflict-free 16-byte
// reads), the four query rows read as broadcasts; P V: lane = output column, probabilities by shuffle.
// MERGE = false (whole-step path): only the in-block part, normalised o_b to `ob_out` and L_b to
// `lse_out`; the prefix statistics are not touched, so this can run beside stages 1-4.
template <typename T, int D, bool MERGE>
__global__ void __launch_bounds__(kBaThreads)
block_attn_merge_kernel(const T* __restrict__ q, const T* __restrict__ k_blk, const T* __restrict__ v_blk,
                        const float* __restrict__ o_p, const float* __restrict__ lse_p,
                        T* __restrict__ out, float* __restrict__ lse_out, float* __restrict__ ob_out,
                        int B, int Hq, int Hkv, float sm_scale) {
  grid_dep_wait();
  constexpr int KS = D + 4;         // padded row of K_b
  constexpr int C = D / 32;
  constexpr int U = 2;              // block keys per lane (B <= 64)
  extern __shared__ __align__(16) float smem[];
  float* Ks = smem;                 // [B][D + 4]
  float* Vs = Ks + B * KS;          // [B][D]
  float* Qs = Vs + B * D;           // [kTokTile * G][D]
  const int t0 = blockIdx.x * kTokTile, kh = blockIdx.y, s = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = Hq / Hkv;
  const int nrow = min(kTokTile, B - t0) * G;
  auto row_of = [&](int r) { return (static_cast<size_t>(s) * B + t0 + r / G) * Hq + kh * G + r % G; };
  for (int idx = tid * 8; idx < nrow * D; idx += kBaThreads * 8) {
    float a[8];
    load8(q + row_of(idx / D) * D + idx % D, a);
    *reinterpret_cast<float4*>(Qs + idx) = make_float4(a[0], a[1], a[2], a[3]);
    *reinterpret_cast<float4*>(Qs + idx + 4) = make_float4(a[4], a[5], a[6], a[7]);
  }
  for (int idx = tid * 8; idx < B * D; idx += kBaThreads * 8) {
    const int t = idx / D, j = idx % D;
    const size_t src = ((static_cast<size_t>(s) * B + t) * Hkv + kh) * D + j;
    float a[8], b[8];
    load8(k_blk + src, a);
    load8(v_blk + src, b);
    *reinterpret_cast<float4*>(Ks + t * KS + j) = make_float4(a[0], a[1], a[2], a[3]);
    *reinterpret_cast<float4*>(Ks + t * KS + j + 4) = make_float4(a[4], a[5], a[6], a[7]);
    *reinterpret_cast<float4*>(Vs + idx) = make_float4(b[0], b[1], b[2], b[3]);
    *reinterpret_cast<float4*>(Vs + idx + 4) = make_float4(b[4], b[5], b[6], b[7]);
  }
  __syncthreads();
  for (int r0 = warp * kBaRows; r0 < nrow; r0 += (kBaThreads / 32) * kBaRows) {
    const int nr = min(kBaRows, nrow - r0);
    // prefix statistics of the rows (MERGE): requested now, used after the arithmetic
    float opv[kBaRows][C], Lp[kBaRows];
#pragma unroll
    for (int r = 0; r < kBaRows; ++r) {
      const size_t row = row_of(r0 + min(r, nr - 1));
#pragma unroll
      for (int c = 0; c < C; ++c) opv[r][c] = MERGE ? o_p[row * D + lane + 32 * c] : 0.f;
      Lp[r] = MERGE ? lse_p[row] : 0.f;
    }
    // ---- scores: lane = block key (two keys per lane when B > 32)
    float sc[U][kBaRows];
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int r = 0; r < kBaRows; ++r) sc[u][r] = 0.f;
    const float* qr = Qs + r0 * D;
#pragma unroll 4
    for (int j = 0; j < D; j += 4) {
      float4 kv[U];
#pragma unroll
      for (int u = 0; u < U; ++u) {
        const int t = lane + 32 * u;
        kv[u] = (t < B) ? *reinterpret_cast<const float4*>(Ks + t * KS + j) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int r = 0; r < kBaRows; ++r) {
        const float4 qv = *reinterpret_cast<const float4*>(qr + min(r, nr - 1) * D + j);
#pragma unroll
        for (int u = 0; u < U; ++u)
          sc[u][r] = fmaf(qv.w, kv[u].w, fmaf(qv.z, kv[u].z, fmaf(qv.y, kv[u].y, fmaf(qv.x, kv[u].x, sc[u][r]))));
      }
    }
    // ---- softmax over the block keys, per row
    float p[U][kBaRows], sum[kBaRows], Lb[kBaRows];
#pragma unroll
    for (int r = 0; r < kBaRows; ++r) {
      float mx = -INFINITY;
#pragma unroll
      for (int u = 0; u < U; ++u) {
        sc[u][r] = (lane + 32 * u < B) ? sc[u][r] * sm_scale : -INFINITY;
        mx = fmaxf(mx, sc[u][r]);
      }
      const float M = warp_max(mx);
      float ps = 0.f;
#pragma unroll
      for (int u = 0; u < U; ++u) { p[u][r] = expf(sc[u][r] - M); ps += p[u][r]; }
      sum[r] = warp_sum(ps);
      Lb[r] = M + logf(sum[r]);
    }
    // ---- P V: lane = output column
    float ob[kBaRows][C];
#pragma unroll
    for (int r = 0; r < kBaRows; ++r)
#pragma unroll
      for (int c = 0; c < C; ++c) ob[r][c] = 0.f;
#pragma unroll 2
    for (int t = 0; t < B; ++t) {
      float v[C];
#pragma unroll
      for (int c = 0; c < C; ++c) v[c] = Vs[t * D + lane + 32 * c];
#pragma unroll
      for (int r = 0; r < kBaRows; ++r) {
        const float pt = __shfl_sync(0xffffffffu, t < 32 ? p[0][r] : p[1][r], t & 31);
#pragma unroll
        for (int c = 0; c < C; ++c) ob[r][c] = fmaf(pt, v[c], ob[r][c]);
      }
    }
#pragma unroll
    for (int r = 0; r < kBaRows; ++r) {
      if (r < nr) {
        const size_t row = row_of(r0 + r);
        if (MERGE) {
          const float M2 = fmaxf(Lp[r], Lb[r]);
          const float L = M2 + logf(expf(Lp[r] - M2) + expf(Lb[r] - M2));
          const float wp = expf(Lp[r] - L), wb = expf(Lb[r] - L) / sum[r];
#pragma unroll
          for (int c = 0; c < C; ++c) {
            const float v = (wp > 0.f ? wp * opv[r][c] : 0.f) + wb * ob[r][c];
            out[row * D + lane + 32 * c] = from_f32<T>(v);
          }
          if (lse_out && lane == 0) lse_out[row] = L;
        } else {
          const float inv = 1.f / sum[r];
#pragma unroll
          for (int c = 0; c < C; ++c) ob_out[row * D + lane + 32 * c] = ob[r][c] * inv;
          if (lane == 0) lse_out[row] = Lb[r];
        }
      }
    }
  }
}

// ---- in-block attention of the whole-step path on the tensor cores (bf16) ---------------------
// The in-block part is a small dense contraction (B keys, all B * G rows of a KV head), and it runs
// beside stages 1-3, where every cycle it holds an SM delays them: mma.sync tiles cut its
// instruction count by more than an order of magnitude against the CUDA-core kernel above.
// CTA = 64 query rows of one (sequence, KV head) (row = block token * G + head of the group), one
// warp per 16 rows.  K_b [key][d] and V_b transposed [d][key] are staged in shared memory as bf16
// (rows padded by 16 bytes: the fragment reads are conflict-free); Q fragments come straight from
// global memory.  S = Q K_b^T in fp32 accumulators, softmax in registers (row statistics over the
// four lanes that share a row), P rounded to bf16 as in stage 4, O = P V_b in fp32, normalised by
// the fp32 sum.  BK = B rounded up to 32 or 64; keys >= B are masked, their V rows zero.
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

constexpr int kMmaRows = 64;       // query rows per CTA
constexpr int kMmaThreads = 128;

// MERGE = true (stage 5 of the six-call path): the in-block part is merged with the prefix
// statistics by log-sum-exp and the attention output is written (Section 2.2 / 4.3); MERGE = false
// (whole-step path): the normalised in-block part goes to `ob_out` and L_b to `lse_out`.
template <int D, int BK, bool MERGE>
__global__ void __launch_bounds__(kMmaThreads)
block_attn_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k_blk,
                      const __nv_bfloat16* __restrict__ v_blk, const void* __restrict__ o_p, int o_p_bf16,
                      const float* __restrict__ lse_p, __nv_bfloat16* __restrict__ out, float* __restrict__ lse_out,
                      float* __restrict__ ob_out, int B, int Hq, int Hkv, float sm_scale) {
  grid_dep_wait();
  constexpr int KS = D + 8;          // padded row of K_b (elements)
  constexpr int VS = BK + 8;         // padded row of V_b^T
  constexpr int NT = BK / 8;         // key tiles of S
  constexpr int NO = D / 8;          // column tiles of O
  __shared__ __align__(16) __nv_bfloat16 Ks[BK * KS];
  __shared__ __align__(16) __nv_bfloat16 Vt[D * VS];
  const int kh = blockIdx.y, s = blockIdx.z;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = Hq / Hkv, nrow = B * G;
  // ---- stage K_b (row-major) and V_b (transposed); keys >= B are zero
  for (int idx = tid; idx < BK * (D / 8); idx += kMmaThreads) {
    const int t = idx % BK, ch = idx / BK;             // key fastest: the transposed stores of a warp fall into one row
    uint4 kv = make_uint4(0u, 0u, 0u, 0u), vv = kv;
    if (t < B) {
      const size_t src = ((static_cast<size_t>(s) * B + t) * Hkv + kh) * D + ch * 8;
      kv = *reinterpret_cast<const uint4*>(k_blk + src);
      vv = *reinterpret_cast<const uint4*>(v_blk + src);
    }
    *reinterpret_cast<uint4*>(Ks + t * KS + ch * 8) = kv;
    const __nv_bfloat16* ve = reinterpret_cast<const __nv_bfloat16*>(&vv);
#pragma unroll
    for (int e = 0; e < 8; ++e) Vt[(ch * 8 + e) * VS + t] = ve[e];
  }
  // ---- this warp's 16 rows: rows g and g + 8 of the tile for this lane
  const int g = lane >> 2, t4 = lane & 3;
  const int lr0 = blockIdx.x * kMmaRows + warp * 16 + g, lr1 = lr0 + 8;
  auto global_row = [&](int lr) {
    const int c = min(lr, nrow - 1);
    return (static_cast<size_t>(s) * B + c / G) * Hq + kh * G + c % G;
  };
  const size_t gr0 = global_row(lr0), gr1 = global_row(lr1);
  const uint32_t* q0 = reinterpret_cast<const uint32_t*>(q + gr0 * D);
  const uint32_t* q1 = reinterpret_cast<const uint32_t*>(q + gr1 * D);
  uint32_t qa[D / 16][4];
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
    qa[ks][0] = q0[ks * 8 + t4];
    qa[ks][1] = q1[ks * 8 + t4];
    qa[ks][2] = q0[ks * 8 + 4 + t4];
    qa[ks][3] = q1[ks * 8 + 4 + t4];
  }
  __syncthreads();
  if (blockIdx.x * kMmaRows + warp * 16 >= nrow) return;       // no row of this warp exists
  // ---- S = Q K_b^T
  float sc[NT][4];
#pragma unroll
  for (int j = 0; j < NT; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) sc[j][e] = 0.f;
#pragma unroll
  for (int ks = 0; ks < D / 16; ++ks) {
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const uint32_t* kr = reinterpret_cast<const uint32_t*>(Ks + (8 * j + g) * KS + 16 * ks);
      mma_bf16_16816(sc[j], qa[ks], kr[t4], kr[4 + t4]);
    }
  }
  // ---- softmax over the keys (natural exponent; the log-normaliser is exported in natural units)
  float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
  for (int j = 0; j < NT; ++j) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int key = 8 * j + 2 * t4 + (e & 1);
      sc[j][e] = key < B ? sc[j][e] * sm_scale : -INFINITY;
    }
    m0 = fmaxf(m0, fmaxf(sc[j][0], sc[j][1]));
    m1 = fmaxf(m1, fmaxf(sc[j][2], sc[j][3]));
  }
  m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
  m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
  m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
  m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
  float l0 = 0.f, l1 = 0.f;
  uint32_t pa[NT][2];                // P as bf16 pairs: [j][0] row g, [j][1] row g + 8
#pragma unroll
  for (int j = 0; j < NT; ++j) {
    const float p0 = expf(sc[j][0] - m0), p1 = expf(sc[j][1] - m0);
    const float p2 = expf(sc[j][2] - m1), p3 = expf(sc[j][3] - m1);
    l0 += p0 + p1;
    l1 += p2 + p3;
    pa[j][0] = pack2_bf16(p0, p1);
    pa[j][1] = pack2_bf16(p2, p3);
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  // ---- O = P V_b
  float o[NO][4];
#pragma unroll
  for (int jn = 0; jn < NO; ++jn)
#pragma unroll
    for (int e = 0; e < 4; ++e) o[jn][e] = 0.f;
#pragma unroll
  for (int kk = 0; kk < BK / 16; ++kk) {
    const uint32_t a[4] = {pa[2 * kk][0], pa[2 * kk][1], pa[2 * kk + 1][0], pa[2 * kk + 1][1]};
#pragma unroll
    for (int jn = 0; jn < NO; ++jn) {
      const uint32_t* vr = reinterpret_cast<const uint32_t*>(Vt + (8 * jn + g) * VS + 16 * kk);
      mma_bf16_16816(o[jn], a, vr[t4], vr[4 + t4]);
    }
  }
  // rows g (accumulator halves 0, 1) and g + 8 (halves 2, 3)
  auto finish_row = [&](int lr, size_t gr, float m, float l, int e0) {
    if (lr >= nrow) return;
    const float Lb = m + logf(l);
    if (MERGE) {
      const float Lp = lse_p[gr];
      const float M2 = fmaxf(Lp, Lb);
      const float L = M2 + logf(expf(Lp - M2) + expf(Lb - M2));
      const float wp = expf(Lp - L), wb = expf(Lb - L) / l;
#pragma unroll
      for (int jn = 0; jn < NO; ++jn) {
        float2 pv;                                   // the cached prefix output as it is stored (fp32 or bf16)
        if (o_p_bf16) pv = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(static_cast<const __nv_bfloat16*>(o_p) + gr * D + 8 * jn + 2 * t4));
        else pv = *reinterpret_cast<const float2*>(static_cast<const float*>(o_p) + gr * D + 8 * jn + 2 * t4);
        const float x = (wp > 0.f ? wp * pv.x : 0.f) + wb * o[jn][e0];
        const float y = (wp > 0.f ? wp * pv.y : 0.f) + wb * o[jn][e0 + 1];
        *reinterpret_cast<__nv_bfloat162*>(out + gr * D + 8 * jn + 2 * t4) = __floats2bfloat162_rn(x, y);
      }
      if (lse_out && t4 == 0) lse_out[gr] = L;
    } else {
      const float inv = 1.f / l;
#pragma unroll
      for (int jn = 0; jn < NO; ++jn)
        *reinterpret_cast<float2*>(ob_out + gr * D + 8 * jn + 2 * t4) = make_float2(o[jn][e0] * inv, o[jn][e0 + 1] * inv);
      if (t4 == 0) lse_out[gr] = Lb;
    }
  };
  finish_row(lr0, gr0, m0, l0, 0);
  finish_row(lr1, gr1, m1, l1, 2);
}

// Whole-step path, last kernel: one warp per (token, head) row merges the prefix statistics with
// the in-block part (Section 2.2 / 4.3), writes the output, and keeps the row's query for the next
// step's Eq. 1; block 0 also bumps the step counters.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
merge_commit_kernel(const T* __restrict__ q, T* __restrict__ q_prev, const float* __restrict__ o_p,
                    const float* __restrict__ lse_p, const float* __restrict__ o_b,
                    const float* __restrict__ lse_b, T* __restrict__ out, float* __restrict__ lse_out,
                    int32_t* __restrict__ step, int N, size_t n_rows) {
  grid_dep_wait();
  const int lane = threadIdx.x & 31;
  const size_t row = static_cast<size_t>(blockIdx.x) * (kThreads / 32) + (threadIdx.x >> 5);
  if (blockIdx.x == 0)
    for (int s = threadIdx.x; s < N; s += kThreads) step[s] += 1;
  if (row >= n_rows) return;
  constexpr int C = D / 32;
  float a[C], b[C];
  T qv[C];
#pragma unroll
  for (int c = 0; c < C; ++c) {
    a[c] = o_p[row * D + lane + 32 * c];
    b[c] = o_b[row * D + lane + 32 * c];
    qv[c] = q[row * D + lane + 32 * c];
  }
  const float Lp = lse_p[row], Lb = lse_b[row];
  const float M = fmaxf(Lp, Lb);
  const float L = M + logf(expf(Lp - M) + expf(Lb - M));
  const float wp = expf(Lp - L), wb = expf(Lb - L);
#pragma unroll
  for (int c = 0; c < C; ++c) {
    out[row * D + lane + 32 * c] = from_f32<T>((wp > 0.f ? wp * a[c] : 0.f) + wb * b[c]);
    q_prev[row * D + lane + 32 * c] = qv[c];
  }
  if (lse_out && lane == 0) lse_out[row] = L;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
commit_step_kernel(const uint4* __restrict__ q, uint4* __restrict__ q_prev, size_t n_vec,
                   int32_t* __restrict__ step, int N) {
  grid_dep_wait();
  for (size_t i = blockIdx.x * static_cast<size_t>(kThreads) + threadIdx.x; i < n_vec;
       i += static_cast<size_t>(gridDim.x) * kThreads)
    q_prev[i] = q[i];
  if (blockIdx.x == 0)
    for (int s = threadIdx.x; s < N; s += kThreads) step[s] += 1;
}

// min / max of column j of logical page p over its valid tokens; tokens at prefix positions >=
// new_from are taken from the block being appended (k_blk) instead of the pool.
template <typename T>
__device__ __forceinline__ void summarise_column(const T* __restrict__ k_pages, const T* __restrict__ k_blk,
                                                 T* __restrict__ kmin, T* __restrict__ kmax,
                                                 size_t page_off, int64_t stride_tok, int valid,
                                                 int page_start, int new_from, size_t blk_off,
                                                 int blk_stride, size_t sum_off, int j) {
  float lo = INFINITY, hi = -INFINITY;
  for (int t = 0; t < valid; ++t) {
    const int pos = page_start + t;
    const float v = (pos >= new_from)
                        ? to_f32(k_blk[blk_off + static_cast<size_t>(pos - new_from) * blk_stride + j])
                        : to_f32(k_pages[page_off + static_cast<size_t>(t) * stride_tok + j]);
    lo = fminf(lo, v);
    hi = fmaxf(hi, v);
  }
  kmin[sum_off + j] = from_f32<T>(lo);
  kmax[sum_off + j] = from_f32<T>(hi);
}

template <typename T>
__global__ void build_summaries_kernel(const T* __restrict__ k_pages, T* __restrict__ kmin,
                                       T* __restrict__ kmax, const int32_t* __restrict__ page_table,
                                       const int32_t* __restrict__ kv_len, int64_t stride_page,
                                       int64_t stride_head, int64_t stride_tok, int Hkv, int D, int g,
                                       int Pmax, int n_phys, int32_t* __restrict__ status) {
  grid_dep_wait();
  const int p = blockIdx.x, kh = blockIdx.y, s = blockIdx.z, j = threadIdx.x;
  const int len = kv_len[s];
  const int valid = min(g, len - p * g);
  if (valid <= 0) return;
  const int phys = page_table[static_cast<size_t>(s) * Pmax + p];
  if (phys < 0 || phys >= n_phys) { set_status(status, LOSA_ERR_BOUNDS); return; }
  summarise_column<T>(k_pages, nullptr, kmin, kmax,
                      static_cast<size_t>(phys) * stride_page + static_cast<size_t>(kh) * stride_head,
                      stride_tok, valid, p * g, INT_MAX, 0, 0,
                      (static_cast<size_t>(phys) * Hkv + kh) * D, j);
}

// Block finalisation: one CTA per (touched page, KV head, sequence) writes the block tokens that
// fall into the page and recomputes the page's summaries; kv_len / step are bumped by a second
// kernel so that every CTA here sees the old length.
template <typename T>
__global__ void append_block_kernel(T* __restrict__ k_pages, T* __restrict__ v_pages, T* __restrict__ kmin,
                                    T* __restrict__ kmax, const T* __restrict__ k_blk,
                                    const T* __restrict__ v_blk, const int32_t* __restrict__ page_table,
                                    const int32_t* __restrict__ kv_len, int64_t stride_page,
                                    int64_t stride_head, int64_t stride_tok, int B, int Hkv, int D,
                                    int g, int Pmax, int n_phys, int32_t* __restrict__ status) {
  grid_dep_wait();
  const int kh = blockIdx.y, s = blockIdx.z, j = threadIdx.x;
  const int L0 = kv_len[s];
  const int p = L0 / g + blockIdx.x;
  if (p > (L0 + B - 1) / g) return;
  if (p >= Pmax) { set_status(status, LOSA_ERR_BOUNDS); return; }
  const int phys = page_table[static_cast<size_t>(s) * Pmax + p];
  if (phys < 0 || phys >= n_phys) { set_status(status, LOSA_ERR_BOUNDS); return; }
  const size_t page_off = static_cast<size_t>(phys) * stride_page + static_cast<size_t>(kh) * stride_head;
  const size_t blk_off = (static_cast<size_t>(s) * B * Hkv + kh) * D;
  const int blk_stride = Hkv * D;
  const int first = max(L0, p * g), last = min(L0 + B, p * g + g);   // prefix positions written here
  for (int pos = first; pos < last; ++pos) {
    const size_t dst = page_off + static_cast<size_t>(pos - p * g) * stride_tok + j;
    const size_t src = blk_off + static_cast<size_t>(pos - L0) * blk_stride + j;
    k_pages[dst] = k_blk[src];
    v_pages[dst] = v_blk[src];
  }
  summarise_column<T>(k_pages, k_blk, kmin, kmax, page_off, stride_tok, last - p * g, p * g, L0,
                      blk_off, blk_stride, (static_cast<size_t>(phys) * Hkv + kh) * D, j);
}

// A sequence whose block did not fit its page-table row (the append kernel reported it and wrote
// nothing beyond the row) keeps its length: later steps must not index pages past P_max.
__global__ void finalize_counters_kernel(int32_t* __restrict__ kv_len, int32_t* __restrict__ step, int N, int B,
                                         int g, int Pmax) {
  grid_dep_wait();
  const int s = threadIdx.x;
  if (s < N) {
    const long long cap = static_cast<long long>(Pmax) * g;
    if (static_cast<long long>(kv_len[s]) + B <= cap) kv_len[s] += B;
    step[s] = 0;
  }
}

template <typename T, int D, bool MERGE>
int32_t launch_merge_t(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk,
                       const losa_state_t* state, void* out, float* lse_out, float* ob_out, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  const int G = sh.n_q_heads / sh.n_kv_heads;
  const size_t smem = (static_cast<size_t>(sh.block_size) * (2 * D + 4) + static_cast<size_t>(kTokTile) * G * D) * sizeof(float);
  if (smem > 48 * 1024)
    LOSA_CUDA_TRY(c, cudaFuncSetAttribute(block_attn_merge_kernel<T, D, MERGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  dim3 grid((sh.block_size + kTokTile - 1) / kTokTile, sh.n_kv_heads, sh.batch);
  launch_k(block_attn_merge_kernel<T, D, MERGE>, grid, kBaThreads, smem, st, 
      static_cast<const T*>(q), static_cast<const T*>(k_blk), static_cast<const T*>(v_blk),
      state ? static_cast<const float*>(state->o_p) : nullptr, state ? state->lse_p : nullptr, static_cast<T*>(out), lse_out, ob_out,
      sh.block_size, sh.n_q_heads, sh.n_kv_heads, sh.sm_scale);
  return after_launch(c);
}

template <typename T, int D>
int32_t launch_merge_commit_t(losa_ctx* c, const void* q, losa_state_t* state, void* out, float* lse_out,
                              cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  const size_t n_rows = static_cast<size_t>(sh.batch) * sh.block_size * sh.n_q_heads;
  const int blocks = static_cast<int>((n_rows + kThreads / 32 - 1) / (kThreads / 32));
  launch_k(merge_commit_kernel<T, D>, blocks, kThreads, 0, st, 
      static_cast<const T*>(q), static_cast<T*>(state->q_prev), static_cast<const float*>(state->o_p), state->lse_p,
      reinterpret_cast<const float*>(c->ws + c->lay.block_o), reinterpret_cast<const float*>(c->ws + c->lay.block_lse),
      static_cast<T*>(out), lse_out, state->step, sh.batch, n_rows);
  return after_launch(c);
}

template <typename T>
int32_t launch_update_t(losa_ctx* c, losa_kv_t* kv, losa_state_t* state, const void* q,
                        const void* k_blk, const void* v_blk, int32_t finalize_block, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  if (!finalize_block) {
    const size_t n_vec = static_cast<size_t>(sh.batch) * sh.block_size * sh.n_q_heads * sh.head_dim * sizeof(T) / 16;
    const int blocks = static_cast<int>(std::min<size_t>((n_vec + kThreads - 1) / kThreads, static_cast<size_t>(c->n_sms) * 4));
    launch_k(commit_step_kernel<T>, std::max(blocks, 1), kThreads, 0, st, 
        static_cast<const uint4*>(q), static_cast<uint4*>(state->q_prev), n_vec, state->step, sh.batch);
    return after_launch(c);
  }
  if (kv->kv_format == LOSA_KV_FP8_E4M3) {
    // FP8 pages: the touched pages are re-quantised from their dequantised old rows and the new rows
    int32_t rc = launch_fp8_append(c, kv, k_blk, v_blk, st);
    if (rc != LOSA_OK) return rc;
    launch_k(finalize_counters_kernel, 1, std::max(32, sh.batch), 0, st, kv->kv_len, state->step, sh.batch, sh.block_size,
             sh.page_size, sh.max_pages_per_seq);
    return after_launch(c);
  }
  dim3 grid((sh.block_size + sh.page_size - 1) / sh.page_size + 1, sh.n_kv_heads, sh.batch);
  launch_k(append_block_kernel<T>, grid, sh.head_dim, 0, st, 
      static_cast<T*>(kv->k_pages), static_cast<T*>(kv->v_pages), static_cast<T*>(kv->kmin),
      static_cast<T*>(kv->kmax), static_cast<const T*>(k_blk), static_cast<const T*>(v_blk),
      kv->page_table, kv->kv_len, kv->stride_page, kv->stride_head, kv->stride_tok, sh.block_size,
      sh.n_kv_heads, sh.head_dim, sh.page_size, sh.max_pages_per_seq, kv->n_phys_pages, status_ptr(c));
  int32_t rc = after_launch(c);
  if (rc != LOSA_OK) return rc;
  launch_k(finalize_counters_kernel, 1, std::max(32, sh.batch), 0, st, kv->kv_len, state->step, sh.batch, sh.block_size,
           sh.page_size, sh.max_pages_per_seq);
  return after_launch(c);
}

template <typename T>
int32_t launch_summaries_t(losa_ctx* c, losa_kv_t* kv, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  if (sh.max_pages_per_seq == 0) return LOSA_OK;
  dim3 grid(sh.max_pages_per_seq, sh.n_kv_heads, sh.batch);
  launch_k(build_summaries_kernel<T>, grid, sh.head_dim, 0, st, 
      static_cast<const T*>(kv->k_pages), static_cast<T*>(kv->kmin), static_cast<T*>(kv->kmax),
      kv->page_table, kv->kv_len, kv->stride_page, kv->stride_head, kv->stride_tok, sh.n_kv_heads,
      sh.head_dim, sh.page_size, sh.max_pages_per_seq, kv->n_phys_pages, status_ptr(c));
  return after_launch(c);
}

}  // namespace

template <int D, int BK, bool MERGE>
int32_t launch_block_attn_mma(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk,
                              const losa_state_t* state, void* out, float* lb, float* ob, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  const int rows = sh.block_size * (sh.n_q_heads / sh.n_kv_heads);
  dim3 grid((rows + kMmaRows - 1) / kMmaRows, sh.n_kv_heads, sh.batch);
  launch_k(block_attn_mma_kernel<D, BK, MERGE>, grid, kMmaThreads, 0, st,
      static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k_blk),
      static_cast<const __nv_bfloat16*>(v_blk), state ? state->o_p : nullptr,
      (state && state->o_p_format == LOSA_STATE_BF16) ? 1 : 0, state ? state->lse_p : nullptr,
      static_cast<__nv_bfloat16*>(out), lb, ob, sh.block_size, sh.n_q_heads, sh.n_kv_heads, sh.sm_scale);
  return after_launch(c);
}

// bf16: the tensor-core kernel, by head dimension and padded key count
template <bool MERGE>
int32_t dispatch_block_attn_mma(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk,
                                const losa_state_t* state, void* out, float* lb, float* ob, cudaStream_t st) {
  const bool wide = c->shape.block_size > 32;
  if (c->shape.head_dim == 128)
    return wide ? launch_block_attn_mma<128, 64, MERGE>(c, q, k_blk, v_blk, state, out, lb, ob, st)
                : launch_block_attn_mma<128, 32, MERGE>(c, q, k_blk, v_blk, state, out, lb, ob, st);
  return wide ? launch_block_attn_mma<64, 64, MERGE>(c, q, k_blk, v_blk, state, out, lb, ob, st)
              : launch_block_attn_mma<64, 32, MERGE>(c, q, k_blk, v_blk, state, out, lb, ob, st);
}

int32_t launch_block_attn_merge(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk,
                                const losa_state_t* state, void* out, float* lse_out_opt, cudaStream_t st) {
  const bool bf = c->shape.dtype == LOSA_BF16;
  if (bf) return dispatch_block_attn_mma<true>(c, q, k_blk, v_blk, state, out, lse_out_opt, nullptr, st);
  if (c->shape.head_dim == 128) return launch_merge_t<float, 128, true>(c, q, k_blk, v_blk, state, out, lse_out_opt, nullptr, st);
  return launch_merge_t<float, 64, true>(c, q, k_blk, v_blk, state, out, lse_out_opt, nullptr, st);
}

int32_t launch_block_attn(losa_ctx* c, const void* q, const void* k_blk, const void* v_blk, cudaStream_t st) {
  const bool bf = c->shape.dtype == LOSA_BF16;
  float* ob = reinterpret_cast<float*>(c->ws + c->lay.block_o);
  float* lb = reinterpret_cast<float*>(c->ws + c->lay.block_lse);
  if (bf) return dispatch_block_attn_mma<false>(c, q, k_blk, v_blk, nullptr, nullptr, lb, ob, st);
  if (c->shape.head_dim == 128) return launch_merge_t<float, 128, false>(c, q, k_blk, v_blk, nullptr, nullptr, lb, ob, st);
  return launch_merge_t<float, 64, false>(c, q, k_blk, v_blk, nullptr, nullptr, lb, ob, st);
}

int32_t launch_merge_commit(losa_ctx* c, const void* q, losa_state_t* state, void* out, float* lse_out_opt,
                            cudaStream_t st) {
  const bool bf = c->shape.dtype == LOSA_BF16;
  if (bf && c->shape.head_dim == 128) return launch_merge_commit_t<__nv_bfloat16, 128>(c, q, state, out, lse_out_opt, st);
  if (bf) return launch_merge_commit_t<__nv_bfloat16, 64>(c, q, state, out, lse_out_opt, st);
  if (c->shape.head_dim == 128) return launch_merge_commit_t<float, 128>(c, q, state, out, lse_out_opt, st);
  return launch_merge_commit_t<float, 64>(c, q, state, out, lse_out_opt, st);
}

int32_t launch_update_prefix_cache(losa_ctx* c, losa_kv_t* kv, losa_state_t* state, const void* q,
                                   const void* k_blk, const void* v_blk, int32_t finalize_block, cudaStream_t st) {
  return c->shape.dtype == LOSA_BF16
             ? launch_update_t<__nv_bfloat16>(c, kv, state, q, k_blk, v_blk, finalize_block, st)
             : launch_update_t<float>(c, kv, state, q, k_blk, v_blk, finalize_block, st);
}

int32_t launch_build_page_summaries(losa_ctx* c, losa_kv_t* kv, cudaStream_t st) {
  if (kv->kv_format == LOSA_KV_FP8_E4M3) return launch_fp8_summaries(c, kv, st);
  return c->shape.dtype == LOSA_BF16 ? launch_summaries_t<__nv_bfloat16>(c, kv, st)
                                     : launch_summaries_t<float>(c, kv, st);
}

}  // namespace losa
