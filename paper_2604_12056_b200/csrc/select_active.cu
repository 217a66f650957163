// Stage 1 — locality score (Eq. 1, Section 3.2) and locality pruning (Section 4.1).
//
// One CTA per (token, sequence) streams the token's row of x_cur and x_prev with 16-byte loads and
// reduces sum (x_cur - x_prev)^2 in fp64 (the selection is an integer decision, so it is taken in
// fp64 like the definition; the work is a few hundred KB).  The last CTA of a sequence to arrive
// (self-resetting counter) ranks the B scores by (Delta descending, token ascending) and emits the
// first m tokens in ascending order.
#include <mutex>

#include "kernels.h"

namespace losa {
namespace {

constexpr int kThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kThreads)
select_active_kernel(const T* __restrict__ x_cur, const T* __restrict__ x_prev, int row_width, int B,
                     const int32_t* __restrict__ m_per_seq, const int32_t* __restrict__ step,
                     int32_t* __restrict__ active_idx, int32_t* __restrict__ n_active,
                     float* __restrict__ delta_opt, double* __restrict__ delta_ws,
                     unsigned int* __restrict__ counters, double tau, int32_t* __restrict__ slot_map) {
  // Wait first, release afterwards: a kernel released by this one may read, before its own wait, what
  // earlier kernels of the stream wrote (the cache's lengths, summaries and step counters), so those
  // must have completed by then.
  grid_dep_wait();
  grid_dep_trigger();
  const int i = blockIdx.x, s = blockIdx.y;
  // what the sequence's last CTA needs at the very end: asked for now, so that it is not one more round trip there
  const int m_given = m_per_seq ? m_per_seq[s] : -1;
  const int step_now = step ? step[s] : 1;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const size_t row = (static_cast<size_t>(s) * B + i) * row_width;
  constexpr int kVec = 8;
  double acc = 0.0;
  // two chunks per pass, all four loads requested before any is used (a row of 4,096 elements is
  // one pass of the CTA)
  for (int c = tid * kVec; c < row_width; c += 2 * kThreads * kVec) {
    const int c2 = c + kThreads * kVec;
    float a[8], b[8], a2[8], b2[8];
    load8(x_cur + row + c, a);
    load8(x_prev + row + c, b);
    if (c2 < row_width) {
      load8(x_cur + row + c2, a2);
      load8(x_prev + row + c2, b2);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) a2[j] = b2[j] = 0.f;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const double df = static_cast<double>(a[j]) - static_cast<double>(b[j]);
      acc = fma(df, df, acc);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const double df = static_cast<double>(a2[j]) - static_cast<double>(b2[j]);
      acc = fma(df, df, acc);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ double s_part[kThreads / 32];
  __shared__ double s_delta[LOSA_MAX_BLOCK];
  __shared__ bool s_last;
  if (lane == 0) s_part[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) t += s_part[w];
    t /= static_cast<double>(row_width);
    delta_ws[s * B + i] = t;
    if (delta_opt) delta_opt[s * B + i] = static_cast<float>(t);
    __threadfence();
    const unsigned int ticket = atomicInc(&counters[s], static_cast<unsigned int>(B - 1));
    s_last = (ticket == static_cast<unsigned int>(B - 1));
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid < B) {
    const double dv = *(reinterpret_cast<volatile double*>(delta_ws) + s * B + tid);
    s_delta[tid] = dv != dv ? static_cast<double>(INFINITY) : dv;    // NaN ranks as +inf: the order below stays total
  }
  __syncthreads();
  if (warp != 0) return;

  int m = m_given;
  const bool first_step = step_now == 0;
  if (m < 0 || m > B || first_step) m = B;
  // token t = lane (+32): rank under (Delta descending, token ascending)
  int rank[2] = {B, B};
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int t = lane + 32 * half;
    if (t < B) {
      const double dt = s_delta[t];
      int r = 0;
      for (int j = 0; j < B; ++j) {
        const double dj = s_delta[j];
        r += (dj > dt || (dj == dt && j < t)) ? 1 : 0;
      }
      rank[half] = r;
    }
  }
  if (tau > 0.0 && !first_step) {
    // threshold variant: the shortest leading part of the ranking whose Delta add up to at least
    // tau times the block's total; both sums run over the ranking in order, in fp64, by one lane
    __shared__ double s_sorted[LOSA_MAX_BLOCK];
#pragma unroll
    for (int half = 0; half < 2; ++half)
      if (lane + 32 * half < B) s_sorted[rank[half]] = s_delta[lane + 32 * half];
    __syncwarp();
    int mt = 0;
    if (lane == 0) {
      double total = 0.0;
      for (int r = 0; r < B; ++r) total += s_sorted[r];
      const double thr = tau * total;
      double cum = 0.0;
      while (mt < B && cum < thr) cum += s_sorted[mt++];
    }
    mt = __shfl_sync(0xffffffffu, mt, 0);
    m = min(m, mt);                                   // m_per_seq, when given, is an upper bound here
  }
  bool act[2];
#pragma unroll
  for (int half = 0; half < 2; ++half) act[half] = rank[half] < m;
  const unsigned b0 = __ballot_sync(0xffffffffu, act[0]);
  const unsigned b1 = __ballot_sync(0xffffffffu, act[1]);
  const unsigned below = (1u << lane) - 1u;
  const int n0 = __popc(b0), n1 = __popc(b1);
  int32_t* out = active_idx + static_cast<size_t>(s) * B;
  if (act[0]) out[__popc(b0 & below)] = lane;
  if (act[1]) out[n0 + __popc(b1 & below)] = lane + 32;
  if (slot_map) {                                     // the inverse map, for the kernel that finishes the step
    if (lane < B) slot_map[s * B + lane] = act[0] ? __popc(b0 & below) : -1;
    if (lane + 32 < B) slot_map[s * B + lane + 32] = act[1] ? n0 + __popc(b1 & below) : -1;
  }
  for (int t = n0 + n1 + lane; t < B; t += 32) out[t] = -1;
  if (lane == 0) n_active[s] = n0 + n1;
}

}  // namespace

int32_t launch_select_active(losa_ctx* c, const void* x_cur, const void* x_prev, int32_t row_width,
                             const int32_t* m_per_seq, const int32_t* step, int32_t* active_idx,
                             int32_t* n_active, float* delta_opt, cudaStream_t st, double tau, int32_t* slot_map_opt) {
  const losa_shape_t& sh = c->shape;
  dim3 grid(sh.block_size, sh.batch);
  double* dws = reinterpret_cast<double*>(c->ws + c->lay.delta);
  unsigned int* ctr = reinterpret_cast<unsigned int*>(c->ws + c->lay.counters);
  if (sh.dtype == LOSA_BF16) {
    launch_k(select_active_kernel<__nv_bfloat16>, grid, kThreads, 0, st, 
        static_cast<const __nv_bfloat16*>(x_cur), static_cast<const __nv_bfloat16*>(x_prev), row_width,
        sh.block_size, m_per_seq, step, active_idx, n_active, delta_opt, dws, ctr, tau, slot_map_opt);
  } else {
    launch_k(select_active_kernel<float>, grid, kThreads, 0, st, 
        static_cast<const float*>(x_cur), static_cast<const float*>(x_prev), row_width, sh.block_size,
        m_per_seq, step, active_idx, n_active, delta_opt, dws, ctr, tau, slot_map_opt);
  }
  return after_launch(c);
}

}  // namespace losa

// ----------------------------------------------------------------------------------------------
// Stage 1 for callers that cannot allocate device memory.
//
// The regular entry point keeps its scratch (the fp64 per-token scores and one arrival counter per
// sequence) in the workspace the caller allocated for the context.  This variant keeps the same
// scratch in a fixed array that is part of the library image, so nothing has to be allocated —
// neither by the caller nor here.  Every GPU that loads the library holds the array (about 33 KB)
// until the process exits.
namespace {

constexpr int kStaticMaxBatch = 64;   // sequences the fixed scratch is sized for
constexpr int kStaticMaxDevices = 64;

struct StaticScratch {
  double delta[kStaticMaxBatch * LOSA_MAX_BLOCK];
  unsigned int counters[kStaticMaxBatch];
};

// Device-side storage.  In host code this name is only a handle for the runtime; the device
// address is obtained once per device with cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

std::mutex g_static_mutex;
StaticScratch* g_static_addr[kStaticMaxDevices] = {};

}  // namespace

extern "C" int32_t losa_select_active_static(const losa_shape_t* shape, const void* x_cur, const void* x_prev,
                                             int32_t row_width, const int32_t* m_per_seq, const int32_t* step,
                                             int32_t* active_idx, int32_t* n_active, float* delta_opt,
                                             void* stream) {
  if (!shape || !x_cur || !x_prev || !active_idx || !n_active || row_width < 1) return LOSA_ERR_INVALID_ARG;
  if (shape->batch < 1 || shape->block_size < 1 || shape->block_size > LOSA_MAX_BLOCK ||
      (shape->dtype != LOSA_F32 && shape->dtype != LOSA_BF16))
    return LOSA_ERR_INVALID_ARG;
  if (shape->batch > kStaticMaxBatch) return LOSA_ERR_UNSUPPORTED;   // beyond the fixed scratch
  if (row_width % 8 != 0 || (reinterpret_cast<uintptr_t>(x_cur) & 15u) || (reinterpret_cast<uintptr_t>(x_prev) & 15u))
    return LOSA_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LOSA_ERR_CUDA;
  if (dev < 0 || dev >= kStaticMaxDevices) return LOSA_ERR_UNSUPPORTED;
  StaticScratch* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
      // set-up, once per device, with that device current
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return LOSA_ERR_CUDA;
      g_static_addr[dev] = static_cast<StaticScratch*>(ptr);
    }
    scratch = g_static_addr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the last call left: the arrival counters must start at zero
  if (cudaMemsetAsync(scratch->counters, 0, sizeof(unsigned int) * shape->batch, st) != cudaSuccess) return LOSA_ERR_CUDA;
  dim3 grid(shape->block_size, shape->batch);
  if (shape->dtype == LOSA_BF16) {
    losa::launch_k(losa::select_active_kernel<__nv_bfloat16>, grid, losa::kThreads, 0, st, 
        static_cast<const __nv_bfloat16*>(x_cur), static_cast<const __nv_bfloat16*>(x_prev), row_width,
        shape->block_size, m_per_seq, step, active_idx, n_active, delta_opt, scratch->delta, scratch->counters, 0.0, nullptr);
  } else {
    losa::launch_k(losa::select_active_kernel<float>, grid, losa::kThreads, 0, st, 
        static_cast<const float*>(x_cur), static_cast<const float*>(x_prev), row_width, shape->block_size,
        m_per_seq, step, active_idx, n_active, delta_opt, scratch->delta, scratch->counters, 0.0, nullptr);
  }
  return cudaGetLastError() == cudaSuccess ? LOSA_OK : LOSA_ERR_CUDA;
}
