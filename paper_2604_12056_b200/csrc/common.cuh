// Shared device/host helpers of the LoSA CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/losa.h"

namespace losa {

// ----------------------------------------------------------------------------- constants
constexpr int kRowsPerGroup = 128;  // query rows (active token x head of a KV head) one CTA keeps
constexpr int kMaxSegments = 1024;  // (sequence, KV head, row group) triples per call
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ----------------------------------------------------------------------------- context
// Workspace layout (byte offsets from the caller's buffer, each 256-byte aligned).
struct WorkspaceLayout {
  size_t status;     // int32[4]  : device status word (+ padding)
  size_t counters;   // uint32[N] : arrival counters of select_active (self-resetting)
  size_t seg_prefix; // int32[kMaxSegments + 1] : item prefix of the segments, left by the stage-4 main kernel for its combine kernel
  size_t slot_map;   // int32[N*B] : slot of every block token in the active list of the whole-step path, -1 = stable
  size_t union_bits;    // uint32[N*H_kv*ceil(P_max/32)] : page bitmaps of the selection that also writes the union (all zero between launches)
  size_t union_tickets; // uint32[N*H_kv] : its arrival counters (self-resetting)
  size_t delta;      // double[N*B]
  size_t scores;     // float[2*N*B*H_q*score_stride]: page scores, or (lower, upper) bound pairs of them
  size_t partials;   // float[n_slots * kRowsPerGroup * (d + 2)]
  size_t block_o;    // float[N*B*H_q*d]  : in-block attention output of the whole-step path
  size_t block_lse;  // float[N*B*H_q]    : its log-normaliser
  size_t total;
  int32_t score_stride;  // P_max rounded up to 64
  int32_t n_slots;       // n_ctas + n_segments
  int32_t n_ctas;        // CTAs of the split-KV attention kernels (one per SM)
  int32_t n_row_groups;  // ceil(B*G / kRowsPerGroup)
  int32_t n_segments;    // N * H_kv * n_row_groups
};

}  // namespace losa

struct losa_ctx {
  losa_shape_t shape;
  losa::WorkspaceLayout lay;
  char* ws;
  int device;
  int n_sms;
  int max_smem_optin;
  int32_t last_cuda_error;
  int64_t launches;
  // cached TMA descriptors of the K / V pools (opaque 128-byte blobs, see sparse_prefix_attn.cu)
  alignas(64) unsigned char tmap_k[128];
  alignas(64) unsigned char tmap_v[128];
  const void* tmap_key_k;
  const void* tmap_key_v;
  int64_t tmap_strides[3];
  int32_t tmap_n_phys;
  int32_t tmap_format;
  void* encode_fn;  // cuTensorMapEncodeTiled, resolved through the runtime
  // second stream and fork/join events of the whole-step path (created on first use)
  cudaStream_t side_stream;
  cudaEvent_t ev_fork, ev_join;
  // selector of the whole-step path: 0 = one list per query head, 1 = pooled over the heads of a KV head,
  // 2 = tensor-core scores under the relaxed list rule (the codes of launch_page_scores_topk)
  int32_t pooled_selection;
  // bound of the mbarrier waits of the bf16 stage-4 kernel in SM clock cycles (0 = the default, about a second)
  int64_t wait_cycles;
  // the stage-4 kernel of this context has had its shared-memory attribute set
  int32_t attn_attr_set;
  int32_t scores_attr_set;   // likewise for the page-score kernel
  int32_t bounds_attr_set;   // and for the tensor-core page-bound kernel
  int32_t approx_attr_set;
  int32_t refine_attr_set;
  // optional timing of the stage-4 main kernel
  int32_t profile;
  cudaEvent_t ev_begin, ev_end;
};

namespace losa {

inline int32_t* status_ptr(const losa_ctx* c) { return reinterpret_cast<int32_t*>(c->ws + c->lay.status); }

// Records a CUDA error in the context and maps it to LOSA_ERR_CUDA.
inline int32_t cuda_fail(losa_ctx* c, cudaError_t e) {
  c->last_cuda_error = static_cast<int32_t>(e);
  return LOSA_ERR_CUDA;
}
#define LOSA_CUDA_TRY(ctx, expr)                             \
  do {                                                       \
    cudaError_t e__ = (expr);                                \
    if (e__ != cudaSuccess) return ::losa::cuda_fail(ctx, e__); \
  } while (0)

inline int32_t after_launch(losa_ctx* c, int n = 1) {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(c, e);
  c->launches += n;
  return LOSA_OK;
}

// ----------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__

// Every kernel of the library is launched with programmatic stream serialisation: its CTAs may be
// scheduled while the previous kernel of the stream is still draining, and it calls grid_dep_wait()
// before its first access to global memory, which returns once that kernel has completed and its
// writes are visible.  Launch latency and the tail of one kernel overlap the start of the next.
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);   // the error, if any, is read by after_launch()
}
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream be scheduled now instead of when this grid has drained: its
// CTAs take free resources, run their prologue and stop at their own grid_dep_wait() until this
// grid has completed and its writes are visible.  Only for kernels whose whole grid is resident at
// once and whose successor has a prologue worth hiding.
__device__ __forceinline__ void grid_dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void set_status(int32_t* status, int32_t code) { atomicCAS(status, 0, code); }

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// 8 consecutive elements starting at a 16-byte (bf16) / 32-byte (fp32) aligned address -> fp32.
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ int pages_of(int len, int g) { return (len + g - 1) / g; }

// ---- shared-memory barriers (mbarrier) -------------------------------------------------------
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

constexpr long long kWaitCycles = 2000000000ll;   // ~1 s: default bound of every mbarrier wait
constexpr long long kDrainCycles = 20000000ll;    // ~10 ms: bound of the waits for work already in flight when a CTA gives up
// Bounded wait.  Returns false (and raises the CTA's abort flag) when the bound runs out or
// another warp has already given up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int32_t* status, long long limit) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > limit) {
      *abort_flag = 1;
      set_status(status, LOSA_ERR_TIMEOUT);
      return false;
    }
  }
}
// Wait of a CTA that has given up, for work it had already put in flight (page copies into its
// shared memory, tensor-core instructions on its tensor memory): bounded by kDrainCycles, ignores
// the abort flag, reports nothing (the status word already holds the reason).
__device__ __forceinline__ void mbar_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity) && clock64() - t0 < kDrainCycles) {}
}

// ---- balanced split of the flattened (segment, union position) list over the CTAs ------------
// Segment seg = rg * (N * H_kv) + (s * H_kv + kh) holds union_count[s, kh] items when its row
// group has rows, else none.  Row-group-major: with more than 128 query rows per KV head (two row
// groups) the two passes over a (sequence, KV head)'s pages lie half the list apart, so the CTAs b
// and b + n/2 stream the same pages at the same time and the second read is served by the L2.  CTA b owns items [b*T/n, (b+1)*T/n).  The partial result a CTA
// produces for a segment goes to slot b + seg, which is unique (b and seg never both stay put
// between consecutive pieces).
__device__ __forceinline__ int rows_in_group(int n_active, int G, int rg) {
  const int r = n_active * G - rg * kRowsPerGroup;
  return r < 0 ? 0 : (r > kRowsPerGroup ? kRowsPerGroup : r);
}
__device__ __forceinline__ long long cta_lo(long long T, int b, int n) { return (T * b) / n; }

// The tensor-core kernel cuts a list in which every non-empty segment is charged segment_pad(rows)
// items on top of its pages (placed before them): entering a segment costs a CTA about as much as
// that many pages (drain of the pipeline, the record, the new Q tile, refill), so equal shares of
// the charged list finish together.  A CTA's share maps back to the pages it contains; the
// combine step finds the CTAs of a segment with the same arithmetic on the charged positions.
constexpr int kSegPadBase = 10, kSegPadRowsPer = 8;
__device__ __forceinline__ int segment_pad(int rows) { return rows > 0 ? kSegPadBase + rows / kSegPadRowsPer : 0; }

// Exclusive prefix of segment item counts into pre[0..n_seg] (shared memory), by one warp; with
// vpre, also the prefix of the charged counts (pages + pad of every non-empty segment).
__device__ __forceinline__ void segment_prefix(int* pre, int n_seg, int n_rg, int H_kv, int G,
                                               const int32_t* n_active, const int32_t* union_count,
                                               int B, int lane, int* vpre = nullptr) {
  int run = 0, vrun = 0;
  for (int base = 0; base < n_seg; base += 32) {
    const int seg = base + lane;
    int c = 0, vc = 0;
    if (seg < n_seg) {
      const int n_sk = n_seg / n_rg, rg = seg / n_sk, sk = seg % n_sk, s = sk / H_kv;
      int na = n_active[s];
      na = na < 0 ? 0 : (na > B ? B : na);
      const int rows = rows_in_group(na, G, rg);
      c = rows > 0 ? max(union_count[sk], 0) : 0;
      vc = c > 0 ? c + segment_pad(rows) : 0;
    }
    int inc = c, vinc = vc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, inc, o);
      const int vt = __shfl_up_sync(0xffffffffu, vinc, o);
      if (lane >= o) { inc += t; vinc += vt; }
    }
    if (seg < n_seg) {
      pre[seg] = run + inc - c;
      if (vpre) vpre[seg] = vrun + vinc - vc;
    }
    run += __shfl_sync(0xffffffffu, inc, 31);
    vrun += __shfl_sync(0xffffffffu, vinc, 31);
  }
  if (lane == 0) {
    pre[n_seg] = run;
    if (vpre) vpre[n_seg] = vrun;
  }
}

#endif  // __CUDACC__

}  // namespace losa
