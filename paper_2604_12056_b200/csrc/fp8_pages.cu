// FP8 (E4M3) K/V pages with one power-of-two scale per (physical page, KV head) and tensor: an
// extension of the cache format (the paper names quantised attention as orthogonal to the method,
// Section 6, and quotes the cached state in FP16, Section 4.5).  Halves the bytes stage 4 streams.
//
//   amax  = largest |x| over the page's valid tokens and d dimensions
//   scale = 2^e, e = the smallest integer with amax <= 448 * 2^e, clamped to [-6, 7]
//   code  = round-to-nearest-even of x / scale onto the E4M3 grid, saturated at +-448
//   dequantised value = scale * value(code): four significant bits, exact in bf16 and in fp16
// Slots of a page past the prefix's end get code 0.  Appending a block re-quantises every touched
// page from its dequantised old values and the new rows together (the scale may have to grow).
// The page summaries (Section 2.3) are the element-wise min / max of the DEQUANTISED keys, so that
// stage 2 bounds the keys stage 4 actually uses.
//
// One CTA per (logical page, KV head, sequence), one thread per head dimension: a thread scans its
// column over the page's tokens (coalesced across the CTA), the CTA reduces the maximum, then every
// thread encodes its own column.
#include <cuda_fp8.h>

#include "kernels.h"

namespace losa {
namespace {

__device__ __forceinline__ float fp8_value(uint8_t code) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw(static_cast<__nv_fp8_storage_t>(code), __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half*>(&h));
}
__device__ __forceinline__ uint8_t fp8_code(float y) {          // round to nearest even, saturate at +-448
  return static_cast<uint8_t>(__nv_cvt_float_to_fp8(y, __NV_SATFINITE, __NV_E4M3));
}
// e = the smallest integer in [-6, 7] with amax <= 448 * 2^e
__device__ __forceinline__ int fp8_scale_exp(float amax) {
  int e = -6;
  while (e < 7 && amax > ldexpf(448.f, e)) ++e;
  return e;
}
// maximum over the CTA (blockDim.x <= 128 threads) of two values at once
__device__ __forceinline__ void cta_max2(float& a, float& b, float (*sm)[2]) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  a = warp_max(a);
  b = warp_max(b);
  if (lane == 0) { sm[warp][0] = a; sm[warp][1] = b; }
  __syncthreads();
  a = sm[0][0];
  b = sm[0][1];
  for (int w = 1; w < (blockDim.x + 31) / 32; ++w) { a = fmaxf(a, sm[w][0]); b = fmaxf(b, sm[w][1]); }
  __syncthreads();
}

struct Fp8Params {
  const __nv_bfloat16* k_src;        // bf16 pool (quantise) — strides below; null otherwise
  const __nv_bfloat16* v_src;
  int64_t src_stride_page, src_stride_head, src_stride_tok;
  uint8_t* k_codes;                  // fp8 pool
  uint8_t* v_codes;
  int64_t stride_page, stride_head, stride_tok;
  float* k_scale;
  float* v_scale;
  __nv_bfloat16* kmin;
  __nv_bfloat16* kmax;
  const int32_t* page_table;
  const int32_t* kv_len;
  const __nv_bfloat16* k_blk;        // [N, B, H_kv, d] (append)
  const __nv_bfloat16* v_blk;
  int32_t* status;
  int B, Hkv, D, g, Pmax, n_phys;
};

// MODE 0: quantise a bf16 pool page by page (+ summaries); MODE 1: summaries of an FP8 pool;
// MODE 2: append the block to the touched pages (re-quantising them, + summaries).
template <int MODE>
__global__ void fp8_pages_kernel(Fp8Params p) {
  grid_dep_wait();
  __shared__ float sm[4][2];
  const int kh = blockIdx.y, s = blockIdx.z, j = threadIdx.x;
  const int L0 = p.kv_len[s];
  int page, n_old, n_all;
  if (MODE == 2) {
    page = L0 / p.g + blockIdx.x;
    if (page > (L0 + p.B - 1) / p.g) return;
    if (page >= p.Pmax) { if (j == 0) set_status(p.status, LOSA_ERR_BOUNDS); return; }
    n_old = max(0, L0 - page * p.g);
    n_all = min(L0 + p.B, (page + 1) * p.g) - page * p.g;
  } else {
    page = blockIdx.x;
    n_old = n_all = min(p.g, L0 - page * p.g);
    if (n_all <= 0) return;
  }
  const int phys = p.page_table[static_cast<size_t>(s) * p.Pmax + page];
  if (phys < 0 || phys >= p.n_phys) { if (j == 0) set_status(p.status, LOSA_ERR_BOUNDS); return; }
  const size_t co = static_cast<size_t>(phys) * p.stride_page + static_cast<size_t>(kh) * p.stride_head + j;
  const size_t so = static_cast<size_t>(phys) * p.Hkv + kh;
  const float ks_old = MODE == 0 ? 1.f : p.k_scale[so], vs_old = MODE == 0 ? 1.f : p.v_scale[so];
  // row t of this thread's column as the value to encode: old rows dequantised, new rows from the block
  auto value = [&](bool is_v, int t) -> float {
    if (MODE == 0) {
      const size_t o = static_cast<size_t>(phys) * p.src_stride_page + static_cast<size_t>(kh) * p.src_stride_head +
                       static_cast<size_t>(t) * p.src_stride_tok + j;
      return __bfloat162float((is_v ? p.v_src : p.k_src)[o]);
    }
    if (t < n_old) return (is_v ? vs_old : ks_old) * fp8_value((is_v ? p.v_codes : p.k_codes)[co + static_cast<size_t>(t) * p.stride_tok]);
    const int row = page * p.g + t - L0;               // block token
    return __bfloat162float((is_v ? p.v_blk : p.k_blk)[((static_cast<size_t>(s) * p.B + row) * p.Hkv + kh) * p.D + j]);
  };
  float ks = ks_old, vs = vs_old;
  if (MODE != 1) {
    float ka = 0.f, va = 0.f;
    for (int t = 0; t < n_all; ++t) {
      ka = fmaxf(ka, fabsf(value(false, t)));
      va = fmaxf(va, fabsf(value(true, t)));
    }
    cta_max2(ka, va, sm);
    const int ke = fp8_scale_exp(ka), ve = fp8_scale_exp(va);
    ks = ldexpf(1.f, ke);
    vs = ldexpf(1.f, ve);
    // every thread has read what it needs of the old codes of ITS column only after this point again
    for (int t = 0; t < p.g; ++t) {
      const size_t at = co + static_cast<size_t>(t) * p.stride_tok;
      const uint8_t kc = t < n_all ? fp8_code(ldexpf(value(false, t), -ke)) : 0;
      const uint8_t vc = t < n_all ? fp8_code(ldexpf(value(true, t), -ve)) : 0;
      p.k_codes[at] = kc;                              // row t of this column is not read again below t
      p.v_codes[at] = vc;
    }
    if (j == 0) { p.k_scale[so] = ks; p.v_scale[so] = vs; }
  }
  // summaries of the dequantised keys
  float lo = INFINITY, hi = -INFINITY;
  for (int t = 0; t < n_all; ++t) {
    const float v = ks * fp8_value(p.k_codes[co + static_cast<size_t>(t) * p.stride_tok]);
    lo = fminf(lo, v);
    hi = fmaxf(hi, v);
  }
  p.kmin[so * p.D + j] = __float2bfloat16_rn(lo);      // exact: four significant bits
  p.kmax[so * p.D + j] = __float2bfloat16_rn(hi);
}

Fp8Params base_params(losa_ctx* c, const losa_kv_t* kv) {
  const losa_shape_t& sh = c->shape;
  Fp8Params p = {};
  p.k_codes = static_cast<uint8_t*>(kv->k_pages);
  p.v_codes = static_cast<uint8_t*>(kv->v_pages);
  p.stride_page = kv->stride_page;
  p.stride_head = kv->stride_head;
  p.stride_tok = kv->stride_tok;
  p.k_scale = kv->k_scale;
  p.v_scale = kv->v_scale;
  p.kmin = static_cast<__nv_bfloat16*>(kv->kmin);
  p.kmax = static_cast<__nv_bfloat16*>(kv->kmax);
  p.page_table = kv->page_table;
  p.kv_len = kv->kv_len;
  p.status = status_ptr(c);
  p.B = sh.block_size;
  p.Hkv = sh.n_kv_heads;
  p.D = sh.head_dim;
  p.g = sh.page_size;
  p.Pmax = sh.max_pages_per_seq;
  p.n_phys = kv->n_phys_pages;
  return p;
}

}  // namespace

int32_t launch_fp8_quantize(losa_ctx* c, const losa_kv_t* src, losa_kv_t* dst, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  if (sh.max_pages_per_seq == 0) return LOSA_OK;
  Fp8Params p = base_params(c, dst);
  p.k_src = static_cast<const __nv_bfloat16*>(src->k_pages);
  p.v_src = static_cast<const __nv_bfloat16*>(src->v_pages);
  p.src_stride_page = src->stride_page;
  p.src_stride_head = src->stride_head;
  p.src_stride_tok = src->stride_tok;
  launch_k(fp8_pages_kernel<0>, dim3(sh.max_pages_per_seq, sh.n_kv_heads, sh.batch), sh.head_dim, 0, st, p);
  return after_launch(c);
}

int32_t launch_fp8_summaries(losa_ctx* c, losa_kv_t* kv, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  if (sh.max_pages_per_seq == 0) return LOSA_OK;
  const Fp8Params p = base_params(c, kv);
  launch_k(fp8_pages_kernel<1>, dim3(sh.max_pages_per_seq, sh.n_kv_heads, sh.batch), sh.head_dim, 0, st, p);
  return after_launch(c);
}

// the kv_len / step counters are bumped by the caller's usual counter kernel afterwards
int32_t launch_fp8_append(losa_ctx* c, losa_kv_t* kv, const void* k_blk, const void* v_blk, cudaStream_t st) {
  const losa_shape_t& sh = c->shape;
  Fp8Params p = base_params(c, kv);
  p.k_blk = static_cast<const __nv_bfloat16*>(k_blk);
  p.v_blk = static_cast<const __nv_bfloat16*>(v_blk);
  const int touched = (sh.block_size + sh.page_size - 1) / sh.page_size + 1;
  launch_k(fp8_pages_kernel<2>, dim3(touched, sh.n_kv_heads, sh.batch), sh.head_dim, 0, st, p);
  return after_launch(c);
}

}  // namespace losa
