// Operand staging for e4m3 weights with 128 x 128 block scales (W8A16, Section 7.1 precision setting): the fp16
// copies the default projection multiplies, and the exact bf16 decode of the bare codes for the fp32-promotion form.
//
// The tensor cores take both operands of one product in the same 16-bit format.  Rounding code x scale to bf16
// (8 significant bits) would cost about 1e-3 relative error per projected value, too close to the state
// tolerance, so both operands go to fp16 (11 significant bits) instead, once per layer:
//
//   weights  w16[c][k] = fp16( decode(code[c][k]) * scale[c/128][k/128] * 2^6 )   k | v rows, then the gate rows
//   anchors  x16[slot][row][k] = fp16( x[page(slot)][row][k] * 2^-6 )              in page-slot order
//
// The powers of two cancel in the product and centre the ranges: anchors up to 4e6 in magnitude stay finite and
// are exact down to 4e-3 (below that the absolute error is at most 2^-19), weights are exact to 2^-12 relative
// for magnitudes from 1e-6 to 1e3.  After this the projection is the same kernel as for bf16 weights.
#include <cuda_fp8.h>

#include "sr_common.cuh"

namespace {

constexpr float W_UP = 64.f, X_DOWN = 1.f / 64.f;

__global__ void __launch_bounds__(256)
sr_stage_weights_fp16_kernel(const uint8_t* __restrict__ codes, const float* __restrict__ scale,
                             const __nv_bfloat16* __restrict__ gate_w, __half* __restrict__ out, long long n16_kv,
                             long long n16_all, int d_model, int row0) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // 16 weights per thread, inside one scale block
  if (i >= n16_all) return;
  const long long e0 = i * 16;
  __align__(16) __half o[16];
  if (i < n16_kv) {
    const int row = (int)(e0 / d_model), k = (int)(e0 % d_model);
    const float sc = scale[(long long)((row0 + row) / 128) * (d_model / 128) + k / 128] * W_UP;
    const uint4 v = *(const uint4*)(codes + e0);
    const uint8_t* e = (const uint8_t*)&v;
#pragma unroll
    for (int q = 0; q < 16; ++q) {
      const __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)e[q], __NV_E4M3);
      o[q] = __float2half_rn(__half2float(__half(hr)) * sc);
    }
  } else {
    const __nv_bfloat16* src = gate_w + (e0 - n16_kv * 16);
#pragma unroll
    for (int q = 0; q < 16; ++q) o[q] = __float2half_rn(__bfloat162float(src[q]) * W_UP);
  }
  *(uint4*)(out + e0) = *(const uint4*)o;
  *(uint4*)(out + e0 + 8) = *(const uint4*)(o + 8);
}

// e4m3 codes -> the same values in bf16 (exact: 4 significant bits fit in 8), no scale applied
__global__ void __launch_bounds__(256)
sr_decode_e4m3_kernel(const uint8_t* __restrict__ codes, __nv_bfloat16* __restrict__ out, long long n16) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;     // 16 codes per thread
  if (i >= n16) return;
  const uint4 v = *(const uint4*)(codes + i * 16);
  const uint8_t* e = (const uint8_t*)&v;
  __align__(16) __nv_bfloat16 o[16];
#pragma unroll
  for (int q = 0; q < 16; ++q) {
    const __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)e[q], __NV_E4M3);
    o[q] = __float2bfloat16_rn(__half2float(__half(hr)));
  }
  *(uint4*)(out + i * 16) = *(const uint4*)o;
  *(uint4*)(out + i * 16 + 8) = *(const uint4*)(o + 8);
}

// one CTA per page slot: 64 rows x d_model, 8 values per thread and step
__global__ void __launch_bounds__(256)
sr_stage_anchors_fp16_kernel(SrSched s, SrPoolView pool, int32_t pool_layer, int32_t d_model, __half* __restrict__ x16) {
  const int slot = blockIdx.x;
  if (slot >= (int)s.status[1] || s.slot_rows[slot] == 0 || !sr_check_page(s, s.slot_page[slot])) return;
  const char* page = pool.base + (int64_t)s.slot_page[slot] * pool.page_stride + (int64_t)pool_layer * pool.layer_stride;
  __half* dst = x16 + (int64_t)slot * SR_PAGE_ROWS * d_model;
  const int per_row = d_model / 8;
  const int n_vec = SR_PAGE_ROWS * per_row;
  auto convert = [&](int i, const uint4& v) {
    const int r = i / per_row, c8 = i % per_row;
    const __nv_bfloat16* e = (const __nv_bfloat16*)&v;
    __align__(16) __half o[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) o[q] = __float2half_rn(__bfloat162float(e[q]) * X_DOWN);
    __stcs((uint4*)(dst + (int64_t)r * d_model + c8 * 8), *(const uint4*)o);
  };
  auto src = [&](int i) { return (const uint4*)(page + (int64_t)(i / per_row) * pool.row_stride + (int64_t)(i % per_row) * 16); };
  int i = threadIdx.x;
  for (; i + 3 * 256 < n_vec; i += 4 * 256) {               // four loads in flight per thread
    const uint4 a = __ldcs(src(i)), b = __ldcs(src(i + 256)), c = __ldcs(src(i + 512)), e = __ldcs(src(i + 768));
    convert(i, a);
    convert(i + 256, b);
    convert(i + 512, c);
    convert(i + 768, e);
  }
  for (; i < n_vec; i += 256) convert(i, __ldcs(src(i)));
}

// W8A8: the activation quantiser.  Every row of a page slot is cut into groups of 128 consecutive channels; per
// (row, group): s = max(amax, 1e-10) / 448 and code = e4m3(x / s), fp32 with IEEE division, round to nearest even,
// saturating (no NaN codes).  Codes go to x8[slot][row][d] (the projection's fp8 operand, page-slot order), scales
// to sx[slot][group][row] (one 64-float run per (slot, group), what an epilogue thread walks along its tokens).
// Rows past the request's end get code 0 and scale 0: they contribute nothing whatever the pool holds there.
// Half a warp per (row, group): 16 lanes x 8 values.
__global__ void __launch_bounds__(256)
sr_quant_anchors_e4m3_kernel(SrSched s, SrPoolView pool, int32_t pool_layer, int32_t d_model, uint8_t* __restrict__ x8,
                             float* __restrict__ sx) {
  const int slot = blockIdx.x;
  if (slot >= (((int)s.status[1] + 3) & ~3)) return;     // the padding slots of the last projection tile are written too
  const int vr = s.slot_rows[slot];
  if (vr > 0 && !sr_check_page(s, s.slot_page[slot])) return;
  const char* page = pool.base + (int64_t)s.slot_page[slot] * pool.page_stride + (int64_t)pool_layer * pool.layer_stride;
  const int groups = d_model / 128;
  const int half = threadIdx.x >> 4, l16 = threadIdx.x & 15;          // 16 half-warps per CTA
  for (int item = half; item < SR_PAGE_ROWS * groups; item += 16) {
    const int r = item / groups, g = item % groups;
    uint2 out = make_uint2(0u, 0u);
    float sc = 0.f;
    if (r < vr) {
      const uint4 v = __ldcs((const uint4*)(page + (int64_t)r * pool.row_stride + (int64_t)g * 256 + l16 * 16));
      const __nv_bfloat16* e = (const __nv_bfloat16*)&v;
      float x[8], amax = 0.f;
#pragma unroll
      for (int q = 0; q < 8; ++q) { x[q] = __bfloat162float(e[q]); amax = fmaxf(amax, fabsf(x[q])); }
#pragma unroll
      for (int off = 8; off > 0; off >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, off));
      sc = __fdiv_rn(fmaxf(amax, 1e-10f), 448.f);
      uint8_t c[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) c[q] = (uint8_t)__nv_cvt_float_to_fp8(__fdiv_rn(x[q], sc), __NV_SATFINITE, __NV_E4M3);
      out = *(const uint2*)c;
    }
    *(uint2*)(x8 + ((int64_t)slot * SR_PAGE_ROWS + r) * d_model + g * 128 + l16 * 8) = out;
    if (l16 == 0) sx[((int64_t)slot * groups + g) * SR_PAGE_ROWS + r] = sc;
  }
}

// test and diagnostic: the quantiser's output re-packed by request (rows in order, no page padding)
__global__ void __launch_bounds__(256)
sr_pack_quantised_kernel(SrSched s, int32_t d_model, const uint8_t* __restrict__ x8, const float* __restrict__ sx,
                         uint8_t* __restrict__ out_codes, float* __restrict__ out_scales, int64_t capacity_rows) {
  const int i = blockIdx.y, p = blockIdx.x;
  const int R = s.req_rows[i];
  if (p * SR_PAGE_ROWS >= R) return;
  const int slot = s.req_slot0[i] + p, rows = s.slot_rows[slot], groups = d_model / 128;
  const int64_t row0 = (int64_t)s.req_row0[i] + (int64_t)p * SR_PAGE_ROWS;
  for (int idx = threadIdx.x; idx < rows * (d_model / 16); idx += blockDim.x) {
    const int r = idx / (d_model / 16), c16 = idx % (d_model / 16);
    if (row0 + r < capacity_rows)
      *(uint4*)(out_codes + (row0 + r) * d_model + c16 * 16) = *(const uint4*)(x8 + ((int64_t)slot * SR_PAGE_ROWS + r) * d_model + c16 * 16);
  }
  for (int idx = threadIdx.x; idx < rows * groups; idx += blockDim.x) {
    const int r = idx / groups, g = idx % groups;
    if (row0 + r < capacity_rows) out_scales[(row0 + r) * groups + g] = sx[((int64_t)slot * groups + g) * SR_PAGE_ROWS + r];
  }
}

}  // namespace

cudaError_t sr_launch_quant_anchors_e4m3(const sr_ctx* ctx, const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                         uint8_t* x8, float* sx, cudaStream_t stream) {
  sr_quant_anchors_e4m3_kernel<<<(unsigned)s.max_slots, 256, 0, stream>>>(s, pool, pool_layer, ctx->desc.d_model, x8, sx);
  return cudaGetLastError();
}

cudaError_t sr_launch_pack_quantised(const sr_ctx* ctx, const SrSched& s, int32_t max_pages, const uint8_t* x8,
                                     const float* sx, void* out_codes, float* out_scales, int64_t capacity_rows,
                                     cudaStream_t stream) {
  dim3 grid((unsigned)max_pages, (unsigned)s.n_requests);
  sr_pack_quantised_kernel<<<grid, 256, 0, stream>>>(s, ctx->desc.d_model, x8, sx, (uint8_t*)out_codes, out_scales,
                                                     capacity_rows);
  return cudaGetLastError();
}

cudaError_t sr_launch_stage_weights_fp16(const sr_ctx* ctx, const sr_layer_weights& w, __half* w16, cudaStream_t stream) {
  const int d = ctx->desc.d_model;
  const long long n16_kv = (long long)(ctx->n_k + ctx->n_v) * d / 16;
  const long long n16_all = n16_kv + (long long)ctx->n_gate * d / 16;
  const uint8_t* src = (const uint8_t*)w.w_qkv + (long long)ctx->n_k * d;      // the q rows are skipped
  sr_stage_weights_fp16_kernel<<<(unsigned)((n16_all + 255) / 256), 256, 0, stream>>>(
      src, w.w_qkv_scale, (const __nv_bfloat16*)w.w_ab, w16, n16_kv, n16_all, d, ctx->n_k);
  return cudaGetLastError();
}

cudaError_t sr_launch_weight_decode(const sr_ctx* ctx, const sr_layer_weights& w, void* decoded, cudaStream_t stream) {
  // the k | v rows of the e4m3 code matrix (the q rows are skipped), 16 codes per thread
  const long long n = (long long)(ctx->n_k + ctx->n_v) * ctx->desc.d_model;
  const uint8_t* src = (const uint8_t*)w.w_qkv + (long long)ctx->n_k * ctx->desc.d_model;
  const long long n16 = n / 16;
  sr_decode_e4m3_kernel<<<(unsigned)((n16 + 255) / 256), 256, 0, stream>>>(src, (__nv_bfloat16*)decoded, n16);
  return cudaGetLastError();
}

cudaError_t sr_launch_stage_anchors_fp16(const sr_ctx* ctx, const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                         __half* x16, cudaStream_t stream) {
  sr_stage_anchors_fp16_kernel<<<(unsigned)s.max_slots, 256, 0, stream>>>(s, pool, pool_layer, ctx->desc.d_model, x16);
  return cudaGetLastError();
}
