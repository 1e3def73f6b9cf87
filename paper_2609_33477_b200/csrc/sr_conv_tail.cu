// Convolution state (Appendix A, "Native cache": the layer keeps the last w-1 inputs of each of
// its C = 2 H_k d_k + H_v d_v convolution channels, in BF16).
//
//   out_conv[slot][c][j] = bf16( Z[R - (w-1) + j][c] ),  j = 0 .. w-2, zero for rows before the window
//
// The k and v channels are read from the raw rows the projection kept.  The q channels are the only use the
// path has for the query projection, so they are computed here, for the last w-1 rows of each
// request only: one skinny GEMM over the whole batch -- (w-1) B gathered anchor rows x channels -- on mma.sync
// tiles (sr_conv_tail_gemm_kernel), so every weight row is read once per 64 rows instead of once per request.
// With block-scaled weights that GEMM covers the k and v channels too (codes and scales in fp32), because the
// projection's copies of those rows went through a rounded 16-bit weight.  Plain dot products, one warp per
// channel, serve the geometries the tiles do not divide.
#include "sr_mma.cuh"

namespace {

__device__ __forceinline__ float e4m3_to_float(uint8_t code) {
  __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)code, __NV_E4M3);
  return __half2float(__half(h));
}

template <bool FP8>
__global__ void __launch_bounds__(256)
sr_conv_tail_kernel(SrSched s, SrPoolView pool, int32_t pool_layer, int32_t d_model, int32_t n_q, int32_t c_begin, int32_t conv_ch,
                    const void* __restrict__ w_qkv, const float* __restrict__ w_scale,
                    const float* __restrict__ zraw, int32_t n_kv,
                    const __nv_bfloat16* __restrict__ hist, char* __restrict__ out_layer, int64_t slot_stride) {
  const int i = blockIdx.y;
  const int out_slot = s.req_out[i];
  if (out_slot < 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = c_begin + blockIdx.x * 8 + warp;
  if (c >= conv_ch) return;
  const int R = s.req_rows[i];
  const int slot0 = s.req_slot0[i];
  if (!sr_check_out(s, out_slot) || (R > 0 && !sr_check_slot(s, slot0 + (R - 1) / SR_PAGE_ROWS))) return;
  float val[SR_CONV_W - 1];
#pragma unroll
  for (int j = 0; j < SR_CONV_W - 1; ++j) val[j] = 0.f;

  if (c >= n_q) {
    if (lane < SR_CONV_W - 1) {
      const int t = R - (SR_CONV_W - 1) + lane;
      float v = 0.f;
      if (t >= 0) {
        // the projection kept the last three valid raw rows of every slot
        const int slot = slot0 + t / SR_PAGE_ROWS, rho = t % SR_PAGE_ROWS;
        const int idx = 3 + rho - max(s.slot_rows[slot] - 3, 0);
        v = zraw[((int64_t)slot * 6 + idx) * n_kv + (c - n_q)];
      }
      val[0] = v;   // lane j holds entry j
    }
  } else {
    const char* rows[SR_CONV_W - 1];
#pragma unroll
    for (int j = 0; j < SR_CONV_W - 1; ++j) {
      const int t = R - (SR_CONV_W - 1) + j;
      rows[j] = nullptr;
      if (t >= 0) {
        const int slot = slot0 + t / SR_PAGE_ROWS;
        if (sr_check_page(s, s.slot_page[slot]))
          rows[j] = pool.base + (int64_t)s.slot_page[slot] * pool.page_stride + (int64_t)pool_layer * pool.layer_stride +
                    (int64_t)(t % SR_PAGE_ROWS) * pool.row_stride;
      }
    }
    float acc[SR_CONV_W - 1];
#pragma unroll
    for (int j = 0; j < SR_CONV_W - 1; ++j) acc[j] = 0.f;
    for (int k0 = lane * 8; k0 < d_model; k0 += 256) {
      float wv[8];
      if (FP8) {
        const uint2 v = *(const uint2*)((const uint8_t*)w_qkv + (int64_t)c * d_model + k0);
        const uint8_t* e = (const uint8_t*)&v;
        const float sc = w_scale[(c / 128) * (d_model / 128) + k0 / 128];
#pragma unroll
        for (int q = 0; q < 8; ++q) wv[q] = e4m3_to_float(e[q]) * sc;
      } else {
        const uint4 v = *(const uint4*)((const __nv_bfloat16*)w_qkv + (int64_t)c * d_model + k0);
        const __nv_bfloat16* e = (const __nv_bfloat16*)&v;
#pragma unroll
        for (int q = 0; q < 8; ++q) wv[q] = __bfloat162float(e[q]);
      }
#pragma unroll
      for (int j = 0; j < SR_CONV_W - 1; ++j) {
        if (rows[j]) {
          const uint4 xv = *(const uint4*)(rows[j] + (int64_t)k0 * 2);
          const __nv_bfloat16* e = (const __nv_bfloat16*)&xv;
#pragma unroll
          for (int q = 0; q < 8; ++q) acc[j] = fmaf(__bfloat162float(e[q]), wv[q], acc[j]);
        }
      }
    }
#pragma unroll
    for (int j = 0; j < SR_CONV_W - 1; ++j) {
      float v = acc[j];
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      acc[j] = v;
    }
    // lane j keeps entry j, as in the other branch
    val[0] = lane == 0 ? acc[0] : (lane == 1 ? acc[1] : acc[2]);
  }
  if (lane < SR_CONV_W - 1) {
    __nv_bfloat16 o = __float2bfloat16_rn(val[0]);
    const int t = R - (SR_CONV_W - 1) + lane;
    // rows before the window: zero, or the inputs of the state this request continues (kept bit for bit)
    if (t < 0 && hist) o = hist[((int64_t)i * conv_ch + c) * (SR_CONV_W - 1) + (SR_CONV_W - 1 + t)];
    __nv_bfloat16* dst = (__nv_bfloat16*)(out_layer + (int64_t)out_slot * slot_stride) + (int64_t)c * (SR_CONV_W - 1);
    dst[lane] = o;
  }
}

// Channels as one GEMM over the batch: out[r][c] = sum_k X[r][k] W[c][k] for the gathered tail rows r = 3 i + j
// (request i, window entry j).  One CTA = 64 rows x 64 channels, four warps (each owns 16 channels for every 16-row block), k in chunks of 64
// through a four-stage ring (cp.async for the anchor rows and for bf16 weights).  Rows without a source (before a request's
// first token, past the batch, skipped requests) read some valid row and are masked on output.
//   FP8 = false: bf16 weights, the q channels only (k, v rows come from the projection).
//   FP8 = true : e4m3 codes with 128 x 128 block scales, every channel q | k | v.  The bare codes are decoded to
//                bf16 (exact) on their way into shared memory, every 128-deep k group is summed on its own and
//                enters the result as scale x partial sum in fp32 -- the weights are never rounded, so the conv
//                state of block-scaled layers is as exact as the one of bf16 layers.
constexpr int QT = 64;            // tile rows, tile channels and k chunk
constexpr int QLD = QT + 8;       // shared-memory pitch (bf16)
constexpr int QNS = 4;            // chunks in flight: the k loop is serial, so its speed is latency / depth
constexpr int QR = 4;             // quarters the k range is always summed in (see the kernel)
constexpr int SPLIT_MAX_ROWS = 256;   // tail rows (3 per request) up to which every quarter gets its own CTA

template <bool FP8, bool A8>
constexpr int conv_gemm_smem() {
  return ((A8 ? 2 : QNS) + (FP8 ? 2 : QNS)) * QT * QLD * 2 + ((A8 ? QNS : 0) + (FP8 ? QNS : 0)) * QT * QT;
}

//   A8 (with FP8): the rows are the quantiser's activation codes instead of the bf16 anchors (W8A8): decoded to
//                bf16 like the weight codes, and a 128-deep partial sum is scaled by weight scale x the row's
//                activation scale of that K group.
template <bool FP8, bool A8>
__global__ void __launch_bounds__(128)
sr_conv_tail_gemm_kernel(SrSched s, SrPoolView pool, int32_t pool_layer, int32_t d_model, int32_t conv_ch,
                         const void* __restrict__ w_rows, const float* __restrict__ w_scale,
                         const uint8_t* __restrict__ x8, const float* __restrict__ sx,
                         const __nv_bfloat16* __restrict__ hist, char* __restrict__ out_layer, int64_t slot_stride,
                         float* __restrict__ part, int32_t part_rows, int32_t part_ch) {
  // Shared memory: a ring of QNS stages per operand.  A 16-bit operand is copied straight into its padded tile
  // (cp.async, 16 bytes); an 8-bit operand lands as raw bytes (cp.async, 8 bytes) and the thread that fetched them
  // decodes them into one of two bf16 tiles just before the chunk is used.
  extern __shared__ __align__(16) uint8_t qsm[];
  constexpr int TILE_B = QT * QLD * 2, RAW_B = QT * QT;
  __half* Xt = (__half*)qsm;                                              // [A8 ? 2 : QNS] tiles
  __half* Wt = (__half*)(qsm + (A8 ? 2 : QNS) * TILE_B);                  // [FP8 ? 2 : QNS] tiles
  uint8_t* Xraw = qsm + ((A8 ? 2 : QNS) + (FP8 ? 2 : QNS)) * TILE_B;      // [QNS] raw chunks (A8)
  uint8_t* Wraw = Xraw + (A8 ? QNS * RAW_B : 0);                          // [QNS] raw chunks (FP8)
  const int tid = threadIdx.x, warp = tid >> 5, l = tid & 31, g8 = l >> 2, t4 = l & 3;
  const int c0 = blockIdx.x * QT, r0 = blockIdx.y * QT;
  const int seg = tid & 7;
  const char* xrow[4];
  const char* wrow[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int m = (tid >> 3) + 16 * q;
    const int gr = r0 + m, i = gr / (SR_CONV_W - 1), j = gr % (SR_CONV_W - 1);
    // stand-in row (masked later): the pool's first row, or the first row of the first slot's codes
    const char* src = A8 ? (const char*)x8 : pool.base + (int64_t)pool_layer * pool.layer_stride;
    if (i < s.n_requests && s.req_out[i] >= 0) {
      const int t = s.req_rows[i] - (SR_CONV_W - 1) + j;
      if (t >= 0) {
        const int slot = s.req_slot0[i] + t / SR_PAGE_ROWS;
        if (A8) {
          if (sr_check_slot(s, slot)) src = (const char*)x8 + ((int64_t)slot * SR_PAGE_ROWS + t % SR_PAGE_ROWS) * d_model;
        } else if (sr_check_slot(s, slot) && sr_check_page(s, s.slot_page[slot])) {
          src = pool.base + (int64_t)s.slot_page[slot] * pool.page_stride + (int64_t)pool_layer * pool.layer_stride +
                (int64_t)(t % SR_PAGE_ROWS) * pool.row_stride;
        }
      }
    }
    xrow[q] = src + seg * (A8 ? 8 : 16);
    // bf16: 16 bytes = 8 weights per thread and row; e4m3: 8 bytes = 8 codes
    wrow[q] = (const char*)w_rows + ((int64_t)(c0 + m) * d_model + seg * 8) * (FP8 ? 1 : 2);
  }
  auto load = [&](int kc, int ring) {  // chunk kc -> ring stage ring % QNS
    const int st = ring % QNS;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int m = (tid >> 3) + 16 * q;
      if (A8) cp_async8(Xraw + st * RAW_B + m * QT + seg * 8, xrow[q] + (int64_t)kc * QT);
      else cp_async16(Xt + st * (QT * QLD) + m * QLD + seg * 8, xrow[q] + (int64_t)kc * QT * 2);
      if (FP8) cp_async8(Wraw + st * RAW_B + m * QT + seg * 8, wrow[q] + (int64_t)kc * QT);
      else cp_async16(Wt + st * (QT * QLD) + m * QLD + seg * 8, wrow[q] + (int64_t)kc * QT * 2);
    }
  };
  auto decode_own = [&](const uint8_t* raw, __half* tile) {      // this thread's own bytes: no barrier needed before
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int m = (tid >> 3) + 16 * q;
      const uint2 codes = *(const uint2*)(raw + m * QT + seg * 8);
      const uint8_t* e = (const uint8_t*)&codes;
      __align__(16) __nv_bfloat16 o[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) o[k] = __float2bfloat16_rn(e4m3_to_float(e[k]));     // exact: 4 significant bits
      *(uint4*)(tile + m * QLD + seg * 8) = *(const uint4*)o;
    }
  };
  // Work split: warp w owns channels 16 w .. 16 w + 15 of the tile for every 16-row block that holds a tail row (the
  // tail rows of a tile are its first n_rb blocks), so one weight fragment serves four row blocks and the products of
  // a step do not wait on one another.  A thread's accumulator rows: 16 rb + g8 and 16 rb + g8 + 8.
  const int rows_here = min(QT, s.n_requests * (SR_CONV_W - 1) - r0);
  const int n_rb = (rows_here + 15) / 16;
  // A8: the activation scales of those rows, one float per K group (stride 64 floats)
  const float* sxrow[4][2];
#pragma unroll
  for (int rb = 0; rb < 4; ++rb)
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      sxrow[rb][hr] = sx;
      if (A8) {
        const int gr = r0 + rb * 16 + g8 + 8 * hr, i = gr / (SR_CONV_W - 1), j = gr % (SR_CONV_W - 1);
        if (i < s.n_requests && s.req_out[i] >= 0) {
          const int t = s.req_rows[i] - (SR_CONV_W - 1) + j;
          if (t >= 0) {
            const int slot = s.req_slot0[i] + t / SR_PAGE_ROWS;
            if (slot >= 0 && slot < s.max_slots) sxrow[rb][hr] = sx + (int64_t)slot * (d_model / 128) * SR_PAGE_ROWS + t % SR_PAGE_ROWS;
          }
        }
      }
    }
  float acc[4][2][4], total[4][2][4];
#pragma unroll
  for (int rb = 0; rb < 4; ++rb)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int c = 0; c < 4; ++c) { acc[rb][n][c] = 0.f; total[rb][n][c] = 0.f; }
  const int nk = d_model / QT;
  const float* scale_row = FP8 ? w_scale + (int64_t)(c0 / 128) * (d_model / 128) : nullptr;
  // The sum over k is ALWAYS formed as ((r_0 + r_1) + r_2) + r_3, r_z the sum over the z-th quarter of the chunks
  // (quarters of the 128-deep groups for block-scaled weights): a small batch gives every quarter its own CTA
  // (gridDim.z = QR, partial sums to `part`, added up by the finishing kernel), a large one walks the quarters in
  // one CTA -- the same numbers added in the same order, so a request's conv state does not depend on the batch it
  // arrives in.
  float fin[4][2][4];
#pragma unroll
  for (int rb = 0; rb < 4; ++rb)
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int c = 0; c < 4; ++c) fin[rb][n][c] = 0.f;
  const int z0 = part ? (int)blockIdx.z : 0, z1 = part ? z0 + 1 : QR;
  for (int z = z0; z < z1; ++z) {
    const int kb = FP8 ? 2 * ((z * (nk / 2)) / QR) : (z * nk) / QR;
    const int ke = FP8 ? 2 * (((z + 1) * (nk / 2)) / QR) : ((z + 1) * nk) / QR;
    for (int kc = kb; kc < kb + QNS - 1; ++kc) {       // fill the ring; one commit group per chunk, empty ones past the end
      if (kc < ke) load(kc, kc - kb);
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    for (int kc = kb; kc < ke; ++kc) {
      const int ring = kc - kb;
      asm volatile("cp.async.wait_group %0;" ::"n"(QNS - 2) : "memory");      // this thread's part of chunk kc has landed
      const __half* xt = A8 ? Xt + (ring & 1) * (QT * QLD) : Xt + (ring % QNS) * (QT * QLD);
      const __half* wt = FP8 ? Wt + (ring & 1) * (QT * QLD) : Wt + (ring % QNS) * (QT * QLD);
      if (A8) decode_own(Xraw + (ring % QNS) * RAW_B, (__half*)xt);
      if (FP8) decode_own(Wraw + (ring % QNS) * RAW_B, (__half*)wt);
      __syncthreads();                  // chunk kc is complete for everyone; everyone is done with chunk kc - 1
      if (kc + QNS - 1 < ke) load(kc + QNS - 1, ring + QNS - 1);             // into the stage chunk kc - 1 used
      asm volatile("cp.async.commit_group;" ::: "memory");
#pragma unroll
      for (int ks = 0; ks < QT / 16; ++ks) {
        uint32_t bf[4];
        ldsm4(bf, bn_addr(wt, QLD, warp * 16, ks * 16, l));
#pragma unroll
        for (int rb = 0; rb < 4; ++rb) {
          if (rb < n_rb) {
            uint32_t a[4];
            ldsm4(a, a_addr(xt, QLD, rb * 16, ks * 16, l));
            mma16816_bf16(acc[rb][0], a, bf[0], bf[1]);
            mma16816_bf16(acc[rb][1], a, bf[2], bf[3]);
          }
        }
      }
      if (FP8 && (kc & 1)) {         // a 128-deep k group is complete: it shares one block scale
        const float sc = __ldg(scale_row + (kc >> 1));
#pragma unroll
        for (int rb = 0; rb < 4; ++rb) {
          if (rb < n_rb) {
            const float s0 = A8 ? sc * __ldg(sxrow[rb][0] + (int64_t)(kc >> 1) * SR_PAGE_ROWS) : sc;
            const float s1 = A8 ? sc * __ldg(sxrow[rb][1] + (int64_t)(kc >> 1) * SR_PAGE_ROWS) : sc;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
              for (int c = 0; c < 4; ++c) { total[rb][n][c] = fmaf(c < 2 ? s0 : s1, acc[rb][n][c], total[rb][n][c]); acc[rb][n][c] = 0.f; }
          }
        }
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                    // the ring is idle before the next quarter refills it
    // this quarter's sum: into the running total, or out to the partial-sum buffer
#pragma unroll
    for (int rb = 0; rb < 4; ++rb)
#pragma unroll
      for (int n = 0; n < 2; ++n) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float r = FP8 ? total[rb][n][c] : acc[rb][n][c];
          fin[rb][n][c] += r;
          acc[rb][n][c] = 0.f;
          total[rb][n][c] = 0.f;
        }
        if (part && rb < n_rb) {
          const int ch = c0 + warp * 16 + n * 8 + 2 * t4;
          float* dstp = part + ((int64_t)z * part_rows + r0 + rb * 16 + g8) * part_ch + ch;
          *(float2*)dstp = make_float2(fin[rb][n][0], fin[rb][n][1]);
          *(float2*)(dstp + (int64_t)8 * part_ch) = make_float2(fin[rb][n][2], fin[rb][n][3]);
        }
      }
  }
  if (part) return;                     // the finishing kernel adds the quarters up and writes the state
#pragma unroll
  for (int rb = 0; rb < 4; ++rb) {
#pragma unroll
    for (int hr = 0; hr < 2; ++hr) {
      const int gr = r0 + rb * 16 + g8 + 8 * hr, i = gr / (SR_CONV_W - 1), j = gr % (SR_CONV_W - 1);
      if (rb >= n_rb || i >= s.n_requests) continue;
      const int out_slot = s.req_out[i];
      if (out_slot < 0 || !sr_check_out(s, out_slot)) continue;
      const int t = s.req_rows[i] - (SR_CONV_W - 1) + j;
      // rows before the window: zero, or the inputs of the state this request continues (kept bit for bit)
      const __nv_bfloat16* old = (t < 0 && hist) ? hist + (int64_t)i * conv_ch * (SR_CONV_W - 1) + (SR_CONV_W - 1 + t) : nullptr;
      __nv_bfloat16* dst = (__nv_bfloat16*)(out_layer + (int64_t)out_slot * slot_stride) + j;
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        const int c = c0 + warp * 16 + n * 8 + 2 * t4;
        const float v0 = fin[rb][n][2 * hr], v1 = fin[rb][n][2 * hr + 1];
        __nv_bfloat16 o0 = __float2bfloat16_rn(t >= 0 ? v0 : 0.f), o1 = __float2bfloat16_rn(t >= 0 ? v1 : 0.f);
        if (old) {
          o0 = old[(int64_t)c * (SR_CONV_W - 1)];
          o1 = old[(int64_t)(c + 1) * (SR_CONV_W - 1)];
        }
        dst[(int64_t)c * (SR_CONV_W - 1)] = o0;
        dst[(int64_t)(c + 1) * (SR_CONV_W - 1)] = o1;
      }
    }
  }
}

// k and v channels from the rows the fused projection kept, and the channels whose k quarters were summed by separate
// CTAs (`part`: [quarter][tail row][channel], channels 0 .. part_ch - 1): one thread per (request, channel), so the
// reads of a row are contiguous across the warp and a thread writes its channel's w-1 entries side by side
__global__ void __launch_bounds__(256)
sr_conv_tail_kv_kernel(SrSched s, int32_t c_begin, int32_t n_q, int32_t conv_ch, const float* __restrict__ zraw, int32_t n_kv,
                       const __nv_bfloat16* __restrict__ hist, char* __restrict__ out_layer, int64_t slot_stride,
                       const float* __restrict__ part, int32_t part_rows, int32_t part_ch) {
  const int i = blockIdx.y;
  const int out_slot = s.req_out[i];
  if (out_slot < 0) return;
  const int c = c_begin + blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= conv_ch) return;
  const bool from_part = part && c < part_ch;
  if (!from_part && c < n_q) return;              // written by the batched kernel itself
  const int R = s.req_rows[i], slot0 = s.req_slot0[i];
  if (!sr_check_out(s, out_slot) || (R > 0 && !sr_check_slot(s, slot0 + (R - 1) / SR_PAGE_ROWS))) return;
  __nv_bfloat16* dst = (__nv_bfloat16*)(out_layer + (int64_t)out_slot * slot_stride) + (int64_t)c * (SR_CONV_W - 1);
#pragma unroll
  for (int j = 0; j < SR_CONV_W - 1; ++j) {
    const int t = R - (SR_CONV_W - 1) + j;
    __nv_bfloat16 o = __float2bfloat16_rn(0.f);
    if (t >= 0) {
      if (from_part) {
        const int64_t gr = (int64_t)i * (SR_CONV_W - 1) + j;
        float v = 0.f;
#pragma unroll
        for (int z = 0; z < QR; ++z) v += part[((int64_t)z * part_rows + gr) * part_ch + c];
        o = __float2bfloat16_rn(v);
      } else {
        const int slot = slot0 + t / SR_PAGE_ROWS, rho = t % SR_PAGE_ROWS;
        const int idx = 3 + rho - max(s.slot_rows[slot] - 3, 0);
        o = __float2bfloat16_rn(zraw[((int64_t)slot * 6 + idx) * n_kv + (c - n_q)]);
      }
    } else if (hist) {
      o = hist[((int64_t)i * conv_ch + c) * (SR_CONV_W - 1) + (SR_CONV_W - 1 + t)];
    }
    dst[j] = o;
  }
}

// hist[request][c][j] = in_conv[state slot of the request][c][j] (zero for requests that write nothing)
__global__ void __launch_bounds__(256)
sr_hist_gather_kernel(SrSched s, const char* __restrict__ in_layer, int64_t slot_stride, int32_t n_vals,
                      __nv_bfloat16* __restrict__ hist) {
  const int i = blockIdx.y;
  const int out_slot = s.req_out[i];
  const __nv_bfloat16* src = out_slot >= 0 ? (const __nv_bfloat16*)(in_layer + (int64_t)out_slot * slot_stride) : nullptr;
  for (int k = blockIdx.x * blockDim.x + threadIdx.x; k < n_vals; k += gridDim.x * blockDim.x)
    hist[(int64_t)i * n_vals + k] = src ? src[k] : __float2bfloat16_rn(0.f);
}

}  // namespace

// kernels one sr_launch_conv_tail call launches: bf16 weights, the batched q GEMM plus the k | v copy; block-scaled
// weights, one GEMM over all channels; geometries the 64-wide tiles do not divide, the single dot-product kernel
// The batched kernel serves every batch size its tiles divide, so that a request's conv state has the same bits
// whatever batch it arrives in.
static bool conv_tail_gemm_fits(const sr_ctx* ctx, int n_requests) {
  const bool fp8 = ctx->desc.weight_format == SR_W_E4M3_BLOCK128;
  if (ctx->w8a8) return true;        // quantised activations: the batched kernel is the only form (checked at sr_create)
  return (fp8 ? ctx->conv_ch : ctx->n_k) % QT == 0 && ctx->desc.d_model % (fp8 ? 128 : QT) == 0 &&
         !(ctx->debug_flags & SR_DEBUG_DOT_CONV_STATE);
}

static bool conv_tail_split(const sr_ctx* ctx, int n_requests) {
  return conv_tail_gemm_fits(ctx, n_requests) && n_requests * (SR_CONV_W - 1) <= SPLIT_MAX_ROWS;
}

int sr_conv_tail_launches(const sr_ctx* ctx, int n_requests) {
  if (!conv_tail_gemm_fits(ctx, n_requests)) return 1;
  return (ctx->desc.weight_format == SR_W_E4M3_BLOCK128 && !conv_tail_split(ctx, n_requests)) ? 1 : 2;
}

// bytes of the partial-sum buffer a lane needs (small batches: the k quarters are summed by separate CTAs)
size_t sr_conv_tail_part_bytes(const sr_ctx* ctx) {
  const size_t ch = ctx->desc.weight_format == SR_W_E4M3_BLOCK128 ? ctx->conv_ch : ctx->n_k;
  return (size_t)QR * SPLIT_MAX_ROWS * ch * sizeof(float);
}

cudaError_t sr_launch_conv_tail(const sr_ctx* ctx, const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                const sr_layer_weights& w, const SrFused& fused, char* out_conv_layer,
                                int64_t slot_stride, cudaStream_t stream) {
  const float* zraw = fused.zraw;
  const __nv_bfloat16* hist = fused.hist;
  const int n_kv = ctx->n_k + ctx->n_v;
  const int tail_rows = s.n_requests * (SR_CONV_W - 1);
  const cudaError_t once = sr_once_per_device(SR_ONCE_CONV_GEMM, [] {
    cudaError_t e = cudaFuncSetAttribute(sr_conv_tail_gemm_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         conv_gemm_smem<false, false>());
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(sr_conv_tail_gemm_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               conv_gemm_smem<true, false>());
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(sr_conv_tail_gemm_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               conv_gemm_smem<true, true>());
    return e;
  });
  if (once != cudaSuccess) return once;
  const bool fp8 = ctx->desc.weight_format == SR_W_E4M3_BLOCK128;
  const int n_q = ctx->n_k;
  if (conv_tail_gemm_fits(ctx, s.n_requests)) {
    // the batched kernel: the q channels (bf16 weights; k and v rows come from the raw rows the projection kept), or
    // every channel from codes and scales in fp32 (block-scaled weights: the conv state never sees a rounded weight)
    const int gemm_ch = fp8 ? ctx->conv_ch : n_q;
    const bool split = conv_tail_split(ctx, s.n_requests) && fused.qpart != nullptr;
    const int row_tiles = (tail_rows + QT - 1) / QT;
    float* part = split ? fused.qpart : nullptr;
    const int part_rows = row_tiles * QT;
    dim3 g((unsigned)(gemm_ch / QT), (unsigned)row_tiles, split ? QR : 1);
    if (!fp8)
      sr_conv_tail_gemm_kernel<false, false><<<g, 128, conv_gemm_smem<false, false>(), stream>>>(
          s, pool, pool_layer, ctx->desc.d_model, ctx->conv_ch, w.w_qkv, nullptr, nullptr, nullptr, hist, out_conv_layer, slot_stride,
          part, part_rows, gemm_ch);
    else if (ctx->w8a8)
      sr_conv_tail_gemm_kernel<true, true><<<g, 128, conv_gemm_smem<true, true>(), stream>>>(
          s, pool, pool_layer, ctx->desc.d_model, ctx->conv_ch, w.w_qkv, w.w_qkv_scale, fused.x8, fused.sx, hist, out_conv_layer,
          slot_stride, part, part_rows, gemm_ch);
    else
      sr_conv_tail_gemm_kernel<true, false><<<g, 128, conv_gemm_smem<true, false>(), stream>>>(
          s, pool, pool_layer, ctx->desc.d_model, ctx->conv_ch, w.w_qkv, w.w_qkv_scale, nullptr, nullptr, hist, out_conv_layer,
          slot_stride, part, part_rows, gemm_ch);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || (fp8 && !split)) return e;
    // the k | v copy (bf16 weights) and, for a split sum, the channels whose quarters are added up here
    const int c_begin = split ? 0 : n_q;
    dim3 gkv((unsigned)((ctx->conv_ch - c_begin + 255) / 256), (unsigned)s.n_requests);
    sr_conv_tail_kv_kernel<<<gkv, 256, 0, stream>>>(s, c_begin, fp8 ? ctx->conv_ch : n_q, ctx->conv_ch, zraw, n_kv, hist, out_conv_layer,
                                                    slot_stride, part, part_rows, gemm_ch);
    return cudaGetLastError();
  }
  dim3 grid((unsigned)((ctx->conv_ch + 7) / 8), (unsigned)s.n_requests);
  if (fp8)
    sr_conv_tail_kernel<true><<<grid, 256, 0, stream>>>(s, pool, pool_layer, ctx->desc.d_model, ctx->conv_ch, 0, ctx->conv_ch, w.w_qkv,
                                                        w.w_qkv_scale, zraw, n_kv, hist, out_conv_layer, slot_stride);
  else
    sr_conv_tail_kernel<false><<<grid, 256, 0, stream>>>(s, pool, pool_layer, ctx->desc.d_model, n_q, 0, ctx->conv_ch, w.w_qkv, nullptr,
                                                         zraw, n_kv, hist, out_conv_layer, slot_stride);
  return cudaGetLastError();
}

cudaError_t sr_launch_conv_tail_from_raw(const sr_ctx* ctx, const SrSched& s, const SrFused& fused, char* out_conv_layer,
                                         int64_t slot_stride, cudaStream_t stream) {
  // every conv channel was projected for every row: the last rows are all in zraw (n_q = 0, n_kv = C)
  dim3 g((unsigned)((ctx->conv_ch + 255) / 256), (unsigned)s.n_requests);
  sr_conv_tail_kv_kernel<<<g, 256, 0, stream>>>(s, 0, 0, ctx->conv_ch, fused.zraw, ctx->conv_ch, nullptr, out_conv_layer, slot_stride, nullptr,
                                                0, 0);
  return cudaGetLastError();
}

cudaError_t sr_launch_hist_gather(const sr_ctx* ctx, const SrSched& s, const char* in_conv_layer, int64_t slot_stride,
                                  __nv_bfloat16* hist, cudaStream_t stream) {
  const int n_vals = ctx->conv_ch * (SR_CONV_W - 1);
  dim3 grid((unsigned)((n_vals + 1023) / 1024), (unsigned)s.n_requests);
  sr_hist_gather_kernel<<<grid, 256, 0, stream>>>(s, in_conv_layer, slot_stride, n_vals, hist);
  return cudaGetLastError();
}
