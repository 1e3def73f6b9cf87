// Per-token outputs of a gated-delta layer, for group-propagated replay (Section 4.1): the half of the layer that
// state-only replay never computes.  With S_0 the state entering a 64-row chunk, g_i the running log-decay inside
// it, n_j = 1/|k_j| and u_j the chunk's pseudo-values (rows of U, left behind by the state chain),
//
//   S_i = e^{g_i} S_0 + sum_{j <= i} e^{g_i - g_j} n_j k_j u_j^T                       (state after the update at row i)
//   o_i = S_i^T q^_i = q^n_i ( e^{g_i} (Q S_0)_i + sum_{j <= i} e^{g_i - g_j} n_j (q_i . k_j) u_j ),
//
// q^_i = q_i / sqrt(|q_i|^2 + eps) / sqrt(d_k).  Then the output gate: y_i = RMSNorm_head(o_i) * o_norm_w * SiLU(z_i)
// (SiLU(z) arrives from the gate GEMM).  One 128-thread CTA per (value head, page slot), all chunks of the batch at
// once; products on mma.sync m16n8k16 with fp16 operands and fp32 sums: Q S_0 (64 x d_v, k = d_k), Q K^T (lower
// triangle incl. the diagonal), M U (64 x d_v, k = 64).  Row block rb (16 rows) belongs to warp 3 - rb, as in the
// chunk-local kernel.
#include "sr_mma.cuh"

namespace {

constexpr int CH = 64;
constexpr int LDK = CH + 8;       // pitch (halfs) of channel-major [channels][64] tiles
constexpr int OT = 128;           // threads
constexpr int SC_FLOATS = 256;    // per (slot, head) factors of the chunk-local kernel: ... | 128: g_i | 192: 1/|k_i|

struct OutParams {
  SrSched s;
  const __half* kv16;             // [slot][ncb * 128][64]: q | k | v tiles
  const __half* dump_s;           // [slot][H_v][d_k][d_v]
  const __half* dump_u;           // [slot][H_v][d_v][64]
  const float* sc;                // [slot][H_v][SC_FLOATS]
  const __nv_bfloat16* zg;        // [rows][H_v d_v]: SiLU of the output-gate projection
  const __nv_bfloat16* o_norm_w;  // [d_v]
  __nv_bfloat16* y;               // [rows][H_v d_v]
  int32_t ncb, k_ch0, n_k_heads, n_v_heads, d_v;
  float eps, norm_eps;
};

__device__ __forceinline__ void pack_left(const float (&x)[2][4], uint32_t (&a)[4]) {
  a[0] = pack_h2(x[0][0], x[0][1]);
  a[1] = pack_h2(x[0][2], x[0][3]);
  a[2] = pack_h2(x[1][0], x[1][1]);
  a[3] = pack_h2(x[1][2], x[1][3]);
}

template <int DK, int NT>          // NT = d_v / 8 output column tiles (d_v = 8 NT)
__global__ void __launch_bounds__(OT) sr_group_output_kernel(const OutParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  constexpr int DV = 8 * NT, LDS = DV + 8;
  __half* Qs = (__half*)smem_raw;             // [DK][LDK]
  __half* Ks = Qs + DK * LDK;                 // [DK][LDK]
  __half* Us = Ks + DK * LDK;                 // [DV][LDK]
  __half* S0 = Us + DV * LDK;                 // [DK][LDS]
  float* g = (float*)(S0 + DK * LDS);         // [64]
  float* ninv = g + CH;                       // [64]
  float* qn = ninv + CH;                      // [64]
  float* part = qn + CH;                      // [2][64]
  const int h = blockIdx.x, slot = blockIdx.y;
  if (slot >= (int)p.s.status[1] || !sr_check_slot(p.s, slot)) return;
  const int vr = p.s.slot_rows[slot];
  if (vr == 0) return;
  const int tid = threadIdx.x, warp = tid >> 5, l = tid & 31, g8 = l >> 2, t4 = l & 3;
  const int kh = h / (p.n_v_heads / p.n_k_heads);
  const bool first = p.s.slot_first[slot] != 0;               // a request's first chunk starts from the zero state
  const long long slot_ch = (long long)slot * p.ncb * 128;
  const __half* tq = p.kv16 + (slot_ch + kh * DK) * CH;
  const __half* tk = p.kv16 + (slot_ch + p.k_ch0 + kh * DK) * CH;
  const __half* tu = p.dump_u + ((long long)slot * p.n_v_heads + h) * DV * CH;
  const __half* ts = p.dump_s + ((long long)slot * p.n_v_heads + h) * DK * DV;
  const float* sc = p.sc + ((long long)slot * p.n_v_heads + h) * SC_FLOATS;

  for (int i = tid; i < DK * (CH / 8); i += OT) {
    const int c = i >> 3, seg = i & 7;
    cp_async16(Qs + c * LDK + seg * 8, tq + c * CH + seg * 8);
    cp_async16(Ks + c * LDK + seg * 8, tk + c * CH + seg * 8);
  }
  for (int i = tid; i < DV * (CH / 8); i += OT) {
    const int c = i >> 3, seg = i & 7;
    cp_async16(Us + c * LDK + seg * 8, tu + c * CH + seg * 8);
  }
  if (!first)
    for (int i = tid; i < DK * (DV / 8); i += OT) {
      const int r = i / (DV / 8), seg = i % (DV / 8);
      cp_async16(S0 + r * LDS + seg * 8, ts + r * DV + seg * 8);
    }
  asm volatile("cp.async.commit_group;" ::: "memory");
  if (tid < CH) {
    g[tid] = sc[128 + tid];
    ninv[tid] = sc[192 + tid];
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  // query norms: two threads per row, half of the channels each
  {
    const int i = tid & 63, half = tid >> 6;
    float ss = 0.f;
    for (int c = half * (DK / 2); c < (half + 1) * (DK / 2); ++c) {
      const float q = __half2float(Qs[c * LDK + i]);
      ss = fmaf(q, q, ss);
    }
    part[half * CH + i] = ss;
  }
  __syncthreads();
  if (tid < CH) qn[tid] = rsqrtf(part[tid] + part[CH + tid] + p.eps) * rsqrtf((float)DK);
  __syncthreads();

  const int rb = 3 - warp;
  const int i0 = rb * 16 + g8, i1 = i0 + 8;
  float acc[NT][4];
#pragma unroll
  for (int n = 0; n < NT; ++n)
#pragma unroll
    for (int c = 0; c < 4; ++c) acc[n][c] = 0.f;

  // ---- e^{g_i} (Q S_0)_i ---------------------------------------------------------------------------
  if (!first) {
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks) {
      uint32_t a[4];
      ldsm4t(a, at_addr(Qs, LDK, ks * 16, rb * 16, l));
#pragma unroll
      for (int nn = 0; nn < NT / 2; ++nn) {
        uint32_t b[4];
        ldsm4t(b, bt_addr(S0, LDS, ks * 16, nn * 16, l));
        mma16816(acc[2 * nn], a, b[0], b[1]);
        mma16816(acc[2 * nn + 1], a, b[2], b[3]);
      }
    }
    const float e0 = __expf(g[i0]), e1 = __expf(g[i1]);
#pragma unroll
    for (int n = 0; n < NT; ++n) { acc[n][0] *= e0; acc[n][1] *= e0; acc[n][2] *= e1; acc[n][3] *= e1; }
  }

  // ---- M = mask(e^{g_i - g_j} n_j (q_i . k_j)), then M U -------------------------------------------
  {
    float pr[4][2][4];
#pragma unroll
    for (int cb = 0; cb < 4; ++cb)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) pr[cb][j][c] = 0.f;
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks) {
      uint32_t a[4], b[4];
      ldsm4t(a, at_addr(Qs, LDK, ks * 16, rb * 16, l));
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        if (cb <= rb) {
          ldsm4t(b, bt_addr(Ks, LDK, ks * 16, cb * 16, l));
          mma16816(pr[cb][0], a, b[0], b[1]);
          mma16816(pr[cb][1], a, b[2], b[3]);
        }
      }
    }
    const float gi0 = g[i0], gi1 = g[i1];
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) {
      if (cb <= rb) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int c0 = cb * 16 + j * 8 + 2 * t4;
          const float2 nj = *(const float2*)(ninv + c0), gj = *(const float2*)(g + c0);
          pr[cb][j][0] = c0 <= i0 ? nj.x * __expf(gi0 - gj.x) * pr[cb][j][0] : 0.f;
          pr[cb][j][1] = c0 + 1 <= i0 ? nj.y * __expf(gi0 - gj.y) * pr[cb][j][1] : 0.f;
          pr[cb][j][2] = c0 <= i1 ? nj.x * __expf(gi1 - gj.x) * pr[cb][j][2] : 0.f;
          pr[cb][j][3] = c0 + 1 <= i1 ? nj.y * __expf(gi1 - gj.y) * pr[cb][j][3] : 0.f;
        }
        uint32_t a[4];
        pack_left(pr[cb], a);
#pragma unroll
        for (int nn = 0; nn < NT / 2; ++nn) {
          uint32_t b[4];
          ldsm4(b, bn_addr(Us, LDK, nn * 16, cb * 16, l));
          mma16816(acc[2 * nn], a, b[0], b[1]);
          mma16816(acc[2 * nn + 1], a, b[2], b[3]);
        }
      }
    }
  }

  // ---- query norm, per-head RMS norm, output gate --------------------------------------------------
  const float q0 = qn[i0], q1 = qn[i1];
  float ss0 = 0.f, ss1 = 0.f;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    acc[n][0] *= q0; acc[n][1] *= q0; acc[n][2] *= q1; acc[n][3] *= q1;
    ss0 += acc[n][0] * acc[n][0] + acc[n][1] * acc[n][1];
    ss1 += acc[n][2] * acc[n][2] + acc[n][3] * acc[n][3];
  }
  ss0 += __shfl_xor_sync(0xffffffffu, ss0, 1); ss0 += __shfl_xor_sync(0xffffffffu, ss0, 2);
  ss1 += __shfl_xor_sync(0xffffffffu, ss1, 1); ss1 += __shfl_xor_sync(0xffffffffu, ss1, 2);
  const float r0 = rsqrtf(ss0 / (float)DV + p.norm_eps), r1 = rsqrtf(ss1 / (float)DV + p.norm_eps);
  const long long ld = (long long)p.n_v_heads * DV;
  const long long row0 = ((long long)slot * CH + i0) * ld + (long long)h * DV, row1 = row0 + 8 * ld;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int c = n * 8 + 2 * t4;
    const float w0 = __bfloat162float(p.o_norm_w[c]), w1 = __bfloat162float(p.o_norm_w[c + 1]);
    const __nv_bfloat162 z0 = *(const __nv_bfloat162*)(p.zg + row0 + c), z1 = *(const __nv_bfloat162*)(p.zg + row1 + c);
    __nv_bfloat162 y0, y1;
    y0.x = __float2bfloat16_rn(i0 < vr ? acc[n][0] * r0 * w0 * __bfloat162float(z0.x) : 0.f);
    y0.y = __float2bfloat16_rn(i0 < vr ? acc[n][1] * r0 * w1 * __bfloat162float(z0.y) : 0.f);
    y1.x = __float2bfloat16_rn(i1 < vr ? acc[n][2] * r1 * w0 * __bfloat162float(z1.x) : 0.f);
    y1.y = __float2bfloat16_rn(i1 < vr ? acc[n][3] * r1 * w1 * __bfloat162float(z1.y) : 0.f);
    *(__nv_bfloat162*)(p.y + row0 + c) = y0;
    *(__nv_bfloat162*)(p.y + row1 + c) = y1;
  }
}

template <int DK, int NT>
cudaError_t launch_out(const OutParams& p, dim3 grid, cudaStream_t stream) {
  constexpr int DV = 8 * NT;
  constexpr int smem = (2 * DK * LDK + DV * LDK + DK * (DV + 8)) * 2 + 5 * CH * 4;
  cudaError_t e = cudaFuncSetAttribute(sr_group_output_kernel<DK, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;           // per launch: cheap next to the call, and right on every device
  sr_group_output_kernel<DK, NT><<<grid, OT, smem, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace

bool sr_group_output_supported(int d_k, int d_v) {
  return (d_k == 64 && d_v == 64) || (d_k == 128 && d_v == 128);
}

cudaError_t sr_launch_group_output(const sr_ctx* ctx, const SrSched& s, const SrFused& fused, const void* split_buf,
                                   const __nv_bfloat16* zg, const __nv_bfloat16* o_norm_w, float norm_eps, __nv_bfloat16* y,
                                   cudaStream_t stream) {
  const sr_model_desc& d = ctx->desc;
  OutParams p;
  p.s = s;
  p.kv16 = fused.kv16;
  p.dump_s = fused.dump_s;
  p.dump_u = fused.dump_u;
  p.sc = (const float*)((const char*)split_buf + (size_t)s.max_slots * d.n_v_heads * (2 * CH * CH) * sizeof(__half));
  p.zg = zg;
  p.o_norm_w = o_norm_w;
  p.y = y;
  p.ncb = fused.ncb;
  p.k_ch0 = fused.k_ch0;
  p.n_k_heads = d.n_k_heads;
  p.n_v_heads = d.n_v_heads;
  p.d_v = d.d_v;
  p.eps = d.l2_eps;
  p.norm_eps = norm_eps;
  dim3 grid((unsigned)d.n_v_heads, (unsigned)s.max_slots);
  if (d.d_k == 64 && d.d_v == 64) return launch_out<64, 8>(p, grid, stream);
  if (d.d_k == 128 && d.d_v == 128) return launch_out<128, 16>(p, grid, stream);
  return cudaErrorInvalidValue;
}
