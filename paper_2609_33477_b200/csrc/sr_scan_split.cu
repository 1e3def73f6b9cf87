// The chunked gated-delta scan (Eq. 4, 64 rows at a time) split in two kernels; this file holds the first.
//
// With g_i the running sum of log alpha inside a chunk, gamma_i = exp(g_i), n_i = 1/sqrt(|k_i|^2 + eps):
//
//   A_ij = beta_i exp(g_i - g_j) n_i n_j (k_i . k_j)  (j < i),   T = (I + A)^-1
//   U~ = T diag(beta) V,  W = T diag(beta gamma n) K,  U = U~ - W S0,
//   S  = gamma_n S0 + K^T diag(exp(g_n - g_j) n_j) U
//
// Only the last two lines involve the state.  Everything before them -- gates, K K^T (whose diagonal
// gives the key norms), A and its inverse -- is local to a chunk, so it is computed for ALL chunks of
// the batch at once by sr_chunk_local_kernel: one CTA per (value head, page slot), thousands of them,
// no serial chain, latency hidden by occupancy.  It leaves T diag(beta), T diag(beta gamma n) (fp16, stored
// transposed: [column][row]) and
// the row factors exp(g_n - g_j) n_j, gamma_n per chunk, and finishes the first three conv rows of chunks
// whose conv history the projection could not see.  The state chain (sr_scan_chain_umma.cu) then walks each
// (head, request) chain.
//
// Products here run on mma.sync m16n8k16, fp16 operands (the 11 significant bits of tf32; bf16's 8 would
// miss the 2e-3 state tolerance), fp32 accumulation.  Row scalings are folded into T's columns and U's
// rows in fp32 before the single rounding to fp16, so k and v are rounded exactly once.
#include "sr_mma.cuh"

namespace {

constexpr int CH = 64;            // chunk rows (= page rows)
constexpr int LDT = CH + 8;       // pitch (halfs) of 64 x 64 fp16 tiles
constexpr int LDK = CH + 8;       // pitch (halfs) of channel-major [d_k][64] key tiles
constexpr int TT_HALFS = 2 * CH * CH;   // per chunk and head: T diag(beta), then T diag(beta gamma n)
constexpr int SC_FLOATS = 256;          // per chunk and head: 64 row factors, gamma_n, padding | 64 running log-decays g_i |
                                        // 64 inverse key norms

// ---------------------------------------------------------------------------------------------------
// chunk-local part

constexpr int LT = 128;           // threads of the chunk-local kernel: small CTAs, many per SM
#ifndef LOCAL_CTAS_PER_SM
#define LOCAL_CTAS_PER_SM 10
#endif

constexpr int LDI = 24;           // pitch (halfs) of the fp16 inverses of the diagonal blocks

template <int DK>
struct LocalSmem {
  union {                         // the key tile is dead once K K^T sits in registers: A takes its place
    __half Ks[DK * LDK];          // keys of the chunk, channel-major
    struct {
      __half A16[CH * LDT];       // A below the block diagonal, fp16 (operand of the block products)
      __half Dinv[4 * 16 * LDI];  // their inverses (I + A_bb)^-1, fp16, row-major
    };
  };
  float g[CH];                    // inclusive running sum of log alpha
  float beta[CH];
  float ninv[CH];
  float colw[CH];                 // beta_j gamma_j n_j
  float Gs[2 * CH];               // gate pre-activations a[0..63], b[0..63]
};

struct LocalParams {
  SrSched s;
  const float* gates;             // [slot][2 H_v][64]
  __half* kv16;                   // [slot][ncb * 128 channels][64]; rows 0..2 are completed here where needed
  const float* zraw;              // [slot][6][n_kv]
  int32_t ncb, n_kv, fix_mod;
  int32_t n_k_heads, n_v_heads;
  int32_t d_v;                    // value head width (the key head width is the template parameter)
  int32_t with_q, k_ch0, v_ch0;   // tile contents (see SrFused); conv channel of projected channel c = conv_ch0 + c
  int32_t conv_ch0;
  int32_t act_identity;
  int32_t erase;                  // 0: decay-only family, A = 0 and T = I
  float eps;
  const __nv_bfloat16* conv_w;
  const float* decay_scale;
  const float* dt_bias;
  __half* tt;                     // [slot][H_v][2][64][64]
  float* sc;                      // [slot][H_v][SC_FLOATS]
};

// A 16 x 16 matrix held by a warp in the accumulator layout of m16n8k16 (x[j][0..1]: row g8, columns 8 j + 2 t4, +1;
// x[j][2..3]: row g8 + 8) as the left operand of a product: pack pairs to fp16, nothing moves between lanes.
__device__ __forceinline__ void pack_left(const float (&x)[2][4], uint32_t (&a)[4]) {
  a[0] = pack_h2(x[0][0], x[0][1]);
  a[1] = pack_h2(x[0][2], x[0][3]);
  a[2] = pack_h2(x[1][0], x[1][1]);
  a[3] = pack_h2(x[1][2], x[1][3]);
}
// transpose of an 8 x 8 fp16 matrix held one packed row-pair per lane
__device__ __forceinline__ uint32_t movm_trans(uint32_t v) {
  uint32_t r;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(r) : "r"(v));
  return r;
}
// the same matrix as the right operand: b[j][0..1] are the two k halves of the operand for output columns 8 j ..
__device__ __forceinline__ void pack_right(const float (&x)[2][4], uint32_t (&b)[2][2]) {
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    b[j][0] = movm_trans(pack_h2(x[j][0], x[j][1]));
    b[j][1] = movm_trans(pack_h2(x[j][2], x[j][3]));
  }
}

template <int DK>
__global__ void __launch_bounds__(LT, LOCAL_CTAS_PER_SM) sr_chunk_local_kernel(const LocalParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  LocalSmem<DK>& sm = *reinterpret_cast<LocalSmem<DK>*>(smem_raw);
  const int h = blockIdx.x, slot = blockIdx.y;
  if (slot >= (int)p.s.status[1] || !sr_check_slot(p.s, slot)) return;
  const int vr = p.s.slot_rows[slot];
  if (vr == 0) return;                                   // padding slot
  const int tid = threadIdx.x, warp = tid >> 5, l = tid & 31, g8 = l >> 2, t4 = l & 3;
  const int kh = h / (p.n_v_heads / p.n_k_heads);
  const int n_k = p.n_k_heads * DK, dv = p.d_v;
  const bool fix = !p.s.slot_first[slot] && (slot % p.fix_mod) == 0;
  const long long slot_ch = (long long)slot * p.ncb * 128;        // first channel row of this slot's tiles
  __half* tk = p.kv16 + (slot_ch + p.k_ch0 + kh * DK) * CH;
  __half* tv = p.kv16 + (slot_ch + p.v_ch0 + h * dv) * CH;
  __half* tq = p.kv16 + (slot_ch + kh * DK) * CH;                  // with_q only: the key head's query channels
  const int qn = p.with_q ? DK : 0;                                // fix-up channels: [q |] k | v of this head

  // ---- fetch: the key tile and the two gate rows of this head ----
  for (int i = tid; i < DK * (CH / 8); i += LT) {
    const int c = i >> 3, seg = i & 7;
    cp_async16(sm.Ks + c * LDK + seg * 8, tk + c * CH + seg * 8);
  }
  if (tid < 2 * (CH / 4)) {
    const int which = tid >> 4, seg = tid & 15;
    cp_async16(sm.Gs + which * CH + seg * 4,
               p.gates + ((long long)slot * (2 * p.n_v_heads) + (which ? p.n_v_heads + h : h)) * CH + seg * 4);
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  // where a fix-up is due: the previous slot's last three raw rows and this slot's rows 0..2 of this thread's
  // channels (the head's d_k key channels, then its d_v value channels), fetched while the key tile is in flight
  constexpr int FIXQ = 4;         // channels per thread: (d_k +) d_k + d_v <= 4 * 128
  float zr[FIXQ][6];
  // channel c of the head's run -> its index among the projected channels
  auto run_channel = [&](int c) { return c < qn ? kh * DK + c : (c < qn + DK ? p.k_ch0 + kh * DK + (c - qn) : p.v_ch0 + h * dv + (c - qn - DK)); };
  if (fix) {
#pragma unroll
    for (int q = 0; q < FIXQ; ++q) {
      const int c = tid + q * LT;
      if (c < qn + DK + dv) {
        const int zc = run_channel(c);
#pragma unroll
        for (int rr = 0; rr < 6; ++rr)
          zr[q][rr] = __ldg(p.zraw + ((long long)(rr < 3 ? slot - 1 : slot) * 6 + (rr < 3 ? 3 + rr : rr - 3)) * p.n_kv + zc);
      }
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  if (fix) {
    // rows 0..2: conv over the raw rows, SiLU, fp16; written back to the tiles for the chain kernel (heads
    // sharing a key head write identical key values)
#pragma unroll
    for (int q = 0; q < FIXQ; ++q) {
      const int c = tid + q * LT;
      if (c < qn + DK + dv) {
        const int zc = run_channel(c);
        const uint2 wv = *(const uint2*)(p.conv_w + (long long)(p.conv_ch0 + zc) * SR_CONV_W);
        const __nv_bfloat16* e = (const __nv_bfloat16*)&wv;
        const float w0 = __bfloat162float(e[0]), w1 = __bfloat162float(e[1]), w2 = __bfloat162float(e[2]),
                    w3 = __bfloat162float(e[3]);
        __half* gdst = c < qn ? tq + c * CH : (c < qn + DK ? tk + (c - qn) * CH : tv + (c - qn - DK) * CH);
#pragma unroll
        for (int rho = 0; rho < 3; ++rho) {
          float y = w0 * zr[q][rho] + w1 * zr[q][rho + 1] + w2 * zr[q][rho + 2] + w3 * zr[q][rho + 3];
          if (!p.act_identity) y = __fdividef(y, 1.f + __expf(-y));
          const __half hy = __float2half_rn(y);
          gdst[rho] = hy;
          if (c >= qn && c < qn + DK) sm.Ks[(c - qn) * LDK + rho] = hy;
        }
      }
    }
    __syncthreads();
  }
  // Row block rb of the chunk belongs to warp 3 - rb: the warp with the lightest K K^T share (rb = 0) also
  // computes the gates, the one with the heaviest has nothing to do in the last phase.
  const int rb = 3 - warp;
  // ---- gates: one warp, two rows per lane, warp prefix sum of log alpha ----------------------------
  if (warp == 3) {
    const float c_h = p.decay_scale[h], delta_h = p.dt_bias[h];
    float la[2], be[2];
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      la[q] = 0.f;
      be[q] = 0.f;
      if (2 * l + q < vr) {                              // rows past the request's end: alpha = 1, beta = 0
        const float a = sm.Gs[2 * l + q] + delta_h;
        la[q] = -c_h * (fmaxf(a, 0.f) + log1pf(expf(-fabsf(a))));
        be[q] = 1.f / (1.f + expf(-sm.Gs[CH + 2 * l + q]));
      }
    }
    float run = la[0] + la[1];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float v = __shfl_up_sync(0xffffffffu, run, off);
      if (l >= off) run += v;
    }
    sm.g[2 * l] = run - la[1];
    sm.g[2 * l + 1] = run;
    sm.beta[2 * l] = be[0];
    sm.beta[2 * l + 1] = be[1];
  }

  // ---- raw = K K^T, 16 x 16 blocks at or below the block diagonal ------------------------------------
  float nd[2][4];               // -A on this warp's diagonal block, accumulator layout (zero on and above the diagonal)
  {
    float acc[4][2][4];
#pragma unroll
    for (int cb = 0; cb < 4; ++cb)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[cb][j][c] = 0.f;
#pragma unroll
    for (int ks = 0; ks < DK / 16; ++ks) {
      uint32_t a[4], b[4];
      ldsm4t(a, at_addr(sm.Ks, LDK, ks * 16, rb * 16, l));
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) {
        if (cb <= rb) {
          ldsm4t(b, bt_addr(sm.Ks, LDK, ks * 16, cb * 16, l));
          mma16816(acc[cb][0], a, b[0], b[1]);
          mma16816(acc[cb][1], a, b[2], b[3]);
        }
      }
    }
    // the diagonal of K K^T is |k_i|^2: every thread that holds a diagonal entry publishes the key norm
#pragma unroll
    for (int cb = 0; cb < 4; ++cb)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const int row = g8 + (c >> 1) * 8, col = j * 8 + 2 * t4 + (c & 1);
          if (cb == rb && row == col) sm.ninv[rb * 16 + row] = rsqrtf(acc[cb][j][c] + p.eps);
        }
    __syncthreads();            // norms and gates visible; every warp has read its keys: the tile's memory becomes A
    // A_ij = beta_i n_i n_j exp(g_i - g_j) raw_ij (j < i), written straight from the accumulators: blocks
    // below the block diagonal go to shared memory as fp16, the diagonal block stays in registers
    const int i0 = rb * 16 + g8, i1 = i0 + 8;
    const float on = p.erase ? 1.f : 0.f;         // without the erase A vanishes: T = I, W is not used
    const float f0 = on * sm.beta[i0] * sm.ninv[i0], f1 = on * sm.beta[i1] * sm.ninv[i1];
    const float gi0 = sm.g[i0], gi1 = sm.g[i1];
#pragma unroll
    for (int cb = 0; cb < 4; ++cb) {
      if (cb <= rb) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int c0 = cb * 16 + j * 8 + 2 * t4;
          const float2 nj = *(const float2*)(sm.ninv + c0), gj = *(const float2*)(sm.g + c0);
          float2 lo, hi;
          lo.x = c0 < i0 ? f0 * nj.x * __expf(gi0 - gj.x) * acc[cb][j][0] : 0.f;
          lo.y = c0 + 1 < i0 ? f0 * nj.y * __expf(gi0 - gj.y) * acc[cb][j][1] : 0.f;
          hi.x = c0 < i1 ? f1 * nj.x * __expf(gi1 - gj.x) * acc[cb][j][2] : 0.f;
          hi.y = c0 + 1 < i1 ? f1 * nj.y * __expf(gi1 - gj.y) * acc[cb][j][3] : 0.f;
          if (cb < rb) {
            *(uint32_t*)(sm.A16 + i0 * LDT + c0) = pack_h2(lo.x, lo.y);
            *(uint32_t*)(sm.A16 + i1 * LDT + c0) = pack_h2(hi.x, hi.y);
          } else {
            nd[j][0] = -lo.x; nd[j][1] = -lo.y; nd[j][2] = -hi.x; nd[j][3] = -hi.y;
          }
        }
      }
    }
  }

  // T = (I + A)^-1 is written out transposed and scaled by column: tt[0][c][i] = T_ic beta_c,
  // tt[1][c][i] = T_ic beta_c gamma_c n_c (fp16).
  __half* tt = p.tt + ((long long)slot * p.n_v_heads + h) * TT_HALFS;

  // ---- the 16 x 16 diagonal block of this warp's rows.  N = -A_bb is nilpotent (N^16 = 0), so
  //      (I - N)^-1 = (I + N)(I + N^2)(I + N^4)(I + N^8): three squarings and three products of 16 x 16 matrices
  //      on mma.sync, operands rounded to fp16, sums kept in fp32.  I + N is exact; the rounded operands only
  //      enter terms of second order in A, so the result is within 1e-4 of the exact inverse -- below the
  //      fp16 rounding of the output.  Everything stays in registers in the accumulator layout; a matrix
  //      becomes a left operand by packing, a right operand by packing and an 8 x 8 transpose (movmatrix).
  {
    float P[2][4], s2[2][4], s4[2][4], s8[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int row = g8 + (c >> 1) * 8, col = j * 8 + 2 * t4 + (c & 1);
        P[j][c] = nd[j][c] + (row == col ? 1.f : 0.f);
        s2[j][c] = 0.f; s4[j][c] = 0.f; s8[j][c] = 0.f;
      }
    uint32_t xa[4], xb[2][2];
    pack_left(nd, xa);
    pack_right(nd, xb);
    mma16816(s2[0], xa, xb[0][0], xb[0][1]);            // N^2
    mma16816(s2[1], xa, xb[1][0], xb[1][1]);
    pack_left(P, xa);
    pack_right(s2, xb);
    mma16816(P[0], xa, xb[0][0], xb[0][1]);             // (I + N)(I + N^2)
    mma16816(P[1], xa, xb[1][0], xb[1][1]);
    pack_left(s2, xa);
    mma16816(s4[0], xa, xb[0][0], xb[0][1]);            // N^4
    mma16816(s4[1], xa, xb[1][0], xb[1][1]);
    pack_left(P, xa);
    pack_right(s4, xb);
    mma16816(P[0], xa, xb[0][0], xb[0][1]);             // ... (I + N^4)
    mma16816(P[1], xa, xb[1][0], xb[1][1]);
    pack_left(s4, xa);
    mma16816(s8[0], xa, xb[0][0], xb[0][1]);            // N^8
    mma16816(s8[1], xa, xb[1][0], xb[1][1]);
    pack_left(P, xa);
    pack_right(s8, xb);
    mma16816(P[0], xa, xb[0][0], xb[0][1]);             // ... (I + N^8) = (I + A_bb)^-1
    mma16816(P[1], xa, xb[1][0], xb[1][1]);

    // the inverse as fp16, row-major, for the block-column chains below
    __half* di = sm.Dinv + (rb * 16) * LDI;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      *(uint32_t*)(di + g8 * LDI + j * 8 + 2 * t4) = pack_h2(P[j][0], P[j][1]);
      *(uint32_t*)(di + (g8 + 8) * LDI + j * 8 + 2 * t4) = pack_h2(P[j][2], P[j][3]);
    }
    if (l < 16) {                                       // column factor of T diag(beta gamma n)
      const int col = 16 * rb + l;
      sm.colw[col] = sm.beta[col] * __expf(sm.g[col]) * sm.ninv[col];
    }
    __syncwarp();
    // transposed output of the diagonal block: scale by column, pack, transpose 8 x 8 pieces, 4-byte stores
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int c0 = 16 * rb + j * 8 + 2 * t4;          // this thread's two columns of T in piece j
      const float b0 = sm.beta[c0], b1 = sm.beta[c0 + 1], w0 = sm.colw[c0], w1 = sm.colw[c0 + 1];
#pragma unroll
      for (int rh = 0; rh < 2; ++rh) {
        const uint32_t tb = movm_trans(pack_h2(P[j][2 * rh] * b0, P[j][2 * rh + 1] * b1));
        const uint32_t tw = movm_trans(pack_h2(P[j][2 * rh] * w0, P[j][2 * rh + 1] * w1));
        // now: row (16 rb + 8 j + g8) of the transposed matrix, entries i = 16 rb + 8 rh + 2 t4, + 1
        __half* dst = tt + (16 * rb + 8 * j + g8) * CH + 16 * rb + 8 * rh + 2 * t4;
        *(uint32_t*)dst = tb;
        *(uint32_t*)(dst + CH * CH) = tw;
      }
    }
    // zeros left of the diagonal block: rows 16 rb .. + 15, entries 0 .. 16 rb - 1
    {
      __half* row = tt + (16 * rb + (l & 15)) * CH;
      for (int q = l >> 4; q < 2 * rb; q += 2) {
        *(uint4*)(row + 8 * q) = make_uint4(0u, 0u, 0u, 0u);
        *(uint4*)(row + CH * CH + 8 * q) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
  }
  __syncthreads();

  // ---- below the diagonal: warp J owns block column J, no further synchronisation.  With X_K = T_KJ:
  //      X_J = D_J,  X_I = -D_I sum_{K=J}^{I-1} A_IK X_K  (I > J).  Computed transposed, so that every X_K^T
  //      stays in registers as an A operand: X_I^T = -(sum_K X_K^T A_IK^T) D_I^T.
  if (rb < 3) {
    const int J = rb;
    uint32_t xa[4][4], xj[4];
    ldsm4t(xj, at_addr(sm.Dinv + (J * 16) * LDI, LDI, 0, 0, l));
#pragma unroll
    for (int K = 0; K < 3; ++K)                       // compile-time indices keep the fragments in registers
#pragma unroll
      for (int q = 0; q < 4; ++q) xa[K][q] = (K == J) ? xj[q] : 0u;
    const int c0 = 16 * J + g8, c1 = c0 + 8;
    const float b0 = sm.beta[c0], b1 = sm.beta[c1], w0 = sm.colw[c0], w1 = sm.colw[c1];
#pragma unroll
    for (int I = 1; I < 4; ++I) {
      if (I > J) {
        float y[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int c = 0; c < 4; ++c) y[j][c] = 0.f;
#pragma unroll
        for (int K = 0; K < 3; ++K) {
          if (K >= J && K < I) {
            uint32_t bf[4];
            ldsm4(bf, bn_addr(sm.A16, LDT, 16 * I, 16 * K, l));
            mma16816(y[0], xa[K], bf[0], bf[1]);
            mma16816(y[1], xa[K], bf[2], bf[3]);
          }
        }
        const uint32_t ya[4] = {pack_h2(y[0][0], y[0][1]), pack_h2(y[0][2], y[0][3]), pack_h2(y[1][0], y[1][1]),
                                pack_h2(y[1][2], y[1][3])};
        uint32_t bf[4];
        ldsm4(bf, bn_addr(sm.Dinv + (I * 16) * LDI, LDI, 0, 0, l));
        float z[2][4];
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int c = 0; c < 4; ++c) z[j][c] = 0.f;
        mma16816(z[0], ya, bf[0], bf[1]);
        mma16816(z[1], ya, bf[2], bf[3]);
        xa[I][0] = pack_h2(-z[0][0], -z[0][1]);
        xa[I][1] = pack_h2(-z[0][2], -z[0][3]);
        xa[I][2] = pack_h2(-z[1][0], -z[1][1]);
        xa[I][3] = pack_h2(-z[1][2], -z[1][3]);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          __half* d0 = tt + c0 * CH + 16 * I + 8 * j + 2 * t4;
          __half* d1 = tt + c1 * CH + 16 * I + 8 * j + 2 * t4;
          *(uint32_t*)d0 = pack_h2(-z[j][0] * b0, -z[j][1] * b0);
          *(uint32_t*)d1 = pack_h2(-z[j][2] * b1, -z[j][3] * b1);
          *(uint32_t*)(d0 + CH * CH) = pack_h2(-z[j][0] * w0, -z[j][1] * w0);
          *(uint32_t*)(d1 + CH * CH) = pack_h2(-z[j][2] * w1, -z[j][3] * w1);
        }
      }
    }
  }
  if (tid < CH + 1) {
    const float g_last = sm.g[CH - 1];
    float* sc = p.sc + ((long long)slot * p.n_v_heads + h) * SC_FLOATS;
    sc[tid] = tid < CH ? __expf(g_last - sm.g[tid]) * sm.ninv[tid] : __expf(g_last);
    if (tid < CH) {                 // for the output kernel of group replay
      sc[128 + tid] = sm.g[tid];
      sc[192 + tid] = sm.ninv[tid];
    }
  }
}

}  // namespace

size_t sr_scan_split_bytes(const sr_ctx* ctx, int64_t max_slots) {
  return (size_t)max_slots * ctx->desc.n_v_heads * (TT_HALFS * sizeof(__half) + SC_FLOATS * sizeof(float));
}

bool sr_chunk_local_supported(int d_k, int d_v) {
  return (d_k == 64 || d_k == 96 || d_k == 128) && d_v % 8 == 0 && d_v > 0 && 2 * d_k + d_v <= 4 * LT;
}

template <int DK>
static cudaError_t launch_chunk_local(const LocalParams& p, dim3 grid, cudaStream_t stream) {
  cudaError_t e = sr_once_per_device(DK == 64 ? SR_ONCE_CHUNK_LOCAL_64 : DK == 96 ? SR_ONCE_CHUNK_LOCAL_96 : SR_ONCE_CHUNK_LOCAL_128, [] {
    return cudaFuncSetAttribute(sr_chunk_local_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)sizeof(LocalSmem<DK>));
  });
  if (e != cudaSuccess) return e;
  sr_chunk_local_kernel<DK><<<grid, LT, sizeof(LocalSmem<DK>), stream>>>(p);
  return cudaGetLastError();
}

cudaError_t sr_launch_chunk_local(const sr_ctx* ctx, const SrSched& s, const sr_layer_weights& w, const SrFused& fused,
                                  void* split_buf, cudaStream_t stream) {
  const sr_model_desc& d = ctx->desc;
  LocalParams p;
  p.s = s;
  p.gates = fused.gates;
  p.kv16 = fused.kv16;
  p.zraw = fused.zraw;
  p.ncb = fused.ncb;
  p.n_kv = fused.n_kv;
  p.fix_mod = fused.fix_mod;
  p.n_k_heads = d.n_k_heads;
  p.n_v_heads = d.n_v_heads;
  p.d_v = d.d_v;
  p.with_q = fused.with_q;
  p.k_ch0 = fused.k_ch0;
  p.v_ch0 = fused.v_ch0;
  p.conv_ch0 = fused.with_q ? 0 : ctx->n_k;
  p.act_identity = d.conv_activation == SR_CONV_IDENTITY;
  p.erase = d.recurrence == SR_REC_GATED_DELTA;
  p.eps = d.l2_eps;
  p.conv_w = (const __nv_bfloat16*)w.conv_w;
  p.decay_scale = w.decay_scale;
  p.dt_bias = w.dt_bias;
  p.tt = (__half*)split_buf;
  p.sc = (float*)((char*)split_buf + (size_t)s.max_slots * d.n_v_heads * TT_HALFS * sizeof(__half));
  dim3 grid((unsigned)d.n_v_heads, (unsigned)s.max_slots);
  switch (d.d_k) {
    case 64: return launch_chunk_local<64>(p, grid, stream);
    case 96: return launch_chunk_local<96>(p, grid, stream);
    case 128: return launch_chunk_local<128>(p, grid, stream);
    default: return cudaErrorInvalidValue;
  }
}
