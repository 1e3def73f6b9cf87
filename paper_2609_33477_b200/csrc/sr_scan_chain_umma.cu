// The state chain of the chunked gated-delta scan (Eq. 4, 64 rows at a time) on tcgen05 tensor cores,
// with the state in tensor memory.
//
// Per chunk, given by the chunk-local kernel: Tb = T diag(beta), Tw = T diag(beta gamma n) (fp16, 64 x 64,
// stored transposed),
// the row factors f_j = exp(g_n - g_j) n_j and gamma_n; given by the projection: the fp16 key and value
// tiles, channel-major ([128 channels][64 rows]).  With S (d_k x d_v) the state entering the chunk:
//
//   W^T  = K^T Tw^T            (d_k x 64)     U~^T = V^T Tb^T            (d_v x 64)
//   U^T  = U~^T - S^T W^T      (d_v x 64)
//   S    = gamma_n S + K^T diag(f) U          (d_k x d_v)
//
// All four products are issued with M = 128: the transposed forms put the 128-wide head dimension on the
// MMA's M axis, so no 64-row MMA shape is needed.  Operand layouts (all 128-byte swizzled, rows of 64 fp16):
//   K^T, V^T   as loaded: [128][64], K-major A operands (K = chunk rows)
//   Tw, Tb     stored transposed, [64 columns][64 rows]: MN-major B operands
//   -W^T       written by the threads from tensor memory as [d_k][64]: an MN-major B operand of S^T W^T
//   S (fp16)   written by the threads as [d_k][d_v] in two 64-column halves: an MN-major A operand
//   (f U)^T    written by the threads as [d_v][64]: a K-major B operand of the state update
// Head widths other than 128: every product keeps M = 128.  Tiles are fetched 128 channels tall whatever d_k and
// d_v are, so lanes past a head's own channels hold its neighbours' channels (or stale scratch): their results
// are never read -- the one contraction over the key index, S^T W^T, runs over d_k only, value columns never mix
// (Eq. 5: the state is linear in the values, column by column), and only rows < d_k, columns < d_v are stored.
// A value head wider than 128 is split into equal column blocks of at most 128, one CTA each; narrower heads
// may be split too, to put more CTAs on a small batch.
// Tensor memory (256 columns per CTA, two CTAs per SM): S fp32 (lanes d_k, 128 columns), U^T (lanes d_v,
// 64 columns), W^T (lanes d_k, 64 columns).  Eight warps move data between tensor memory and shared memory
// (warp w works on lanes 32 (w % 4) .. and on one half of the columns); a ninth warp's first lane issues the
// TMA loads and the MMAs.  The decay gamma_n S is applied in the same pass that writes the fp16 copy of S.
// W^T and U~^T do not depend on the state: they are issued one chunk ahead (behind the previous chunk's state
// update, as soon as tensor memory for them is drained), and the key tiles are double-buffered so that loads
// run two chunks ahead.  On the serial chain remain: drain S and W^T, S^T W^T, drain U^T, the state update.
// For group-propagated replay (Section 4.1) the passes that drain S and U^T also leave the fp16 state ENTERING
// every chunk and the chunk's U^T (before the row factors) in memory: the output kernel forms the layer's per-token
// outputs from them.
// Every mbarrier wait is bounded; on expiry the kernel raises SR_DEV_WAIT_EXPIRED, stops issuing work,
// frees its tensor memory and returns.
#include "sr_umma.cuh"

namespace {

constexpr int CH = 64;
constexpr int D = 128;                   // tile height and MMA M: head widths up to 128 per CTA
constexpr int TT_HALFS = 2 * CH * CH;
constexpr int SC_FLOATS = 256;
constexpr int COMPUTE_THREADS = 256;
constexpr int THREADS = COMPUTE_THREADS + 32;
constexpr int TILE_KV = D * CH * 2;      // 16 KB: [128][64] fp16
constexpr int TILE_T = CH * CH * 2;      // 8 KB: [64][64] fp16
constexpr int SC_BYTES = 272;            // 64 row factors + gamma_n, rounded up to 16 bytes

constexpr int SC_STRIDE = 80;            // floats between the two row-factor buffers (320 bytes)

// 112 KB of tiles + 1 KB: two CTAs per SM fit only without alignment slack, so the kernel relies on the
// dynamic shared memory window starting on a 1024-byte boundary (checked at run time).
struct Smem {
  uint8_t KT[2][TILE_KV];    // key tiles of two consecutive chunks
  uint8_t VT[TILE_KV];
  uint8_t Tb[TILE_T];
  uint8_t Tw[TILE_T];
  uint8_t WU[TILE_KV];       // -W^T, later (f U)^T
  uint8_t S16[2 * TILE_KV];  // fp16 state: columns 0..63, then columns 64..127
  float sc[2][SC_STRIDE];
  uint64_t bar_k[2], bar_v[2], bar_m1[2], bar_m2[2], bar_m3[2];
  uint32_t tmem_slot;
  int abort_flag;
};

struct ChainUmmaParams {
  SrSched s;
  const float* sc;
  int32_t ncb;
  int32_t n_k_heads, n_v_heads;
  int32_t d_k, d_v;          // head widths
  int32_t dvb;               // value columns per CTA (d_v / gridDim.z, a multiple of 4, at most 128)
  char* out_layer;
  int64_t slot_stride;
  int32_t erase;             // 0: decay-only family, U = U~ (no W S term)
  const char* in_layer;      // states to continue from (same slot addressing as the output), or null = zero
  int64_t in_slot_stride;
  int32_t k_ch0, v_ch0;      // first key / value channel inside a slot's tiles
  __half* dump_s;            // group replay: [slot][H_v][d_k][d_v] state entering each chunk (fp16), or null
  __half* dump_u;            // group replay: [slot][H_v][d_v][64] pseudo-values of each chunk (fp16), or null
  long long wait_limit;      // cycles a wait may take before it gives up
  int32_t withhold_first_keys;   // fault injection (SR_DEBUG_EXPIRE_WAIT): chunk 0's key tile is never requested, so
                                 // the waits on it run out
};

// instruction descriptor: D fp32, A and B fp16, M x N, operand majors (0 = K-major, 1 = MN-major)
__host__ __device__ constexpr uint32_t idesc_f16(int m, int n, int a_mn, int b_mn) {
  return (1u << 4) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
// shared-memory matrix descriptor, 128-byte swizzle: byte offsets between 8-row groups (sbo) and, for
// MN-major operands wider than 64 elements, between 64-element column blocks (lbo)
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
// 32 consecutive fp16 values (columns c0 .. c0+31, c0 a multiple of 32) of row r of a [rows][64] swizzled tile
__device__ __forceinline__ void store_row32(uint8_t* tile, int r, int c0, const float* v) {
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int chunk = (c0 >> 3) + q;
    uint4 u = make_uint4(pack_h2(v[8 * q], v[8 * q + 1]), pack_h2(v[8 * q + 2], v[8 * q + 3]),
                         pack_h2(v[8 * q + 4], v[8 * q + 5]), pack_h2(v[8 * q + 6], v[8 * q + 7]));
    *(uint4*)(tile + r * 128 + ((chunk ^ (r & 7)) << 4)) = u;
  }
}

__global__ void __launch_bounds__(THREADS, 2)
sr_scan_chain_umma_kernel(const __grid_constant__ CUtensorMap map_kv, const __grid_constant__ CUtensorMap map_tt,
                          const ChainUmmaParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
  const int h = blockIdx.x, req = p.s.req_order[blockIdx.y];       // longest chains first
  if (!sr_check(p.s, req >= 0 && req < p.s.n_requests)) return;
  const int out_slot = p.s.req_out[req];
  if (out_slot < 0) return;
  const int R = p.s.req_rows[req];
  if (!sr_check_out(p.s, out_slot) || (R > 0 && !sr_check_slot(p.s, p.s.req_slot0[req] + (R - 1) / CH))) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int dk = p.d_k, dv = p.d_v, dvb = p.dvb, col0 = (int)blockIdx.z * dvb;     // this CTA: value columns col0 .. col0 + dvb
  const int64_t head_off = (int64_t)h * dk * dv + col0;
  float* out = (float*)(p.out_layer + (int64_t)out_slot * p.slot_stride) + head_off;
  const int kh = h / (p.n_v_heads / p.n_k_heads);
  const int slot0 = p.s.req_slot0[req];
  const int n_chunks = (R + CH - 1) / CH;
  const float* init = p.in_layer ? (const float*)(p.in_layer + (int64_t)out_slot * p.in_slot_stride) + head_off : nullptr;
  const bool has_init = init != nullptr;
  const bool erase = p.erase != 0;
  if (n_chunks == 0) {                 // nothing to replay: the state is handed through (or zero)
    if (init != out) {
      const int q4 = dvb / 4;          // float4 pieces per row of this CTA's block
      for (int i = tid; i < dk * q4; i += THREADS) {
        const int64_t at = (int64_t)(i / q4) * dv + (i % q4) * 4;
        *(float4*)(out + at) = has_init ? *(const float4*)(init + at) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    return;
  }
  if ((smem_u32(smem_raw) & 1023u) != 0) {          // swizzled tiles need 1024-byte alignment
    if (tid == 0) atomicOr(p.s.status, SR_DEV_WAIT_EXPIRED);
    return;
  }
  volatile int* abort_flag = &sm.abort_flag;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm.bar_k[i], 1); mbar_init(&sm.bar_v[i], 1);
      mbar_init(&sm.bar_m1[i], 1); mbar_init(&sm.bar_m2[i], 1); mbar_init(&sm.bar_m3[i], 1);
    }
    sm.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 8) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_slot)), "r"(256));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = sm.tmem_slot;
  const uint32_t tm_S = tmem_base, tm_U = tmem_base + 128, tm_W = tmem_base + 192;

  // tile rows in the tensor maps: channel c of slot s is row s * (ncb * 128) + c (keys of key head a from
  // a * d_k, values of value head h from H_k d_k + h * d_v), 128 rows fetched whatever the head width;
  // T matrices of (slot, head) start at row (slot*H_v + head)*128 (Tb), +64 (Tw)
  const int k_row = p.k_ch0 + kh * dk, v_row = p.v_ch0 + h * dv + col0, slot_rows = p.ncb * D;
  auto load_v = [&](int ck) {          // V^T, Tb, Tw of chunk ck (one buffer)
    const int slot = slot0 + ck;
    uint64_t* bar = &sm.bar_v[ck & 1];
    mbar_expect_tx(bar, TILE_KV + 2 * TILE_T);
    tma_load_2d(sm.VT, &map_kv, bar, 0, slot * slot_rows + v_row);
    tma_load_2d(sm.Tb, &map_tt, bar, 0, (slot * p.n_v_heads + h) * 2 * CH);
    tma_load_2d(sm.Tw, &map_tt, bar, 0, (slot * p.n_v_heads + h) * 2 * CH + CH);
  };
  auto load_k = [&](int ck) {          // K^T and the row factors of chunk ck (buffer ck & 1)
    const int slot = slot0 + ck;
    uint64_t* bar = &sm.bar_k[ck & 1];
    mbar_expect_tx(bar, TILE_KV + SC_BYTES);
    tma_load_2d(sm.KT[ck & 1], &map_kv, bar, 0, slot * slot_rows + k_row);
    bulk_load(sm.sc[ck & 1], p.sc + ((long long)slot * p.n_v_heads + h) * SC_FLOATS, SC_BYTES, bar);
  };

  bool ok = true;
  if (warp == 8) {
    // ---------------- control: TMA loads and MMA issue (one lane) ----------------
    // The two products that do not depend on the state, U~^T = V^T Tb^T and W^T = K^T Tw^T, are issued one
    // chunk ahead, behind the previous chunk's state update, so that only S^T W^T and the update itself are
    // on the chain.  Loads run two chunks ahead of their use.
    auto issue_ahead = [&](int ck) -> bool {
      const uint32_t par = (uint32_t)((ck >> 1) & 1);
      const int b = ck & 1;
      if (!(mbar_wait(&sm.bar_v[b], par, abort_flag, p.s.status, p.wait_limit) && mbar_wait(&sm.bar_k[b], par, abort_flag, p.s.status, p.wait_limit)))
        return false;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t i64 = idesc_f16(D, CH, 0, 1);     // the T tiles are stored [column][row]: MN-major B operands
      const uint64_t a_v = smem_desc(smem_u32(sm.VT), 16, 1024), b_tb = smem_desc(smem_u32(sm.Tb), 16, 1024);
#pragma unroll
      for (int k = 0; k < CH / 16; ++k) umma_bf16(tm_U, a_v + 2 * k, b_tb + 128 * k, i64, k != 0);   // U~^T = V^T Tb^T
      if (erase && (ck > 0 || has_init)) {
        const uint64_t a_k = smem_desc(smem_u32(sm.KT[b]), 16, 1024), b_tw = smem_desc(smem_u32(sm.Tw), 16, 1024);
#pragma unroll
        for (int k = 0; k < CH / 16; ++k) umma_bf16(tm_W, a_k + 2 * k, b_tw + 128 * k, i64, k != 0); // W^T = K^T Tw^T
      }
      umma_commit(&sm.bar_m1[b]);
      if (ck + 1 < n_chunks) {
        // once these (and everything issued before them) are done, V^T, Tb, Tw and the other key buffer are free
        if (!mbar_wait(&sm.bar_m1[b], par, abort_flag, p.s.status, p.wait_limit)) return false;
        load_v(ck + 1);
        if (ck > 0) load_k(ck + 1);
      }
      return true;
    };
    if (lane == 0) {
      load_v(0);
      if (!p.withhold_first_keys) load_k(0);
      if (n_chunks > 1) load_k(1);
      ok = issue_ahead(0);
    }
    for (int ck = 0; ck < n_chunks; ++ck) {
      const int b = ck & 1;
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();                                                 // S1: -W^T and the fp16 state are in shared memory
      if (lane == 0 && ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (erase && (ck > 0 || has_init)) {
          const uint32_t imn = idesc_f16(D, CH, 1, 1);
          const uint64_t a_s = smem_desc(smem_u32(sm.S16), TILE_KV, 1024), b_w = smem_desc(smem_u32(sm.WU), 16, 1024);
#pragma unroll
          for (int k = 0; k < D / 16; ++k)                                                                // U^T -= S^T W^T,
            if (16 * k < dk) umma_bf16(tm_U, a_s + 128 * k, b_w + 128 * k, imn, 1u);                      // summed over d_k only
        }
        umma_commit(&sm.bar_m2[b]);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();                                                 // S2: (f U)^T is in shared memory, S is decayed
      if (lane == 0 && ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t i128 = idesc_f16(D, D, 0, 0);
        const uint64_t a_k = smem_desc(smem_u32(sm.KT[b]), 16, 1024), b_u = smem_desc(smem_u32(sm.WU), 16, 1024);
#pragma unroll
        for (int k = 0; k < CH / 16; ++k) umma_bf16(tm_S, a_k + 2 * k, b_u + 2 * k, i128, (ck > 0 || has_init || k != 0) ? 1u : 0u);
        umma_commit(&sm.bar_m3[b]);
        if (ck + 1 < n_chunks) ok = issue_ahead(ck + 1);               // tensor memory of U and W was drained before S2
      }
    }
  } else {
    // ---------------- compute: tensor memory <-> shared memory ----------------
    const int quarter = warp & 3, half = warp >> 2;
    const int row = quarter * 32 + lane;                                // tensor-memory lane = d_k or d_v index
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    if (has_init) {
      // the state this request continues: row `row`, this warp's 64 columns, into tensor memory (zero outside
      // the head's own rows and this CTA's columns)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float v[32];
        const int cbase = half * 64 + c * 32;
        const float* src = init + (int64_t)row * dv + cbase;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *(float4*)(v + 4 * q) = (row < dk && cbase + 4 * q < dvb) ? *(const float4*)(src + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
        tmem_st32(tm_S + lane_off + (uint32_t)cbase, v);
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    for (int ck = 0; ck < n_chunks; ++ck) {
      const uint32_t par = (uint32_t)((ck >> 1) & 1);
      const int b = ck & 1;
      const float* sc = sm.sc[b];
      if (ok) ok = mbar_wait(&sm.bar_k[b], par, abort_flag, p.s.status, p.wait_limit);     // row factors and gamma_n
      if ((ck > 0 || has_init) && ok) {
        // the state left by the previous chunk (or the initial one): fp16 copy for S^T W^T, then decay in place
        if (ck > 0) ok = mbar_wait(&sm.bar_m3[b ^ 1], (uint32_t)(((ck - 1) >> 1) & 1), abort_flag, p.s.status, p.wait_limit);
        if (ok) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const float decay = sc[CH];
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            float v[32];
            tmem_ld32(tm_S + lane_off + (uint32_t)(half * 64 + c * 32), v);
            if (erase) store_row32(sm.S16 + half * TILE_KV, row, c * 32, v);
            if (p.dump_s && row < dk) {          // the state entering this chunk, for the layer's per-token outputs
              __half* ds = p.dump_s + (((long long)(slot0 + ck) * p.n_v_heads + h) * dk + row) * dv + col0 + half * 64 + c * 32;
#pragma unroll
              for (int q = 0; q < 4; ++q)
                if (half * 64 + c * 32 + 8 * q < dvb)
                  *(uint4*)(ds + 8 * q) = make_uint4(pack_h2(v[8 * q], v[8 * q + 1]), pack_h2(v[8 * q + 2], v[8 * q + 3]),
                                                     pack_h2(v[8 * q + 4], v[8 * q + 5]), pack_h2(v[8 * q + 6], v[8 * q + 7]));
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] *= decay;
            tmem_st32(tm_S + lane_off + (uint32_t)(half * 64 + c * 32), v);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
        // -W^T: this warp's 32 of the 64 chunk-row columns
        if (ok && erase) ok = mbar_wait(&sm.bar_m1[b], par, abort_flag, p.s.status, p.wait_limit);
        if (ok && erase) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          float v[32];
          tmem_ld32(tm_W + lane_off + (uint32_t)(half * 32), v);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = -v[i];
          store_row32(sm.WU, row, half * 32, v);
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();                                                 // S1
      if (ok) ok = mbar_wait(&sm.bar_m2[b], par, abort_flag, p.s.status, p.wait_limit);
      if (ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        float v[32];
        tmem_ld32(tm_U + lane_off + (uint32_t)(half * 32), v);
        if (p.dump_u && row < dvb) {             // U^T of this chunk: value index `row`, chunk rows half * 32 ..
          __half* du = p.dump_u + (((long long)(slot0 + ck) * p.n_v_heads + h) * dv + col0 + row) * CH + half * 32;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            *(uint4*)(du + 8 * q) = make_uint4(pack_h2(v[8 * q], v[8 * q + 1]), pack_h2(v[8 * q + 2], v[8 * q + 3]),
                                               pack_h2(v[8 * q + 4], v[8 * q + 5]), pack_h2(v[8 * q + 6], v[8 * q + 7]));
        }
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] *= sc[half * 32 + i];              // f_j of chunk row j
        store_row32(sm.WU, row, half * 32, v);
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();                                                 // S2
    }
    // ---------------- the final state ----------------
    if (ok) ok = mbar_wait(&sm.bar_m3[(n_chunks - 1) & 1], (uint32_t)(((n_chunks - 1) >> 1) & 1), abort_flag, p.s.status, p.wait_limit);
    if (ok) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float v[32];
        const int cbase = half * 64 + c * 32;
        tmem_ld32(tm_S + lane_off + (uint32_t)cbase, v);
        float* dst = out + (int64_t)row * dv + cbase;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          if (row < dk && cbase + 4 * q < dvb) *(float4*)(dst + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 8) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(256));
  }
}

bool encode_tiles(CUtensorMap* map, const void* base, uint64_t rows, uint32_t box_rows) {
  // a stack of [rows][64] fp16 tiles, 128-byte rows, 128-byte swizzle
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {CH, rows};
  cuuint64_t strides[1] = {CH * 2};
  cuuint32_t box[2] = {CH, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Column blocks a value head is split into: as few as keep a block within 128 columns (a multiple of 4, for the
// vector stores), one more doubling while the chains would otherwise leave most SMs without a CTA.
int sr_scan_chain_value_blocks(int d_v, long long chains, int sm_count) {
  int n = (d_v + D - 1) / D;
  while (d_v % n != 0 || (d_v / n) % 4 != 0) ++n;
  if (chains * n < sm_count && (d_v / n) % 8 == 0 && d_v / (2 * n) >= 32) n *= 2;
  return n;
}

bool sr_scan_chain_supported(int d_k, int d_v) {
  return d_k % 16 == 0 && d_k >= 16 && d_k <= D && d_v % 4 == 0 && d_v > 0 && d_v <= 8 * D;
}

cudaError_t sr_launch_scan_chain_umma(const sr_ctx* ctx, const SrSched& s, const SrFused& fused, const void* split_buf,
                                      char* out_ssm_layer, int64_t slot_stride, int ctx_sm_count, cudaStream_t stream) {
  // fused.in_ssm_layer: states to continue from (may be the output array itself: every CTA reads its block before
  // it writes it)
  const sr_model_desc& d = ctx->desc;
  const int smem_bytes = (int)sizeof(Smem);
  const cudaError_t once = sr_once_per_device(SR_ONCE_CHAIN_UMMA, [] {
    return cudaFuncSetAttribute(sr_scan_chain_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
  });
  if (once != cudaSuccess) return once;
  CUtensorMap map_kv, map_tt;
  if (!encode_tiles(&map_kv, fused.kv16, (uint64_t)s.max_slots * fused.ncb * D, D)) return cudaErrorInvalidValue;
  if (!encode_tiles(&map_tt, split_buf, (uint64_t)s.max_slots * d.n_v_heads * 2 * CH, CH)) return cudaErrorInvalidValue;
  ChainUmmaParams p;
  p.s = s;
  p.sc = (const float*)((const char*)split_buf + (size_t)s.max_slots * d.n_v_heads * TT_HALFS * sizeof(__half));
  p.ncb = fused.ncb;
  p.n_k_heads = d.n_k_heads;
  p.n_v_heads = d.n_v_heads;
  p.d_k = d.d_k;
  p.d_v = d.d_v;
  const int n_vb = sr_scan_chain_value_blocks(d.d_v, (long long)d.n_v_heads * s.n_requests, ctx_sm_count);
  p.dvb = d.d_v / n_vb;
  p.out_layer = out_ssm_layer;
  p.slot_stride = slot_stride;
  p.erase = d.recurrence == SR_REC_GATED_DELTA;
  p.k_ch0 = fused.k_ch0;
  p.v_ch0 = fused.v_ch0;
  p.dump_s = fused.dump_s;
  p.dump_u = fused.dump_u;
  p.in_layer = fused.in_ssm_layer;
  p.in_slot_stride = fused.in_ssm_slot_stride;
  p.withhold_first_keys = (ctx->debug_flags & SR_DEBUG_EXPIRE_WAIT) ? 1 : 0;
  p.wait_limit = p.withhold_first_keys ? 2000000ll : WAIT_LIMIT_CYCLES;      // about a millisecond for the injected fault
  dim3 grid((unsigned)d.n_v_heads, (unsigned)s.n_requests, (unsigned)n_vb);
  sr_scan_chain_umma_kernel<<<grid, THREADS, smem_bytes, stream>>>(map_kv, map_tt, p);
  return cudaGetLastError();
}
