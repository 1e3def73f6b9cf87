// In-projection fused with the anchor gather in front of it and the causal conv + SiLU behind it
// (Section 2.1: keys, values and gates are projections of the layer input; Section 5.1: anchors are
// read through the page table).
//
// The MMA is issued with the roles of the two operands swapped with respect to the plain projection:
//
//   D[channel][token] = sum_j W[channel][j] * X[token][j]        M = 128 channels, N = 256 tokens
//
// so a tensor-memory lane is a channel and its columns are consecutive tokens (four 64-row page slots).
// Each epilogue thread therefore owns one channel and walks its tokens in order: the width-4 causal conv
// is a sliding window in registers, with no exchange between threads and no shared-memory traffic next to
// the operand reads of the tensor core.  What reaches memory is the scan's input format (SrFused):
// fp16 SiLU(conv(Z)) tiles, channel-major, the raw fp32 gate rows, and a few raw fp32 projection rows per
// slot: the last three valid ones (they are the k, v part of the conv state) and, for the first slot of a
// tile, rows 0..2, whose conv history sits in another tile and which the scan therefore finishes itself.
//
// Structure as in the plain projection: persistent, one CTA per SM, warp 0 TMA producer (one 128-channel
// weight box and four anchor-page boxes per 64-wide k block, 4-stage ring), warp 1 tcgen05.mma issuer with
// a double-buffered accumulator in tensor memory, epilogue warps behind.  SCALED handles e4m3 weights with
// 128 x 128 block scales: 128-deep K groups are accumulated separately and added as scale x partial sum in
// fp32 registers by eight epilogue warps (one scale per K group per tile, since a tile is one 128-channel
// block).  sr_proj_w8a8_kernel (below) runs the 8-bit form.  All waits are bounded.
#include <type_traits>

#include "sr_umma.cuh"

namespace {

constexpr int BM = 128;                  // channels per tile (MMA M)
constexpr int BN = 256;                  // tokens per tile (MMA N) = SLOTS page slots
constexpr int SLOTS = BN / SR_PAGE_ROWS;
constexpr int BK = 64, STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;     // 16 KB of weights
constexpr int B_BYTES = BN * BK * 2;     // 32 KB of anchors
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int NUM_THREADS = 192;         // producer warp, MMA warp, 4 epilogue warps
constexpr int NUM_THREADS_SCALED = 320;  // producer warp, MMA warp, 8 epilogue warps
constexpr long long WEIGHT_BLOCK_BYTES = 30ll << 20;   // weights held in L2 while the token tiles stream past

struct FusedParams {
  SrSched s;
  int32_t pool_layer;
  int32_t k_blocks;      // d_model / 64
  int32_t n_q;           // rows of W_qkv in front of the k block (conv channel offset)
  int32_t w_row0;        // row of the weight tensor map where the k | v block starts
  int32_t n_ct;          // 128-channel tiles of k | v; tile index n_ct is the gate tile
  int32_t n_gate;        // 2 H_v
  int32_t ncb;
  int32_t n_kv;
  int32_t act_identity;
  const float* w_scale;  // SCALED
  int32_t scale_ld;      // SCALED: d / 128
  const float* sx;       // W8A8: activation scales [slot][d / 128][64]
  int32_t gate_only;     // pair form: only the gate tile (the W8A8 path runs the bf16 gate rows on their own)
  const __nv_bfloat16* conv_w;
  __half* kv16;
  float* zraw;
  float* gates;
  const __nv_bfloat16* hist;   // conv state each request continues from, [request][C][3], or null
  int32_t conv_ch;
  int32_t fp16_stage;    // operands are the fp16 staging copies: fp16 MMA formats, anchors in slot order (page = slot)
  int32_t slot_order;    // the row operand is a packed buffer in slot order (page = slot), bf16 (group replay)
  int32_t group_t;       // token tiles per rasterisation group
  int32_t group_c;       // channel tiles (pair tiles in the two-CTA form) per block inside a group
  unsigned int* next_tile;     // two-CTA form: tiles handed out so far beyond the first one of every pair
  unsigned long long* mail;    // two-CTA form: [pair][SR_SCHED_RING] (sequence number << 32 | tile + 1; tile + 1 = 0: no more)
};

__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
  __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// One page slot (64 tokens, in v) of one channel: conv + SiLU -> fp16 tile row, raw rows -> zraw;
// or, for the gate tile, the raw values -> gates.  z1, z2, z3 carry the three previous raw tokens.
__device__ __forceinline__ void emit_slot(const FusedParams& p, bool gate, int ch, int ch_local, int ct, int slot,
                                          bool head_rows, int vr, float* v, const float (&cw)[4], float& z1,
                                          float& z2, float& z3) {
  // Rows past the request's end (a partial last page, a padding slot) are not part of the window: whatever the
  // pool holds there -- stale anchors, never-written memory, NaN -- must not reach the scan, whose products mix
  // the rows of a chunk.  vr is uniform over the warp.
  if (vr < SR_PAGE_ROWS) {
#pragma unroll
    for (int i = 0; i < SR_PAGE_ROWS; ++i)
      if (i >= vr) v[i] = 0.f;
  }
  if (!gate && ch >= p.n_kv) return;     // the last channel tile may reach past the k | v block
  if (!sr_check_slot(p.s, slot)) return;
  if (gate) {
    if (ch < p.n_gate) {
      float* g = p.gates + ((long long)slot * p.n_gate + ch) * SR_PAGE_ROWS;
#pragma unroll
      for (int q = 0; q < 16; ++q) __stcs((float4*)(g + 4 * q), make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]));
    }
    return;
  }
  uint32_t packed[32];
#pragma unroll
  for (int i = 0; i < 64; i += 2) {
    float y0 = cw[0] * z3 + cw[1] * z2 + cw[2] * z1 + cw[3] * v[i];
    float y1 = cw[0] * z2 + cw[1] * z1 + cw[2] * v[i] + cw[3] * v[i + 1];
    z3 = z1;
    z2 = v[i];
    z1 = v[i + 1];
    if (!p.act_identity) {
      y0 = __fdividef(y0, 1.f + __expf(-y0));
      y1 = __fdividef(y1, 1.f + __expf(-y1));
    }
    packed[i >> 1] = pack_h2(y0, y1);
  }
  __half* dst = p.kv16 + (((long long)slot * p.ncb + ct) * BM + ch_local) * SR_PAGE_ROWS;
#pragma unroll
  for (int q = 0; q < 8; ++q)     // streaming stores: the tiles are next read by another kernel, long after they left L2
    __stcs((uint4*)(dst + 8 * q), make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]));
  float* zr = p.zraw + (long long)slot * 6 * p.n_kv + ch;
  if (head_rows) {
    zr[0] = v[0];
    zr[p.n_kv] = v[1];
    zr[2 * (long long)p.n_kv] = v[2];
  }
  if (vr == SR_PAGE_ROWS) {                       // the usual case: a full slot, last rows 61..63
    zr[3 * (long long)p.n_kv] = v[61];
    zr[4 * (long long)p.n_kv] = v[62];
    zr[5 * (long long)p.n_kv] = v[63];
  } else {                                        // a request's partial last slot (uniform over the warp)
    const int lo = max(vr - 3, 0);
#pragma unroll
    for (int i = 0; i < 64; ++i)
      if (i >= lo && i < vr) zr[(long long)(3 + i - lo) * p.n_kv] = v[i];
  }
}

// conv history of a slot that opens its request: zeros, or the last three inputs of the state it continues
__device__ __forceinline__ void load_history(const FusedParams& p, bool gate, int first, int ch, float& z1, float& z2,
                                             float& z3) {
  z1 = 0.f; z2 = 0.f; z3 = 0.f;
  if (first && p.hist && !gate && ch < p.n_kv) {
    const __nv_bfloat16* h = p.hist + ((long long)(first - 1) * p.conv_ch + p.n_q + ch) * (SR_CONV_W - 1);
    z3 = __bfloat162float(h[0]);
    z2 = __bfloat162float(h[1]);
    z1 = __bfloat162float(h[2]);
  }
}

template <bool SCALED>
__global__ void __launch_bounds__(SCALED ? NUM_THREADS_SCALED : NUM_THREADS, 1)
sr_proj_fused_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                     const __grid_constant__ CUtensorMap map_g, const FusedParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = (uint64_t*)(smem + STAGES * STAGE_BYTES);
  uint64_t* empty_bar = full_bar + STAGES;
  uint64_t* tfull_bar = empty_bar + STAGES;      // [2] accumulator (or K group) ready for the epilogue
  uint64_t* tempty_bar = tfull_bar + 2;          // [2] accumulator drained
  uint32_t* tmem_slot = (uint32_t*)(tempty_bar + 2);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_slots = (int)p.s.status[1];
  const int t_tiles = (n_slots + SLOTS - 1) / SLOTS;
  const int c_tiles = p.n_ct + 1;
  const long long total_tiles = (long long)t_tiles * c_tiles;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull_bar[i], 1); mbar_init(&tempty_bar[i], SCALED ? 8 : 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  // tile index -> (channel tile, token tile): token tiles in groups of group_t (by default one group, all of
  // them); inside a group the channel tiles are walked in blocks of group_c, and inside a block every token
  // tile of the group passes over the block's weights, channel-fastest.  The launch function picks the sizes.
  auto tile_coords = [&](long long tile, int& ct, int& tt) {
    const long long per_group = (long long)p.group_t * c_tiles;
    const int g = (int)(tile / per_group);
    int r = (int)(tile % per_group);
    const int gt = min(p.group_t, t_tiles - g * p.group_t);    // token tiles in this group
    const int per_block = gt * p.group_c;                       // tiles in a full channel block
    const int cb = r / per_block;
    r -= cb * per_block;
    const int gc = min(p.group_c, c_tiles - cb * p.group_c);    // channel tiles in this block
    ct = cb * p.group_c + r % gc;
    tt = g * p.group_t + r / gc;
  };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        int ct, tt;
        tile_coords(tile, ct, tt);
        int page[SLOTS];
#pragma unroll
        for (int q = 0; q < SLOTS; ++q) page[q] = (p.fp16_stage || p.slot_order) ? SLOTS * tt + q : p.s.slot_page[SLOTS * tt + q];
        const bool gate = ct == p.n_ct;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.s.status)) { ok = false; break; }
          uint8_t* a_dst = smem + stage * STAGE_BYTES;
          uint8_t* b_dst = a_dst + A_BYTES;
          mbar_expect_tx(&full_bar[stage], STAGE_BYTES);
          if (gate) tma_load_2d(a_dst, &map_g, &full_bar[stage], kb * BK, 0);
          else tma_load_2d(a_dst, &map_w, &full_bar[stage], kb * BK, p.w_row0 + ct * BM);
#pragma unroll
          for (int q = 0; q < SLOTS; ++q)
            tma_load_4d(b_dst + q * (B_BYTES / SLOTS), &map_x, &full_bar[stage], kb * BK, 0, p.pool_layer, page[q]);
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      const uint32_t idesc = umma_idesc(BM, BN, p.fp16_stage != 0);
      for (long long tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
        // SCALED: one accumulator buffer per 128-deep K group (2 stages); otherwise one per tile
        const int blocks_per_acc = SCALED ? 2 : p.k_blocks;
        for (int kb0 = 0; ok && kb0 < p.k_blocks; kb0 += blocks_per_acc) {
          if (!mbar_wait(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, p.s.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
          for (int kb = kb0; kb < kb0 + blocks_per_acc; ++kb) {
            if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.s.status)) { ok = false; break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = smem_u32(smem + stage * STAGE_BYTES);
            const uint64_t a_desc = umma_smem_desc(a_addr);
            const uint64_t b_desc = umma_smem_desc(a_addr + A_BYTES);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              umma_bf16(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                        (kb != kb0 || k != 0) ? 1u : 0u);
            umma_commit(&empty_bar[stage]);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          umma_commit(&tfull_bar[acc]);
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // epilogue: thread = channel (tensor-memory lane 32*(warp%4) + lane)
    const int quarter = warp & 3;
    const int ch_local = quarter * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (long long tile = blockIdx.x; ok && tile < total_tiles; tile += gridDim.x) {
      int ct, tt;
      tile_coords(tile, ct, tt);
      const bool gate = ct == p.n_ct;
      const int ch = gate ? ch_local : ct * BM + ch_local;
      float cw[4] = {0.f, 0.f, 0.f, 0.f};
      if (!gate && ch < p.n_kv) {
        const uint2 wv = *(const uint2*)(p.conv_w + (long long)(p.n_q + ch) * SR_CONV_W);
        const __nv_bfloat16* e = (const __nv_bfloat16*)&wv;
#pragma unroll
        for (int q = 0; q < 4; ++q) cw[q] = __bfloat162float(e[q]);
      }
      float z1 = 0.f, z2 = 0.f, z3 = 0.f;
      if (SCALED) {
        // this warp's half of the tile: page slots 2*half, 2*half + 1 (tensor-memory columns half*128 ..)
        const int half = (warp - 2) >> 2;
        const float* scale_row = gate ? nullptr : p.w_scale + (long long)((p.n_q + ct * BM) / 128) * p.scale_ld;
        float sum[128];
#pragma unroll
        for (int i = 0; i < 128; ++i) sum[i] = 0.f;
        const int k_groups = p.k_blocks / 2;
        for (int kg = 0; kg < k_groups; ++kg) {
          if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag, p.s.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const float sc = gate ? 1.f : __ldg(scale_row + kg);
          const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN + (uint32_t)half * 128;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            float v[32];
            tmem_ld32(taddr + (uint32_t)(c * 32), v);
#pragma unroll
            for (int i = 0; i < 32; ++i) sum[c * 32 + i] = fmaf(sc, v[i], sum[c * 32 + i]);
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&tempty_bar[acc]);
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
        if (!ok) break;
#pragma unroll
        for (int sl = 0; sl < 2; ++sl) {
          const int slot = SLOTS * tt + 2 * half + sl;
          if (sl == 0 || p.s.slot_first[slot]) load_history(p, gate, p.s.slot_first[slot], ch, z1, z2, z3);
          emit_slot(p, gate, ch, ch_local, ct, slot, sl == 0, p.s.slot_rows[slot], sum + sl * 64, cw, z1, z2, z3);
        }
      } else {
        if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag, p.s.status)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN;
#pragma unroll 1
        for (int sl = 0; sl < SLOTS; ++sl) {
          const int slot = SLOTS * tt + sl;
          float v[64];
          tmem_ld32(taddr + (uint32_t)(sl * 64), v);
          tmem_ld32(taddr + (uint32_t)(sl * 64 + 32), v + 32);
          if (sl == 0 || p.s.slot_first[slot]) load_history(p, gate, p.s.slot_first[slot], ch, z1, z2, z3);
          emit_slot(p, gate, ch, ch_local, ct, slot, sl == 0, p.s.slot_rows[slot], v, cw, z1, z2, z3);
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty_bar[acc]);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

// Tile scheduler of the persistent kernels below (the two-CTA form; the 8-bit form, where a "pair" is one CTA).
// Tiles are handed out in index order at run time (a pair that finishes early
// takes the next one), so the pairs that share an anchor tile -- neighbours in the tile order -- always work on it at
// nearly the same time, however far the pairs have drifted apart; with a fixed assignment the drift decides how often
// the shared tile is still in L2.  The leader's producer thread draws the tile and publishes it, with its sequence
// number, in the pair's ring of mailboxes in global memory; every other role of the pair (the partner's producer, the
// MMA issuer, the epilogue warps of both CTAs) reads it there.  Nobody runs more than six tiles ahead of the slowest
// role (operand ring + two accumulators), so a ring of sixteen is never overrun.
__device__ __forceinline__ void sched_publish(unsigned long long* mail, int pair, uint32_t seq, long long tile) {
  const unsigned long long v = ((unsigned long long)seq << 32) | (unsigned long long)(uint32_t)(tile + 1);
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(mail + (size_t)pair * SR_SCHED_RING + (seq % SR_SCHED_RING)), "l"(v) : "memory");
}
// the tile of sequence number seq; -1: no more tiles; -2: gave up (bounded like every wait).  Without mailboxes (a
// launch of at most one tile per pair) the assignment is fixed: tile = pair.
__device__ __forceinline__ long long sched_get(const unsigned long long* mail, int pair, uint32_t seq, long long total_tiles,
                                               volatile int* abort_flag, uint32_t* status) {
  if (!mail) return seq == 1 && pair < total_tiles ? (long long)pair : -1;
  const unsigned long long* slot = mail + (size_t)pair * SR_SCHED_RING + (seq % SR_SCHED_RING);
  const long long t0 = clock64();
  uint32_t spins = 0;
  for (;;) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(slot) : "memory");
    if ((uint32_t)(v >> 32) == seq) return (long long)(uint32_t)v - 1;
    if ((++spins & 0xFFu) == 0u) {
      if (*abort_flag) return -2;
      if (clock64() - t0 > WAIT_LIMIT_CYCLES) {
        *abort_flag = 1;
        atomicOr(status, SR_DEV_WAIT_EXPIRED);
        return -2;
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------------
// W8A8: e4m3 weight codes (as the caller stores them) x e4m3 activation codes (written by the quantiser, page-slot
// order), tcgen05 kind::f8f6f4, one 128-byte row of K per stage.  Both operands carry block scales that are plain
// fp32 numbers, not the hardware's power-of-two block format, so every 128-deep K group has to enter the result as
//     total[token][channel] += w_scale[channel block][group] * x_scale[token][group] * partial[token][channel]
// outside the tensor core: one multiply-add per output element per group.  To make that fold cost nothing but the
// multiply-add, this kernel puts the TOKENS on the MMA's M axis (128 tokens = two page slots; N = 256 channels =
// two 128-channel scale blocks): a tensor-memory lane -- a thread -- is then a token, a warpgroup owns one scale
// block, and the scale product of a group is ONE number per thread, fetched two groups ahead.
// Layout: three warpgroups.  Warpgroup 0 holds the TMA producer and the MMA issuer and gives most of its registers
// away (setmaxnreg); warpgroups 1 and 2 take them and keep the TOTALS IN REGISTERS (one token x 128 channels per
// thread), while the partial sums of a group are double-buffered in tensor memory (2 x 256 columns), so the tensor
// core works on group g + 1 while group g is folded.  The waits on that short chain (group done -> fold -> buffer
// free -> next group) poll instead of suspending.
// The conv + SiLU epilogue wants the other orientation (a thread walks the tokens of one channel): after the last
// group each warpgroup turns its totals around through shared memory, 64 channels at a time -- every thread writes
// its token's totals as a column, then reads one channel's 64 tokens of one page slot as a row -- and the epilogue
// of the 16-bit kernels runs unchanged (every slot's first three rows are finished later by the chunk-local kernel,
// like the first rows of a tile in the 16-bit kernels).
constexpr int W8_BK = 128;                       // bytes (= codes) of K per stage
constexpr int W8_THREADS = 384;
constexpr int W8_TOK = 128;                      // tokens per tile (MMA M)
constexpr int W8_SLOTS = W8_TOK / SR_PAGE_ROWS;
constexpr int W8_CH = 256;                       // channels per tile (MMA N)
constexpr int W8_STAGES = 3;
constexpr int W8_X_BYTES = W8_TOK * W8_BK;       // 16 KB of activation codes
constexpr int W8_W_BYTES = W8_CH * W8_BK;        // 32 KB of weight codes
constexpr int W8_STAGE_BYTES = W8_X_BYTES + W8_W_BYTES;
constexpr int W8_TR_LD = W8_TOK + 4;             // floats per channel row of a turn-around buffer (bank spread)
constexpr int W8_TR_BYTES = 64 * W8_TR_LD * 4;   // 64 channels x 128 tokens per warpgroup and round
constexpr int W8_SMEM_BYTES = W8_STAGES * W8_STAGE_BYTES + 2 * W8_TR_BYTES + 1024 + 256;

__global__ void __launch_bounds__(W8_THREADS, 1)
sr_proj_w8a8_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const FusedParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  float* turn = (float*)(smem + W8_STAGES * W8_STAGE_BYTES);     // [2 warpgroups][64][W8_TR_LD]
  uint64_t* full_bar = (uint64_t*)(smem + W8_STAGES * W8_STAGE_BYTES + 2 * W8_TR_BYTES);
  uint64_t* empty_bar = full_bar + W8_STAGES;
  uint64_t* pfull_bar = empty_bar + W8_STAGES;   // [2] partial sums of a group complete in buffer b
  uint64_t* pempty_bar = pfull_bar + 2;          // [2] ... folded into the totals by the eight folding warps
  uint32_t* tmem_slot = (uint32_t*)(pempty_bar + 2);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_slots = (int)p.s.status[1];
  const int t_tiles = (n_slots + W8_SLOTS - 1) / W8_SLOTS;
  const int c_tiles = (p.n_ct + 1) / 2;          // 256-channel tiles of k | v (the last may be half empty); the bf16
                                                 // gate rows go through their own launch
  const long long total_tiles = (long long)t_tiles * c_tiles;
  const int k_groups = p.k_blocks;               // one stage = one 128-deep group

  if (threadIdx.x == 0) {
    for (int i = 0; i < W8_STAGES; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&pfull_bar[i], 1); mbar_init(&pempty_bar[i], 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  // Tile order: channel-fastest.  The 8-bit k | v weights of a layer (tens of MB) stay in L2 as a whole; the CTAs
  // work on a handful of neighbouring token tiles at a time, whose codes are read from HBM once.
  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    if (warp == 0 && lane == 0) {                // TMA producer
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      long long tile = (long long)blockIdx.x < total_tiles ? (long long)blockIdx.x : -1;
      for (uint32_t seq = 1;; ++seq) {
        if (p.mail) sched_publish(p.mail, blockIdx.x, seq, ok ? tile : -1);
        else tile = sched_get(p.mail, blockIdx.x, seq, total_tiles, abort_flag, p.s.status);
        if (tile < 0 || !ok) break;
        unsigned int drawn = 0;
        if (p.mail) drawn = atomicAdd(p.next_tile, 1u);            // the tile after this one
        const int tt = (int)(tile / c_tiles), ct = (int)(tile % c_tiles);
        for (int kb = 0; kb < k_groups; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.s.status)) { ok = false; break; }
          uint8_t* x_dst = smem + stage * W8_STAGE_BYTES;
          uint8_t* w_dst = x_dst + W8_X_BYTES;
          mbar_expect_tx(&full_bar[stage], W8_STAGE_BYTES);
#pragma unroll
          for (int q = 0; q < W8_SLOTS; ++q)
            tma_load_4d(x_dst + q * (W8_X_BYTES / W8_SLOTS), &map_x, &full_bar[stage], kb * W8_BK, 0, 0, W8_SLOTS * tt + q);
#pragma unroll
          for (int h = 0; h < 2; ++h)            // rows past the weight matrix arrive as zeros
            tma_load_2d(w_dst + h * (W8_W_BYTES / 2), &map_w, &full_bar[stage], kb * W8_BK, p.w_row0 + ct * W8_CH + h * BM);
          if (++stage == W8_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (p.mail) {
          const long long t = (long long)drawn + gridDim.x;
          tile = t < total_tiles ? t : -1;
        }
      }
    } else if (warp == 1 && lane == 0) {         // MMA issue
      int stage = 0;
      uint32_t phase = 0, gcount = 0;
      bool ok = true;
      const uint32_t idesc = umma_idesc_e4m3(W8_TOK, W8_CH);
      for (uint32_t seq = 1; ok; ++seq) {
        if (sched_get(p.mail, blockIdx.x, seq, total_tiles, abort_flag, p.s.status) < 0) break;
        for (int kg = 0; kg < k_groups; ++kg, ++gcount) {
          const uint32_t b = gcount & 1u;
          // buffer b was folded two groups ago
          if (!mbar_wait_spin(&pempty_bar[b], ((gcount >> 1) & 1u) ^ 1u, abort_flag, p.s.status)) { ok = false; break; }
          if (!mbar_wait_spin(&full_bar[stage], phase, abort_flag, p.s.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t x_addr = smem_u32(smem + stage * W8_STAGE_BYTES);
          const uint64_t a_desc = umma_smem_desc(x_addr), b_desc = umma_smem_desc(x_addr + W8_X_BYTES);
#pragma unroll
          for (int k = 0; k < W8_BK / 32; ++k)
            umma_e4m3(tmem_base + b * (uint32_t)W8_CH, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, k != 0 ? 1u : 0u);
          umma_commit(&pfull_bar[b]);
          umma_commit(&empty_bar[stage]);
          if (++stage == W8_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 232;");
    // fold: tensor-memory lanes 32 * (warp % 4) .. = tokens of the tile, columns wg * 128 .. + 127 = channels
    const int quarter = warp & 3, wg = (warp >> 2) - 1;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    float* buf = turn + wg * (W8_TR_BYTES / 4);
    const int tid = quarter * 32 + lane;                   // the token while folding; (slot, channel) = (tid / 64, tid % 64) after
    const int last_block = (p.n_q + p.n_kv - 1) / 128;     // last row of the weight-scale matrix
    uint32_t gcount = 0;
    bool ok = true;
    for (uint32_t seq = 1;; ++seq) {
      int tile_lo = 0;
      if (lane == 0) tile_lo = (int)sched_get(p.mail, blockIdx.x, seq, total_tiles, abort_flag, p.s.status);
      const long long tile = __shfl_sync(0xffffffffu, tile_lo, 0);
      // one decision for all eight warps (they meet at named barriers below, so none may leave alone)
      if (named_bar_or(1, 256, tile == -2 || *abort_flag != 0) || tile < 0) break;
      const int tt = (int)(tile / c_tiles), ct = (int)(tile % c_tiles);
      const int cb = 2 * ct + wg;                          // this warpgroup's 128-channel block of k | v
      const float* ws = p.w_scale + (long long)min((p.n_q + cb * BM) / 128, last_block) * p.scale_ld;
      const float* xs = p.sx + (long long)(W8_SLOTS * tt + (tid >> 6)) * k_groups * SR_PAGE_ROWS + (tid & 63);
      // what the epilogue will need, fetched before the K loop
      const int sl = tid >> 6, slot = W8_SLOTS * tt + sl;
      const int vr = p.s.slot_rows[slot], first = p.s.slot_first[slot];
      uint2 cwv[2];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int ch = cb * BM + r * 64 + (tid & 63);
        cwv[r] = ch < p.n_kv ? __ldg((const uint2*)(p.conv_w + (long long)(p.n_q + ch) * SR_CONV_W)) : make_uint2(0u, 0u);
      }
      float tot[128];
#pragma unroll
      for (int i = 0; i < 128; ++i) tot[i] = 0.f;
      // the scales of group kg + 2 are fetched while group kg is folded
      float w_cur = __ldg(ws), x_cur = __ldg(xs);
      float w_nxt = k_groups > 1 ? __ldg(ws + 1) : 0.f, x_nxt = k_groups > 1 ? __ldg(xs + SR_PAGE_ROWS) : 0.f;
      for (int kg = 0; kg < k_groups; ++kg, ++gcount) {
        const uint32_t b = gcount & 1u, par = (gcount >> 1) & 1u;
        float w_far = 0.f, x_far = 0.f;
        if (kg + 2 < k_groups) {
          w_far = __ldg(ws + kg + 2);
          x_far = __ldg(xs + (long long)(kg + 2) * SR_PAGE_ROWS);
        }
        if (ok) ok = mbar_wait_spin(&pfull_bar[b], par, abort_flag, p.s.status);
        if (ok) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const float comb = w_cur * x_cur;
          const uint32_t taddr = tmem_base + lane_off + b * (uint32_t)W8_CH + (uint32_t)(wg * 128);
          float v0[32], v1[32];
          tmem_ld32_issue(taddr, v0);
#pragma unroll
          for (int c = 0; c < 4; c += 2) {
            tmem_ld32_issue(taddr + (uint32_t)((c + 1) * 32), v1);
            tmem_wait_ld();                      // waits for both; the second is consumed after the first chunk's math
#pragma unroll
            for (int i = 0; i < 32; ++i) tot[c * 32 + i] = fmaf(comb, v0[i], tot[c * 32 + i]);
            if (c + 2 < 4) tmem_ld32_issue(taddr + (uint32_t)((c + 2) * 32), v0);
#pragma unroll
            for (int i = 0; i < 32; ++i) tot[(c + 1) * 32 + i] = fmaf(comb, v1[i], tot[(c + 1) * 32 + i]);
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(&pempty_bar[b]);        // also after a failed wait: nobody is left waiting on this warp
        w_cur = w_nxt; x_cur = x_nxt;
        w_nxt = w_far; x_nxt = x_far;
      }
      // One decision for all eight warps (none may leave a tile alone: the other warps of its warpgroup wait for it
      // at the named barriers below): a wait that gave up anywhere in the CTA has raised the flag.
      if (named_bar_or(1, 256, *abort_flag != 0)) break;
      // The tile's totals are complete.  Two rounds of 64 channels: every thread writes its token's 64 totals as a
      // column, then reads one channel's 64 tokens of one page slot as a row and runs conv + SiLU on them.
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        if (r) asm volatile("bar.sync %0, 128;" ::"r"(2 + wg) : "memory");     // round 0 has been read
#pragma unroll
        for (int c = 0; c < 64; ++c) buf[c * W8_TR_LD + tid] = tot[r * 64 + c];
        asm volatile("bar.sync %0, 128;" ::"r"(2 + wg) : "memory");
        const int ch_local = r * 64 + (tid & 63), ch = cb * BM + ch_local;
        float v[64];
        const float4* row = (const float4*)(buf + (tid & 63) * W8_TR_LD + sl * SR_PAGE_ROWS);
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          const float4 a = row[q];
          v[4 * q] = a.x; v[4 * q + 1] = a.y; v[4 * q + 2] = a.z; v[4 * q + 3] = a.w;
        }
        const __nv_bfloat16* w4 = (const __nv_bfloat16*)&cwv[r];
        float cw[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) cw[q] = __bfloat162float(w4[q]);
        float z1, z2, z3;
        load_history(p, false, first, ch, z1, z2, z3);
        emit_slot(p, false, ch, ch_local, cb, slot, true, vr, v, cw, z1, z2, z3);
      }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

// ---------------------------------------------------------------------------------------------------
// Two-CTA form (bf16 weights): a pair of CTAs on neighbouring SMs shares one MMA tile of 256 channels x
// 256 tokens (tcgen05 cta_group::2).  Each CTA stages only its own 128 channels of weights and its own
// 128 tokens (two page slots) of anchors -- 32 KB per k block instead of 48 KB -- and the tensor core reads
// the token operand from both shared memories, so every byte staged feeds twice the work: less shared
// memory and L2 traffic per flop, and room for a 6-stage ring.  The leader CTA (rank 0) issues the MMAs;
// both CTAs run their own TMA producer and their own epilogue (the 128 channels in their tensor memory).

constexpr int STAGES2 = 6;
constexpr int A2_BYTES = BM * BK * 2;                 // 16 KB: 128 channels of weights
constexpr int B2_BYTES = (BN / 2) * BK * 2;           // 16 KB: 128 tokens of anchors
constexpr int STAGE2_BYTES = A2_BYTES + B2_BYTES;
constexpr int SMEM2_BYTES = STAGES2 * STAGE2_BYTES + 1024 + 256;

// Several layers in ONE launch (small batches: a single hit fills the device for a fraction of one wave per layer, and
// the launches of a call's layers would run one after the other): the tile space is (layer, channel tile, token
// tile), layer-major, and what differs from layer to layer -- the weight and gate-weight tensor maps, the conv
// weights, the layer's hand-over buffers, its conv history and its place in the pool -- comes from a table in the
// kernel's parameter space.
constexpr int PROJ_BATCH_MAX = 24;
struct alignas(64) BatchLayer {
  CUtensorMap map_w, map_g;
  const __nv_bfloat16* conv_w;
  __half* kv16;
  float* zraw;
  float* gates;
  const __nv_bfloat16* hist;
  int32_t pool_layer;
};
struct alignas(64) BatchTable {
  int32_t n_layers;
  BatchLayer layer[PROJ_BATCH_MAX];
};
struct NoBatch {};

template <class Table>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(NUM_THREADS, 1)
sr_proj_fused2_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                      const __grid_constant__ CUtensorMap map_g, const FusedParams p, const __grid_constant__ Table bt) {
  constexpr bool BATCHED = !std::is_same<Table, NoBatch>::value;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = (uint64_t*)(smem + STAGES2 * STAGE2_BYTES);   // used in the leader CTA only
  uint64_t* empty_bar = full_bar + STAGES2;                          // one set per CTA
  uint64_t* tfull_bar = empty_bar + STAGES2;                         // [2] one set per CTA
  uint64_t* tempty_bar = tfull_bar + 2;                              // [2] used in the leader CTA only
  uint32_t* tmem_slot = (uint32_t*)(tempty_bar + 2);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_slots = (int)p.s.status[1];
  const int t_tiles = (n_slots + SLOTS - 1) / SLOTS;
  const int n_pt = (p.n_ct + 1) / 2;              // 256-channel tiles of k | v (the last may be half empty); tile
                                                  // index n_pt is the gate tile
  const int c_tiles = p.gate_only ? 1 : n_pt + 1;
  const long long layer_tiles = (long long)t_tiles * c_tiles;
  long long total_tiles = layer_tiles;
  if constexpr (BATCHED) total_tiles = layer_tiles * bt.n_layers;

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES2; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&tfull_bar[i], 1); mbar_init(&tempty_bar[i], 8); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();               // the partner's barriers exist before anything signals them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  auto tile_coords = [&](long long tile, int& layer, int& pt, int& tt) {
    layer = 0;
    if constexpr (BATCHED) {
      layer = (int)(tile / layer_tiles);
      tile -= layer * layer_tiles;
    }
    if (p.gate_only) { pt = n_pt; tt = (int)tile; return; }
    const long long per_group = (long long)p.group_t * c_tiles;
    const int g = (int)(tile / per_group);
    int r = (int)(tile % per_group);
    const int gt = min(p.group_t, t_tiles - g * p.group_t);
    const int per_block = gt * p.group_c;
    const int cb = r / per_block;
    r -= cb * per_block;
    const int gc = min(p.group_c, c_tiles - cb * p.group_c);
    pt = cb * p.group_c + r % gc;
    tt = g * p.group_t + r / gc;
  };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t w_policy = l2_policy_evict_last();    // the weight block is the operand the tile order holds in L2
      long long tile = pair < total_tiles ? pair : -1;      // the leader's view; the partner reads the mailbox
      for (uint32_t seq = 1;; ++seq) {
        if (rank == 0 && p.mail) sched_publish(p.mail, pair, seq, ok ? tile : -1);
        if (rank != 0 || !p.mail) tile = sched_get(p.mail, pair, seq, total_tiles, abort_flag, p.s.status);
        if (tile < 0 || !ok) break;
        unsigned int drawn = 0;
        if (rank == 0 && p.mail) drawn = atomicAdd(p.next_tile, 1u);     // the tile after this one; used when this one is loaded
        int layer, pt, tt;
        tile_coords(tile, layer, pt, tt);
        const CUtensorMap* mw = &map_w;
        const CUtensorMap* mg = &map_g;
        int pool_layer = p.pool_layer;
        if constexpr (BATCHED) {
          mw = &bt.layer[layer].map_w;
          mg = &bt.layer[layer].map_g;
          pool_layer = bt.layer[layer].pool_layer;
        }
        const int slot_a = SLOTS * tt + 2 * rank;
        const bool by_slot = p.fp16_stage || p.slot_order;
        int page0 = by_slot ? slot_a : p.s.slot_page[slot_a], page1 = by_slot ? slot_a + 1 : p.s.slot_page[slot_a + 1];
        if (!by_slot && p.s.check_bounds) {      // a bad page id would only read the fill value (TMA clips), but say so
          if (!sr_check_page(p.s, page0)) page0 = 0;
          if (!sr_check_page(p.s, page1)) page1 = 0;
        }
        const bool gate = pt == n_pt;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.s.status)) { ok = false; break; }
          uint8_t* a_dst = smem + stage * STAGE2_BYTES;
          uint8_t* b_dst = a_dst + A2_BYTES;
          if (rank == 0) mbar_expect_tx(&full_bar[stage], 2 * STAGE2_BYTES);     // both CTAs' loads land on this barrier
          if (gate) tma_load_2d_pair(a_dst, mg, &full_bar[stage], kb * BK, rank * BM);
          else tma_load_2d_pair_hint(a_dst, mw, &full_bar[stage], kb * BK, p.w_row0 + pt * 2 * BM + rank * BM, w_policy);
          tma_load_4d_pair(b_dst, &map_x, &full_bar[stage], kb * BK, 0, pool_layer, page0);
          tma_load_4d_pair(b_dst + B2_BYTES / 2, &map_x, &full_bar[stage], kb * BK, 0, pool_layer, page1);
          if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
        }
        if (rank == 0 && p.mail) {
          const long long t = (long long)drawn + n_pairs;
          tile = t < total_tiles ? t : -1;
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      const uint32_t idesc = umma_idesc(2 * BM, BN, p.fp16_stage != 0);
      for (uint32_t seq = 1; ok; ++seq) {
        if (sched_get(p.mail, pair, seq, total_tiles, abort_flag, p.s.status) < 0) break;
        if (!mbar_wait(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, p.s.status)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * BN;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.s.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(smem + stage * STAGE2_BYTES);
          const uint64_t a_desc = umma_smem_desc(a_addr);
          const uint64_t b_desc = umma_smem_desc(a_addr + A2_BYTES);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&empty_bar[stage]);          // frees the stage in both CTAs
          if (++stage == STAGES2) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(&tfull_bar[acc]);              // accumulator complete, in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // epilogue: thread = channel (tensor-memory lane 32*(warp%4) + lane) of this CTA's 128 channels
    const int quarter = warp & 3;
    const int ch_local = quarter * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (uint32_t seq = 1;; ++seq) {
      int tile_lo = 0;
      if (lane == 0) tile_lo = (int)sched_get(p.mail, pair, seq, total_tiles, abort_flag, p.s.status);
      const long long tile = __shfl_sync(0xffffffffu, tile_lo, 0);
      if (tile < 0) break;
      int layer, pt, tt;
      tile_coords(tile, layer, pt, tt);
      FusedParams q = p;                                  // this tile's layer: its buffers, conv weights and history
      if constexpr (BATCHED) {
        const BatchLayer& bl = bt.layer[layer];
        q.conv_w = bl.conv_w;
        q.kv16 = bl.kv16;
        q.zraw = bl.zraw;
        q.gates = bl.gates;
        q.hist = bl.hist;
      }
      const bool gate = pt == n_pt;
      const int ct = 2 * pt + rank;                       // this CTA's 128-channel block
      const int ch = gate ? rank * BM + ch_local : ct * BM + ch_local;
      float cw[4] = {0.f, 0.f, 0.f, 0.f};
      if (!gate && ch < p.n_kv) {
        const uint2 wv = *(const uint2*)(q.conv_w + (long long)(p.n_q + ch) * SR_CONV_W);
        const __nv_bfloat16* e = (const __nv_bfloat16*)&wv;
#pragma unroll
        for (int q = 0; q < 4; ++q) cw[q] = __bfloat162float(e[q]);
      }
      float z1 = 0.f, z2 = 0.f, z3 = 0.f;
      if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag, p.s.status)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * BN;
#pragma unroll 1
      for (int sl = 0; sl < SLOTS; ++sl) {
        const int slot = SLOTS * tt + sl;
        float v[64];
        tmem_ld32(taddr + (uint32_t)(sl * 64), v);
        tmem_ld32(taddr + (uint32_t)(sl * 64 + 32), v + 32);
        if (sl == 0 || p.s.slot_first[slot]) load_history(q, gate, p.s.slot_first[slot], ch, z1, z2, z3);
        emit_slot(q, gate, ch, ch_local, ct, slot, sl == 0, p.s.slot_rows[slot], v, cw, z1, z2, z3);
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&tempty_bar[acc]);
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  cluster_sync_all();               // neither CTA leaves (or frees tensor memory) while the other may still signal it
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512));
  }
}

}  // namespace

bool sr_proj_fused_supported(const sr_ctx* ctx) {
  // any head geometry: the projection works on channels, in tiles of 128 (the last one may be partial)
  if (ctx->desc.d_model % BK != 0 || ctx->n_gate > 2 * BM) return false;
  if (ctx->desc.weight_format == SR_W_E4M3_BLOCK128) return ctx->desc.d_model % 128 == 0;
  return true;
}

// fp32 promotion of bare-code partial sums needs every 128-channel tile inside one row block of the scales
bool sr_proj_fused_exact_fp8_supported(const sr_ctx* ctx) {
  return ctx->n_k % BM == 0 && (ctx->n_k + ctx->n_v) % BM == 0 && ctx->n_gate <= BM;
}

cudaError_t sr_launch_proj_fused(const sr_ctx* ctx, const SrSched& s, const sr_anchor_pool& pool, int32_t pool_layer,
                                 const sr_layer_weights& w, const void* decoded, const SrFused& fused, int sm_count,
                                 cudaStream_t stream) {
  // block-scaled weights: the fp16 staging copies feed the plain kernels (`stage`), or bare codes with fp32 promotion
  // of the partial sums (`scaled`), or 8-bit operands on both sides (`a8`: quantised activations)
  const bool stage = ctx->fp16_stage;
  const bool a8 = ctx->w8a8;
  const bool scaled = ctx->desc.weight_format == SR_W_E4M3_BLOCK128 && !stage && !a8;
  if (scaled && !decoded) return cudaErrorInvalidValue;
  if (stage && (!fused.x16 || !fused.w16)) return cudaErrorInvalidValue;
  if (a8 && (!fused.x8 || !fused.sx)) return cudaErrorInvalidValue;
  const int d = ctx->desc.d_model;
  // channels this launch projects: k | v, or q | k | v for group replay (bf16 weights only)
  if (fused.with_q && (stage || a8 || scaled)) return cudaErrorInvalidValue;
  const int n_kv = fused.with_q ? ctx->conv_ch : ctx->n_k + ctx->n_v;
  const int ch0 = fused.with_q ? 0 : ctx->n_k;          // row of W_qkv / conv channel of projected channel 0
  CUtensorMap map_x, map_w, map_g;
  if (stage) {
    sr_anchor_pool staged = pool;                       // the layer's anchors in slot order: "page" = slot
    staged.base = fused.x16;
    staged.n_pool_layers = 1;
    staged.n_phys_pages = s.max_slots;
    staged.row_stride_bytes = (int64_t)d * 2;
    staged.layer_stride_bytes = (int64_t)SR_PAGE_ROWS * d * 2;
    staged.page_stride_bytes = (int64_t)SR_PAGE_ROWS * d * 2;
    if (!encode_pool_map(&map_x, staged, d, BK)) return cudaErrorInvalidValue;
    if (!encode_2d(&map_w, fused.w16, (uint64_t)d, (uint64_t)n_kv, (uint64_t)d * 2, BK, BM)) return cudaErrorInvalidValue;
    if (!encode_2d(&map_g, fused.w16 + (size_t)n_kv * d, (uint64_t)d, (uint64_t)ctx->n_gate, (uint64_t)d * 2, BK, BM))
      return cudaErrorInvalidValue;
  } else {
    if (!encode_pool_map(&map_x, pool, d, BK)) return cudaErrorInvalidValue;
    if (scaled) {
      if (!encode_2d(&map_w, decoded, (uint64_t)d, (uint64_t)n_kv, (uint64_t)d * 2, BK, BM)) return cudaErrorInvalidValue;
    } else if (!a8) {
      if (!encode_2d(&map_w, w.w_qkv, (uint64_t)d, (uint64_t)ctx->conv_ch, (uint64_t)d * 2, BK, BM)) return cudaErrorInvalidValue;
    }
    if (!encode_2d(&map_g, w.w_ab, (uint64_t)d, (uint64_t)ctx->n_gate, (uint64_t)d * 2, BK, BM)) return cudaErrorInvalidValue;
  }

  FusedParams p;
  p.s = s;
  p.pool_layer = stage ? 0 : pool_layer;
  p.fp16_stage = stage;
  p.slot_order = fused.x_slot_order;
  p.hist = fused.hist;
  p.conv_ch = ctx->conv_ch;
  p.k_blocks = d / BK;
  p.n_q = ch0;
  p.w_row0 = (scaled || stage) ? 0 : ch0;
  p.n_ct = (n_kv + BM - 1) / BM;
  p.n_gate = ctx->n_gate;
  p.ncb = fused.ncb;
  p.n_kv = n_kv;
  p.act_identity = ctx->desc.conv_activation == SR_CONV_IDENTITY;
  p.w_scale = (scaled || a8) ? w.w_qkv_scale : nullptr;
  p.scale_ld = d / 128;
  p.sx = nullptr;
  p.gate_only = 0;
  p.conv_w = (const __nv_bfloat16*)w.conv_w;
  p.kv16 = fused.kv16;
  p.zraw = fused.zraw;
  p.gates = fused.gates;
  p.group_c = 1;
  p.group_t = 1 << 30;
  p.next_tile = nullptr;
  p.mail = nullptr;

  cudaError_t once = sr_once_per_device(SR_ONCE_PROJ_FUSED, [] {
    cudaError_t e = cudaFuncSetAttribute(sr_proj_fused_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(sr_proj_fused_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(sr_proj_w8a8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, W8_SMEM_BYTES);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(sr_proj_fused2_kernel<NoBatch>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES);
    return e;
  });
  if (once != cudaSuccess) return once;
  const long long t_tiles = s.max_slots / SLOTS;
  // CTA pairs by default; the one-CTA form serves the block-scaled forms that promote partial sums and (on request) the tests
  const bool pair_form = !scaled && !a8 && sm_count >= 2 && (!(ctx->debug_flags & SR_DEBUG_SINGLE_CTA_MMA) || ctx->n_gate > BM);
  // Tile order: the channel tiles are cut into equal blocks of about WEIGHT_BLOCK_BYTES of weights; a block
  // stays in L2 while every token tile streams past it once (channel-fastest inside a block), so weights are
  // read from HBM once and anchors once per block.  Holding anchors instead and streaming the weights past
  // them costs more: measured 17.7 ms against 15.9 ms per launch at 254 400 tokens, d = 5120.
  {
    const long long c_tiles = pair_form ? (p.n_ct + 1) / 2 + 1 : (a8 ? p.n_ct : p.n_ct + 1);
    const long long tile_bytes = (long long)(pair_form ? 2 * BM : BM) * d * (a8 ? 1 : 2);
    const long long blocks = (c_tiles * tile_bytes + WEIGHT_BLOCK_BYTES - 1) / WEIGHT_BLOCK_BYTES;
    p.group_c = (int32_t)((c_tiles + blocks - 1) / blocks);
  }
  auto launch_pairs = [&](FusedParams pp, long long pair_tiles) {
    long long pairs = sm_count / 2;
    if (pair_tiles < pairs) pairs = pair_tiles;
    if (pairs > SR_SCHED_MAX_PAIRS) pairs = SR_SCHED_MAX_PAIRS;
    if (pairs < 1) pairs = 1;
    pp.next_tile = nullptr;
    pp.mail = nullptr;
    if (pair_tiles > pairs) {       // more than one tile per pair: tiles are handed out at run time
      if (!fused.tile_sched) return cudaErrorInvalidValue;
      cudaError_t e = cudaMemsetAsync(fused.tile_sched, 0, SR_TILE_SCHED_BYTES, stream);     // counter and mailboxes
      if (e != cudaSuccess) return e;
      pp.next_tile = (unsigned int*)fused.tile_sched;
      pp.mail = (unsigned long long*)((char*)fused.tile_sched + 256);
    }
    sr_proj_fused2_kernel<NoBatch><<<(unsigned)(2 * pairs), NUM_THREADS, SMEM2_BYTES, stream>>>(map_x, map_w, map_g, pp, NoBatch{});
    return cudaGetLastError();
  };
  if (pair_form) return launch_pairs(p, t_tiles * ((p.n_ct + 1) / 2 + 1));
  if (a8) {
    // (1) the bf16 gate rows on the unquantised anchors: the pair kernel restricted to its gate tile
    if (sm_count < 2) return cudaErrorNotSupported;
    FusedParams pg = p;
    pg.gate_only = 1;
    pg.w_scale = nullptr;
    map_w = map_g;                                       // not read: every tile of this launch is the gate tile
    cudaError_t e = launch_pairs(pg, t_tiles);
    if (e != cudaSuccess) return e;
    // (2) k | v on 8-bit operands: weight codes as stored, activation codes in slot order
    sr_anchor_pool staged = pool;
    staged.base = fused.x8;
    staged.n_pool_layers = 1;
    staged.n_phys_pages = s.max_slots;
    staged.row_stride_bytes = (int64_t)d;
    staged.layer_stride_bytes = (int64_t)SR_PAGE_ROWS * d;
    staged.page_stride_bytes = (int64_t)SR_PAGE_ROWS * d;
    if (!encode_pool_map(&map_x, staged, d, 2 * BK, true)) return cudaErrorInvalidValue;
    if (!encode_2d(&map_w, w.w_qkv, (uint64_t)d, (uint64_t)ctx->conv_ch, (uint64_t)d, 2 * BK, BM, true)) return cudaErrorInvalidValue;
    p.pool_layer = 0;
    p.k_blocks = d / (2 * BK);
    p.sx = fused.sx;
  }
  const long long max_tiles = a8 ? (long long)(s.max_slots / W8_SLOTS) * ((p.n_ct + 1) / 2) : t_tiles * (p.n_ct + 1);
  int grid = (int)(max_tiles < sm_count ? max_tiles : sm_count);
  if (grid < 1) grid = 1;
  if (a8) {
    if (grid > SR_SCHED_MAX_PAIRS) grid = SR_SCHED_MAX_PAIRS;
    if (max_tiles > grid) {         // more than one tile per CTA: tiles are handed out at run time
      if (!fused.tile_sched) return cudaErrorInvalidValue;
      cudaError_t e = cudaMemsetAsync(fused.tile_sched, 0, SR_TILE_SCHED_BYTES, stream);
      if (e != cudaSuccess) return e;
      p.next_tile = (unsigned int*)fused.tile_sched;
      p.mail = (unsigned long long*)((char*)fused.tile_sched + 256);
    }
    sr_proj_w8a8_kernel<<<grid, W8_THREADS, W8_SMEM_BYTES, stream>>>(map_x, map_w, p);
  }
  else if (scaled) sr_proj_fused_kernel<true><<<grid, NUM_THREADS_SCALED, SMEM_BYTES, stream>>>(map_x, map_w, map_g, p);
  else sr_proj_fused_kernel<false><<<grid, NUM_THREADS, SMEM_BYTES, stream>>>(map_x, map_w, map_g, p);
  return cudaGetLastError();
}

// Plain bf16 weights, state-only replay, and at most one wave of pair tiles per layer: the layers of such a call go
// through ONE launch (see BatchTable), up to sr_proj_fused_batch_max() of them at a time.
bool sr_proj_fused_batchable(const sr_ctx* ctx, int64_t max_slots, int sm_count) {
  if (ctx->desc.weight_format != SR_W_BF16 || ctx->fp16_stage || ctx->w8a8 || ctx->wdec_bytes) return false;
  if (ctx->debug_flags & SR_DEBUG_SINGLE_CTA_MMA) return false;
  const long long n_ct = (ctx->n_k + ctx->n_v + BM - 1) / BM;
  return sm_count >= 2 && (max_slots / SLOTS) * ((n_ct + 1) / 2 + 1) <= sm_count / 2;
}
int sr_proj_fused_batch_max() { return PROJ_BATCH_MAX; }

cudaError_t sr_launch_proj_fused_batch(const sr_ctx* ctx, const SrSched& s, const sr_anchor_pool& pool, int n,
                                       const int32_t* pool_layers, const sr_layer_weights* const* w, const SrFused* fused,
                                       int sm_count, cudaStream_t stream) {
  if (n < 1 || n > PROJ_BATCH_MAX || !sr_proj_fused_batchable(ctx, s.max_slots, sm_count)) return cudaErrorInvalidValue;
  const int d = ctx->desc.d_model;
  const int n_kv = ctx->n_k + ctx->n_v;
  CUtensorMap map_x;
  if (!encode_pool_map(&map_x, pool, d, BK)) return cudaErrorInvalidValue;
  BatchTable bt;
  bt.n_layers = n;
  for (int i = 0; i < n; ++i) {
    BatchLayer& bl = bt.layer[i];
    if (fused[i].with_q || fused[i].x_slot_order) return cudaErrorInvalidValue;
    if (!encode_2d(&bl.map_w, w[i]->w_qkv, (uint64_t)d, (uint64_t)ctx->conv_ch, (uint64_t)d * 2, BK, BM)) return cudaErrorInvalidValue;
    if (!encode_2d(&bl.map_g, w[i]->w_ab, (uint64_t)d, (uint64_t)ctx->n_gate, (uint64_t)d * 2, BK, BM)) return cudaErrorInvalidValue;
    bl.conv_w = (const __nv_bfloat16*)w[i]->conv_w;
    bl.kv16 = fused[i].kv16;
    bl.zraw = fused[i].zraw;
    bl.gates = fused[i].gates;
    bl.hist = fused[i].hist;
    bl.pool_layer = pool_layers[i];
  }
  FusedParams p;
  p.s = s;
  p.pool_layer = 0;
  p.fp16_stage = 0;
  p.slot_order = 0;
  p.hist = nullptr;
  p.conv_ch = ctx->conv_ch;
  p.k_blocks = d / BK;
  p.n_q = ctx->n_k;
  p.w_row0 = ctx->n_k;
  p.n_ct = (n_kv + BM - 1) / BM;
  p.n_gate = ctx->n_gate;
  p.ncb = fused[0].ncb;
  p.n_kv = n_kv;
  p.act_identity = ctx->desc.conv_activation == SR_CONV_IDENTITY;
  p.w_scale = nullptr;
  p.scale_ld = d / 128;
  p.sx = nullptr;
  p.gate_only = 0;
  p.conv_w = nullptr;
  p.kv16 = nullptr;
  p.zraw = nullptr;
  p.gates = nullptr;
  p.group_c = (p.n_ct + 1) / 2 + 1;      // one block: a layer's weights are its own L2 working set
  p.group_t = 1 << 30;
  p.next_tile = nullptr;
  p.mail = nullptr;
  cudaError_t e = sr_once_per_device(SR_ONCE_PROJ_FUSED2, [] {
    return cudaFuncSetAttribute(sr_proj_fused2_kernel<BatchTable>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM2_BYTES);
  });
  if (e != cudaSuccess) return e;
  const long long pair_tiles = (long long)n * (s.max_slots / SLOTS) * ((p.n_ct + 1) / 2 + 1);
  long long pairs = sm_count / 2;
  if (pair_tiles < pairs) pairs = pair_tiles;
  if (pairs > SR_SCHED_MAX_PAIRS) pairs = SR_SCHED_MAX_PAIRS;
  if (pairs < 1) pairs = 1;
  if (pair_tiles > pairs) {
    if (!fused[0].tile_sched) return cudaErrorInvalidValue;
    e = cudaMemsetAsync(fused[0].tile_sched, 0, SR_TILE_SCHED_BYTES, stream);
    if (e != cudaSuccess) return e;
    p.next_tile = (unsigned int*)fused[0].tile_sched;
    p.mail = (unsigned long long*)((char*)fused[0].tile_sched + 256);
  }
  CUtensorMap unused = map_x;              // the per-layer maps come from the table
  sr_proj_fused2_kernel<BatchTable><<<(unsigned)(2 * pairs), NUM_THREADS, SMEM2_BYTES, stream>>>(map_x, unused, unused, p, bt);
  return cudaGetLastError();
}
