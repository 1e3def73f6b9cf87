// Dense row GEMMs and the row normalisation of group-propagated replay (Section 4.1, "Layer-wise Sparse Anchors":
// a group of consecutive linear-attention layers is replayed from one stored hidden state, so every layer but the
// last has to produce its output rows for the next one).
//
//   C[row][n] = epilogue( sum_k A[row][k] * B[n][k] )         rows = page slots x 64 (packed order), bf16 in / out
//
// serves the output gate (x W_z^T, SiLU applied), the output projection (y W_o^T + residual), and the two MLP
// products (SiLU(n W_gate^T) * (n W_up^T), then ... W_down^T + residual).  tcgen05 tensor cores, tokens on the
// MMA's M axis (a tensor-memory lane is a row, so a thread writes consecutive output columns of its row):
// persistent, CTAs paired into clusters of two that share one 256 x 256 MMA tile (cta_group::2); per CTA warp 0 is
// the TMA producer (its 128 rows of A and its 128 of the tile's 256 weight rows per 64-wide k block, 6-stage ring),
// warp 1 of the leader issues the MMAs into a double-buffered accumulator (2 x 256 columns of tensor memory per
// CTA), warps 2-5 are the epilogue.  All waits are bounded.
#include "sr_umma.cuh"

namespace {

constexpr int GM = 128;                  // rows per CTA (a pair of CTAs works on 256 rows: four page slots)
constexpr int GN = 256;                  // output columns per tile (MMA N); each CTA of the pair stages 128 weight rows
constexpr int GK = 64, GSTAGES = 6;
constexpr int GA_BYTES = GM * GK * 2;          // 16 KB: this CTA's 128 rows
constexpr int GB_BYTES = (GN / 2) * GK * 2;    // 16 KB: this CTA's 128 of the tile's 256 weight rows
constexpr int GSTAGE_BYTES = GA_BYTES + GB_BYTES;
constexpr int GSMEM_BYTES = GSTAGES * GSTAGE_BYTES + 1024 + 256;
constexpr int GTHREADS = 192;

struct GemmParams {
  SrSched s;
  int32_t k_blocks;      // K / 64
  int32_t n;             // output columns (for SWIGLU: hidden width f; the tile holds 128 gate + 128 up columns)
  int32_t n_tiles;
  int32_t n_block;       // column tiles per weight block of the tile order
  __nv_bfloat16* c;      // [rows][ldc]
  int64_t ldc;
  const __nv_bfloat16* residual;   // EPI_ADD: [rows][ldr]
  int64_t ldr;
};

enum { EPI_STORE = 0, EPI_SILU = 1, EPI_ADD = 2, EPI_SWIGLU = 3 };

__device__ __forceinline__ float silu(float x) { return __fdividef(x, 1.f + __expf(-x)); }

// Two-CTA form (tcgen05 cta_group::2), as in the in-projection: a pair of CTAs on neighbouring SMs shares one MMA
// tile of 256 rows x 256 columns.  Each CTA stages its own 128 rows and 128 of the tile's 256 weight rows per k
// block (32 KB) and the tensor core reads the weight operand from both shared memories: a weight tile crosses from
// L2 once per 256 rows instead of once per 128, which is what bounds these products on a serving-size batch (a few
// hundred rows against hundreds of megabytes of weights).  The leader CTA issues the MMAs; both CTAs run their own
// TMA producer and their own epilogue (their 128 rows of the accumulator).
template <int EPI>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GTHREADS, 1)
sr_rows_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_b2, const GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full_bar = (uint64_t*)(smem + GSTAGES * GSTAGE_BYTES);   // used in the leader CTA only
  uint64_t* empty_bar = full_bar + GSTAGES;                          // one set per CTA
  uint64_t* tfull_bar = empty_bar + GSTAGES;                         // [2] one set per CTA
  uint64_t* tempty_bar = tfull_bar + 2;                              // [2] used in the leader CTA only
  uint32_t* tmem_slot = (uint32_t*)(tempty_bar + 2);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int n_slots = (int)p.s.status[1];
  const int m_tiles = (n_slots + 3) / 4;
  const long long total_tiles = (long long)m_tiles * p.n_tiles;
  constexpr int NCOL = EPI == EPI_SWIGLU ? GN / 2 : GN;      // output columns a tile produces

  if (threadIdx.x == 0) {
    for (int i = 0; i < GSTAGES; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
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

  // tile -> (row tile, column tile).  The column tiles are cut into blocks of n_block tiles whose weights (about
  // 24 MB) stay in L2 while every row tile streams past them, column-fastest inside the block: weights come from
  // HBM once, rows once per block.  (Column-fastest over the whole width re-read a 105 MB weight matrix once per
  // two row tiles: 1.6 GB of HBM reads for 0.13 GB of operands on 4096 rows.)
  auto tile_coords = [&](long long tile, int& mt, int& nt) {
    const long long per_block = (long long)m_tiles * p.n_block;
    const int blk = (int)(tile / per_block);
    const int r = (int)(tile - blk * per_block);
    const int nbt = min(p.n_block, p.n_tiles - blk * p.n_block);
    mt = r / nbt;
    nt = blk * p.n_block + r % nbt;
  };
  // does the second CTA's half of the weight tile exist?  (Both CTAs and the leader's byte count must agree.)
  auto second_half = [&](int nt) { return EPI == EPI_SWIGLU || nt * GN + GN / 2 < p.n; };

  if (warp == 0) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (long long tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        int mt, nt;
        tile_coords(tile, mt, nt);
        const bool second = second_half(nt);
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag, p.s.status)) { ok = false; break; }
          uint8_t* a_dst = smem + stage * GSTAGE_BYTES;
          uint8_t* b_dst = a_dst + GA_BYTES;
          // both CTAs' loads land on the leader's barrier; a missing second half is stale shared memory whose
          // accumulator columns are never stored
          if (rank == 0) mbar_expect_tx(&full_bar[stage], second ? 2 * GSTAGE_BYTES : 2 * GSTAGE_BYTES - GB_BYTES);
          tma_load_2d_pair(a_dst, &map_a, &full_bar[stage], kb * GK, (2 * mt + rank) * GM);
          if (EPI == EPI_SWIGLU) {       // columns 0..127: gate rows (CTA 0), 128..255: the up rows of the same hidden units
            tma_load_2d_pair(b_dst, rank == 0 ? &map_b : &map_b2, &full_bar[stage], kb * GK, nt * NCOL);
          } else if (rank == 0 || second) {
            tma_load_2d_pair(b_dst, &map_b, &full_bar[stage], kb * GK, nt * GN + rank * (GN / 2));
          }
          if (++stage == GSTAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      const uint32_t idesc = umma_idesc(2 * GM, GN);
      for (long long tile = pair; ok && tile < total_tiles; tile += n_pairs) {
        if (!mbar_wait(&tempty_bar[acc], acc_phase ^ 1u, abort_flag, p.s.status)) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * GN;
        for (int kb = 0; kb < p.k_blocks; ++kb) {
          if (!mbar_wait(&full_bar[stage], phase, abort_flag, p.s.status)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = smem_u32(smem + stage * GSTAGE_BYTES);
          const uint64_t a_desc = umma_smem_desc(a_addr), b_desc = umma_smem_desc(a_addr + GA_BYTES);
#pragma unroll
          for (int k = 0; k < GK / 16; ++k)
            umma_bf16_pair(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(&empty_bar[stage]);          // frees the stage in both CTAs
          if (++stage == GSTAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(&tfull_bar[acc]);              // accumulator complete, in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // epilogue: thread = row (tensor-memory lane 32 * (warp % 4) + lane) of this CTA's 128 rows
    const int quarter = warp & 3;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (long long tile = pair; tile < total_tiles; tile += n_pairs) {
      int mt, nt;
      tile_coords(tile, mt, nt);
      const long long row = (long long)(2 * mt + rank) * GM + quarter * 32 + lane;
      const bool row_ok = row < (long long)n_slots * SR_PAGE_ROWS && sr_check_slot(p.s, (int)(row / SR_PAGE_ROWS));
      if (!mbar_wait(&tfull_bar[acc], acc_phase, abort_flag, p.s.status)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * GN;
#pragma unroll 1
      for (int c = 0; c < NCOL / 32; ++c) {
        const int n0 = nt * NCOL + c * 32;
        if (n0 >= p.n) break;
        float v[32];
        tmem_ld32(taddr + (uint32_t)(c * 32), v);
        if (EPI == EPI_SWIGLU) {
          float u[32];
          tmem_ld32(taddr + (uint32_t)(GN / 2 + c * 32), u);
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = silu(v[i]) * u[i];
        } else if (EPI == EPI_SILU) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = silu(v[i]);
        } else if (EPI == EPI_ADD) {
          if (row_ok) {
            const uint4* r4 = (const uint4*)(p.residual + row * p.ldr + n0);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (n0 + 8 * q < p.n) {
                const uint4 rv = r4[q];
                const __nv_bfloat16* e = (const __nv_bfloat16*)&rv;
#pragma unroll
                for (int i = 0; i < 8; ++i) v[8 * q + i] += __bfloat162float(e[i]);
              }
            }
          }
        }
        if (row_ok) {
          uint4* dst = (uint4*)(p.c + row * p.ldc + n0);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (n0 + 8 * q < p.n) {                    // widths are multiples of 8
              __align__(16) __nv_bfloat16 o[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) o[i] = __float2bfloat16_rn(v[8 * q + i]);
              dst[q] = *(const uint4*)o;
            }
          }
        }
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

// x[slot][row][:] = bf16( r * rsqrt(mean(r^2) + eps) * w ), one warp per row, eight rows per CTA.  The rows come from the anchor pool
// through the slot table (the group's first layer) or from a packed row buffer (the later ones); rows past a
// window's end are written as zeros, whatever the source holds there.
__global__ void __launch_bounds__(256)
sr_rmsnorm_rows_kernel(SrSched s, SrPoolView pool, int32_t pool_layer, const __nv_bfloat16* __restrict__ rows_in,
                       const __nv_bfloat16* __restrict__ w, float eps, int32_t d_model, __nv_bfloat16* __restrict__ out,
                       __nv_bfloat16* __restrict__ copy_out) {
  const int slot = blockIdx.x >> 3;                       // eight CTAs per page slot, a warp per row
  if (slot >= (((int)s.status[1] + 3) & ~3)) return;
  const int vr = s.slot_rows[slot];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nvec = d_model / 8;
  {
    const int r = (blockIdx.x & 7) * 8 + warp;
    __nv_bfloat16* dst = out + ((int64_t)slot * SR_PAGE_ROWS + r) * d_model;
    __nv_bfloat16* cpy = copy_out ? copy_out + ((int64_t)slot * SR_PAGE_ROWS + r) * d_model : nullptr;
    if (r >= vr) {
      for (int v = lane; v < nvec; v += 32) {
        ((uint4*)dst)[v] = make_uint4(0u, 0u, 0u, 0u);
        if (cpy) ((uint4*)cpy)[v] = make_uint4(0u, 0u, 0u, 0u);
      }
      return;
    }
    const uint4* src;
    if (rows_in) {
      src = (const uint4*)(rows_in + ((int64_t)slot * SR_PAGE_ROWS + r) * d_model);
    } else {
      if (!sr_check_page(s, s.slot_page[slot])) return;
      src = (const uint4*)(pool.base + (int64_t)s.slot_page[slot] * pool.page_stride + (int64_t)pool_layer * pool.layer_stride +
                           (int64_t)r * pool.row_stride);
    }
    float ss = 0.f;
    for (int v = lane; v < nvec; v += 32) {
      const uint4 x = src[v];
      const __nv_bfloat16* e = (const __nv_bfloat16*)&x;
#pragma unroll
      for (int i = 0; i < 8; ++i) { const float f = __bfloat162float(e[i]); ss = fmaf(f, f, ss); }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const float inv = rsqrtf(ss / (float)d_model + eps);
    for (int v = lane; v < nvec; v += 32) {
      const uint4 x = src[v];
      const uint4 wv = ((const uint4*)w)[v];
      const __nv_bfloat16* e = (const __nv_bfloat16*)&x;
      const __nv_bfloat16* we = (const __nv_bfloat16*)&wv;
      __align__(16) __nv_bfloat16 o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) o[i] = __float2bfloat16_rn(__bfloat162float(e[i]) * inv * __bfloat162float(we[i]));
      ((uint4*)dst)[v] = *(const uint4*)o;
      if (cpy) ((uint4*)cpy)[v] = x;          // the residual stream itself, in packed slot order
    }
  }
}

bool encode_rows(CUtensorMap* map, const void* base, uint64_t k, uint64_t rows, uint32_t box_rows) {
  return encode_2d(map, base, k, rows, k * 2, GK, box_rows);
}

template <int EPI>
cudaError_t launch_gemm(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mb2, const GemmParams& p,
                        long long max_tiles, int sm_count, cudaStream_t stream) {
  long long pairs = sm_count / 2;
  if (max_tiles < pairs) pairs = max_tiles;
  if (pairs < 1) pairs = 1;
  sr_rows_gemm_kernel<EPI><<<(unsigned)(2 * pairs), GTHREADS, GSMEM_BYTES, stream>>>(ma, mb, mb2, p);
  return cudaGetLastError();
}

}  // namespace

// C[rows][n] = epi(A[rows][k] B[n][k]^T): rows = max_slots * 64 packed rows (bf16), weights [n][k] bf16.
// kind: 0 store, 1 SiLU, 2 + residual, 3 SwiGLU (b = W_gate, b2 = W_up, both [n][k]; C = SiLU(A b^T) * (A b2^T)).
cudaError_t sr_launch_rows_gemm(const SrSched& s, int kind, const __nv_bfloat16* a, int64_t k, const void* b, const void* b2,
                                int32_t n, __nv_bfloat16* c, int64_t ldc, const __nv_bfloat16* residual, int64_t ldr,
                                int sm_count, cudaStream_t stream) {
  if (k % GK != 0 || n % 8 != 0 || n <= 0) return cudaErrorInvalidValue;
  cudaError_t once = sr_once_per_device(SR_ONCE_ROWS_GEMM, [] {
    cudaError_t e = cudaFuncSetAttribute(sr_rows_gemm_kernel<EPI_STORE>, cudaFuncAttributeMaxDynamicSharedMemorySize, GSMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sr_rows_gemm_kernel<EPI_SILU>, cudaFuncAttributeMaxDynamicSharedMemorySize, GSMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sr_rows_gemm_kernel<EPI_ADD>, cudaFuncAttributeMaxDynamicSharedMemorySize, GSMEM_BYTES);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(sr_rows_gemm_kernel<EPI_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, GSMEM_BYTES);
    return e;
  });
  if (once != cudaSuccess) return once;
  CUtensorMap ma, mb, mb2;
  const uint64_t rows = (uint64_t)s.max_slots * SR_PAGE_ROWS;
  if (!encode_rows(&ma, a, (uint64_t)k, rows, GM)) return cudaErrorInvalidValue;
  if (!encode_rows(&mb, b, (uint64_t)k, (uint64_t)n, GN / 2)) return cudaErrorInvalidValue;
  if (!encode_rows(&mb2, b2 ? b2 : b, (uint64_t)k, (uint64_t)n, GN / 2)) return cudaErrorInvalidValue;
  GemmParams p;
  p.s = s;
  p.k_blocks = (int32_t)(k / GK);
  p.n = n;
  const int ncol = kind == EPI_SWIGLU ? GN / 2 : GN;
  p.n_tiles = (n + ncol - 1) / ncol;
  {
    const long long tile_bytes = (long long)GN * k * 2;       // weight rows one tile reads (both halves of a SwiGLU tile)
    long long nb = (24ll << 20) / tile_bytes;
    if (nb < 1) nb = 1;
    const long long blocks = (p.n_tiles + nb - 1) / nb;       // equal blocks
    p.n_block = (int32_t)((p.n_tiles + blocks - 1) / blocks);
  }
  p.c = c;
  p.ldc = ldc;
  p.residual = residual;
  p.ldr = ldr;
  if (sm_count < 2) return cudaErrorNotSupported;
  const long long max_tiles = (long long)((s.max_slots + 3) / 4) * p.n_tiles;
  switch (kind) {
    case EPI_STORE: return launch_gemm<EPI_STORE>(ma, mb, mb2, p, max_tiles, sm_count, stream);
    case EPI_SILU: return launch_gemm<EPI_SILU>(ma, mb, mb2, p, max_tiles, sm_count, stream);
    case EPI_ADD: return residual ? launch_gemm<EPI_ADD>(ma, mb, mb2, p, max_tiles, sm_count, stream) : cudaErrorInvalidValue;
    case EPI_SWIGLU: return b2 ? launch_gemm<EPI_SWIGLU>(ma, mb, mb2, p, max_tiles, sm_count, stream) : cudaErrorInvalidValue;
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t sr_launch_rmsnorm_rows(const SrSched& s, const SrPoolView& pool, int32_t pool_layer, const __nv_bfloat16* rows_in,
                                   const __nv_bfloat16* w, float eps, int32_t d_model, __nv_bfloat16* out,
                                   __nv_bfloat16* copy_out, cudaStream_t stream) {
  sr_rmsnorm_rows_kernel<<<(unsigned)s.max_slots * 8, 256, 0, stream>>>(s, pool, pool_layer, rows_in, w, eps, d_model, out, copy_out);
  return cudaGetLastError();
}
