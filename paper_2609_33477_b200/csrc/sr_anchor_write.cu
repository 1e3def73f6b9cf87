// Anchor write path (Section 5.1, "Writing anchors"): the host builds a destination table for the step, and
// indexed copies inside the step's graph write the selected hidden states straight to their sidecar rows;
// positions that are not sampled carry a scratch address and are ignored.
//
//   for every token t with dest_page[t] >= 0, for every written layer w:
//     pool[dest_page[t]][pool_layer[w]][dest_row[t]][0:d] = hidden[w][t][0:d]
//
// One warp per (token, layer): the destination is read first, so rows that are not sampled cost one 4-byte load
// (the compaction of a prefill step happens here, not in a separate pass); a row moves as 16-byte vectors.
// A destination outside the pool is skipped and flagged, never written.
#include "sr_common.cuh"

namespace {

constexpr int WRITE_THREADS = 256;
constexpr int MAX_WRITE_LAYERS = 64;

struct WriteLayers {
  int32_t pool_layer[MAX_WRITE_LAYERS];
};

__global__ void __launch_bounds__(WRITE_THREADS)
sr_anchor_write_kernel(char* __restrict__ pool_base, int64_t page_stride, int64_t layer_stride, int64_t row_stride,
                       int32_t n_phys_pages, WriteLayers layers, const char* __restrict__ hidden,
                       int64_t hidden_layer_stride, int64_t hidden_row_stride, const int32_t* __restrict__ dest_page,
                       const int32_t* __restrict__ dest_row, int32_t n_tokens, int32_t row_bytes,
                       uint32_t* __restrict__ status) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int t = blockIdx.x * (WRITE_THREADS / 32) + warp;
  if (t >= n_tokens) return;
  const int page = dest_page[t];
  if (page < 0) return;                                  // scratch address: not sampled
  const int row = dest_row[t];
  if (page >= n_phys_pages || row < 0 || row >= SR_PAGE_ROWS) {
    if (lane == 0 && status) atomicOr(status, SR_DEV_BAD_PAGE_ID);
    return;
  }
  const int w = blockIdx.y;
  const uint4* src = (const uint4*)(hidden + (int64_t)w * hidden_layer_stride + (int64_t)t * hidden_row_stride);
  uint4* dst = (uint4*)(pool_base + (int64_t)page * page_stride + (int64_t)layers.pool_layer[w] * layer_stride +
                        (int64_t)row * row_stride);
  const int n_vec = row_bytes / 16;
  int i = lane;
  for (; i + 96 < n_vec; i += 128) {                     // four loads in flight per lane
    const uint4 a = __ldcs(src + i), b = __ldcs(src + i + 32), c = __ldcs(src + i + 64), e = __ldcs(src + i + 96);
    dst[i] = a;
    dst[i + 32] = b;
    dst[i + 64] = c;
    dst[i + 96] = e;
  }
  for (; i < n_vec; i += 32) dst[i] = __ldcs(src + i);
}

}  // namespace

cudaError_t sr_launch_anchor_write(const sr_anchor_pool& pool, const int32_t* pool_layers, int32_t n_layers,
                                   const void* hidden, int64_t hidden_layer_stride, int64_t hidden_row_stride,
                                   const int32_t* dest_page, const int32_t* dest_row, int32_t n_tokens, int32_t d_model,
                                   uint32_t* status, cudaStream_t stream) {
  for (int32_t l0 = 0; l0 < n_layers; l0 += MAX_WRITE_LAYERS) {
    const int32_t n = n_layers - l0 < MAX_WRITE_LAYERS ? n_layers - l0 : MAX_WRITE_LAYERS;
    WriteLayers wl;
    for (int32_t i = 0; i < n; ++i) wl.pool_layer[i] = pool_layers[l0 + i];
    dim3 grid((unsigned)((n_tokens + WRITE_THREADS / 32 - 1) / (WRITE_THREADS / 32)), (unsigned)n);
    sr_anchor_write_kernel<<<grid, WRITE_THREADS, 0, stream>>>(
        (char*)pool.base, pool.page_stride_bytes, pool.layer_stride_bytes, pool.row_stride_bytes, pool.n_phys_pages, wl,
        (const char*)hidden + (int64_t)l0 * hidden_layer_stride, hidden_layer_stride, hidden_row_stride, dest_page,
        dest_row, n_tokens, d_model * 2, status);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}
