// Batch packing on the device (Section 5.2, "Batched replay": the replay suffixes of a batch
// are packed into one variable-length execution and device-side boundaries identify each
// request's segment and destination state slot; padding segments carry a sentinel slot).
//
// One block validates every request, prefix-sums the page counts into "page slots" of the
// packed row space (slot s covers packed rows [64 s, 64 s + 64)), and records for each slot the
// physical pool page it reads.  Everything downstream indexes through these tables, so the
// replay lengths never have to be known on the host.
#include "sr_common.cuh"

namespace {

constexpr int kSchedThreads = 1024;

__global__ void __launch_bounds__(kSchedThreads)
sr_schedule_kernel(SrSched s, const int32_t* __restrict__ pages, const int32_t* __restrict__ state_slots,
                   const int32_t* __restrict__ replay_lens, int32_t max_pages, int32_t max_replay_len,
                   int64_t max_total_rows, int32_t n_phys_pages, int32_t n_state_slots) {
  __shared__ long long part_pages[kSchedThreads];
  __shared__ long long part_rows[kSchedThreads];
  __shared__ unsigned int flags;
  const int tid = threadIdx.x;
  const int B = s.n_requests;
  if (tid == 0) flags = 0u;
  __syncthreads();

  // 1. validate each request; req_rows <- rows, req_out <- destination (or -1), req_slot0 <- page count
  for (int i = tid; i < B; i += kSchedThreads) {
    int R = replay_lens[i];
    int out = state_slots ? state_slots[i] : i;
    unsigned int bad = 0u;
    if (out == -1) {            // sentinel: a padding segment, silently skipped
      R = 0;
    } else if (out < -1 || (n_state_slots > 0 && out >= n_state_slots)) {
      bad = SR_DEV_BAD_SLOT;
    } else if (R < 0 || R > max_replay_len) {
      bad = SR_DEV_BAD_REPLAY_LEN;
    } else {
      int n_pages = (R + SR_PAGE_ROWS - 1) / SR_PAGE_ROWS;
      for (int p = 0; p < n_pages; ++p) {
        int id = pages[(size_t)i * max_pages + p];
        if (id < 0 || id >= n_phys_pages) bad = SR_DEV_BAD_PAGE_ID;
      }
    }
    if (bad) {
      atomicOr(&flags, bad);
      R = 0;
      out = -1;
    }
    s.req_rows[i] = R;
    s.req_out[i] = out;
  }
  __syncthreads();

  // 2. exclusive prefix sums over requests (pages -> slot0, rows -> row0)
  const int per = (B + kSchedThreads - 1) / kSchedThreads;
  const int lo = min(B, tid * per), hi = min(B, lo + per);
  long long my_pages = 0, my_rows = 0;
  for (int i = lo; i < hi; ++i) {
    int R = s.req_rows[i];
    my_pages += (R + SR_PAGE_ROWS - 1) / SR_PAGE_ROWS;
    my_rows += R;
  }
  part_pages[tid] = my_pages;
  part_rows[tid] = my_rows;
  __syncthreads();
  for (int off = 1; off < kSchedThreads; off <<= 1) {
    long long a = 0, b = 0;
    if (tid >= off) { a = part_pages[tid - off]; b = part_rows[tid - off]; }
    __syncthreads();
    part_pages[tid] += a;
    part_rows[tid] += b;
    __syncthreads();
  }
  long long at_pages = part_pages[tid] - my_pages, at_rows = part_rows[tid] - my_rows;
  for (int i = lo; i < hi; ++i) {
    int R = s.req_rows[i];
    int n_pages = (R + SR_PAGE_ROWS - 1) / SR_PAGE_ROWS;
    if (at_pages + n_pages > (long long)s.max_slots || at_rows + R > max_total_rows) {
      // does not fit the bounds the caller sized the workspace for: treat as a miss
      atomicOr(&flags, SR_DEV_ROWS_OVERFLOW);
      s.req_rows[i] = 0;
      s.req_out[i] = -1;
      s.req_slot0[i] = 0;
      s.req_row0[i] = 0;
    } else {
      s.req_slot0[i] = (int)at_pages;
      s.req_row0[i] = (int)at_rows;
    }
    at_pages += n_pages;
    at_rows += R;
  }
  __syncthreads();

  // 3. requests by replay length, longest first: the state chains are launched in this order, so the
  //    long chains start first and the short ones fill the tail (rank by counting; ties by index)
  for (int i = tid; i < B; i += kSchedThreads) {
    const int R = s.req_rows[i];
    int rank = 0;
    for (int j = 0; j < B; ++j) {
      const int Rj = s.req_rows[j];
      rank += (Rj > R) || (Rj == R && j < i);
    }
    s.req_order[rank] = i;
  }

  // 4. per-slot tables
  const long long items = (long long)B * max_pages;
  for (long long it = tid; it < items; it += kSchedThreads) {
    int i = (int)(it / max_pages), p = (int)(it % max_pages);
    int R = s.req_rows[i];
    if (p * SR_PAGE_ROWS < R) {
      int slot = s.req_slot0[i] + p;
      s.slot_page[slot] = pages[(size_t)i * max_pages + p];
      s.slot_rows[slot] = min(SR_PAGE_ROWS, R - p * SR_PAGE_ROWS);
      s.slot_first[slot] = p == 0 ? i + 1 : 0;      // request index + 1 where the slot opens its request
    }
  }
  __syncthreads();
  if (tid == 0) {
    long long n_slots = 0, rows = 0;
    for (int i = B - 1; i >= 0; --i) {      // last request that kept its rows ends the packed space
      if (s.req_rows[i] > 0) {
        n_slots = s.req_slot0[i] + (s.req_rows[i] + SR_PAGE_ROWS - 1) / SR_PAGE_ROWS;
        rows = (long long)s.req_row0[i] + s.req_rows[i];
        break;
      }
    }
    // the projection walks slots in groups of up to four: pad the last group with harmless slots
    for (long long q = n_slots; (q & 3) && q < s.max_slots; ++q) {
      s.slot_page[q] = n_slots > 0 ? s.slot_page[n_slots - 1] : 0;
      s.slot_rows[q] = 0;
      s.slot_first[q] = 1;
    }
    s.status[0] = flags;
    s.status[1] = (uint32_t)n_slots;
    s.status[2] = (uint32_t)rows;
  }
}

__global__ void __launch_bounds__(256)
sr_debug_gather_kernel(SrSched s, SrPoolView pool, int32_t pool_layer, int32_t d_model,
                       __nv_bfloat16* __restrict__ out, int64_t capacity_rows) {
  // one block per (request, page of the request); 16-byte vector copies, a row at a time per warp
  const int i = blockIdx.y;
  const int R = s.req_rows[i];
  const int p = blockIdx.x;
  if (p * SR_PAGE_ROWS >= R) return;
  const int slot = s.req_slot0[i] + p;
  if (!sr_check_slot(s, slot) || !sr_check_page(s, s.slot_page[slot])) return;
  const int rows = s.slot_rows[slot];
  const char* src = pool.base + (int64_t)s.slot_page[slot] * pool.page_stride + (int64_t)pool_layer * pool.layer_stride;
  const int64_t row0 = (int64_t)s.req_row0[i] + (int64_t)p * SR_PAGE_ROWS;
  const int vec_per_row = d_model / 8;     // 8 bf16 = 16 bytes
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = warp; r < rows; r += 8) {
    if (row0 + r >= capacity_rows) continue;
    const uint4* a = (const uint4*)(src + (int64_t)r * pool.row_stride);
    uint4* b = (uint4*)(out + (row0 + r) * (int64_t)d_model);
    for (int v = lane; v < vec_per_row; v += 32) b[v] = a[v];
  }
}

}  // namespace

cudaError_t sr_launch_schedule(const SrSched& s, const int32_t* pages, const int32_t* state_slots,
                               const int32_t* replay_lens, int32_t max_pages, int32_t max_replay_len,
                               int64_t max_total_rows, int32_t n_phys_pages, int32_t n_state_slots,
                               cudaStream_t stream) {
  sr_schedule_kernel<<<1, kSchedThreads, 0, stream>>>(s, pages, state_slots, replay_lens, max_pages,
                                                      max_replay_len, max_total_rows, n_phys_pages, n_state_slots);
  return cudaGetLastError();
}

cudaError_t sr_launch_debug_gather(const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                   int32_t d_model, int32_t max_pages, void* out_rows,
                                   int64_t out_capacity_rows, cudaStream_t stream) {
  dim3 grid((unsigned)max_pages, (unsigned)s.n_requests);
  sr_debug_gather_kernel<<<grid, 256, 0, stream>>>(s, pool, pool_layer, d_model, (__nv_bfloat16*)out_rows,
                                                   out_capacity_rows);
  return cudaGetLastError();
}
