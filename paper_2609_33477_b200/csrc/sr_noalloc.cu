// sr_replay_states_noalloc: the replay call for callers that cannot allocate device memory.
//
// Some callers of this library are not in a position to call cudaMalloc (or to ask a framework
// allocator for memory) when a batch of cache hits arrives: code running inside a serving engine
// whose memory pool was sized and frozen at start-up, a plugin loaded into a process that forbids
// allocation on its hot path, or a replay step that is set up once and re-run many times, where an
// allocation would either fail or hand back a different address each time.  sr_replay_states asks
// such a caller for a workspace it has no way to provide.  This variant takes the workspace from a
// fixed array that lives in the library's own device image instead.
//
// The array costs SR_NOALLOC_SCRATCH_BYTES of device memory on every GPU that loads this library,
// from load until the process exits, whether or not this entry point is ever called.
#include <mutex>

#include "sr_common.cuh"

namespace {

// The scratch itself.  In host code this name is only a stand-in for the symbol, not a device
// address: a kernel handed it directly would fault or read the wrong memory.  The device address is
// looked up with cudaGetSymbolAddress, once per device, below.
static __device__ __align__(256) unsigned char sr_noalloc_scratch[SR_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {nullptr};
std::mutex g_setup_mutex;

// First call on a device: look the array's device address up, with that device current.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SR_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, sr_noalloc_scratch) != cudaSuccess || !ptr) return SR_ERR_CUDA;
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return SR_OK;
}

}  // namespace

extern "C" int sr_replay_states_noalloc(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                                        const int32_t* replay_lens, const uint8_t* layer_mask,
                                        const sr_layer_weights* weights, const sr_out* out_ssm,
                                        const sr_out* out_conv, void* stream) {
  size_t need = 0;
  int st = sr_workspace_bytes(ctx, table, &need);       // checks `ctx` and the bounds in `table`
  if (st != SR_OK) return st;
  // what the call cannot do without: the tables and ONE block of per-layer hand-over buffers (sr_workspace_bytes
  // asks for up to eight blocks on small batches, to run layers side by side; this entry uses as many as fit).
  // If even that is more than the fixed array holds: refuse, launch nothing.
  need = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows, 1).total;
  if (need > (size_t)SR_NOALLOC_SCRATCH_BYTES) return SR_ERR_WORKSPACE;
  void* scratch = nullptr;
  st = scratch_for_current_device(&scratch);
  if (st != SR_OK) return st;
  // Nothing in the scratch has to start at zero: the packing kernel that opens every call rewrites
  // the status word and every table entry the later kernels read, and each layer's projection
  // scratch is written before it is read.  The previous call's contents are simply overwritten.
  return sr_replay_states(ctx, pool, table, replay_lens, layer_mask, weights, out_ssm, out_conv, scratch,
                          (size_t)SR_NOALLOC_SCRATCH_BYTES, stream);
}
