// Shared declarations of the suffix-replay CUDA library: context, workspace layout and the
// host-side launch functions each kernel file exports.  Internal; the public boundary is
// include/sr_replay.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "sr_replay.h"

#define SR_PAGE_ROWS 64
#define SR_CONV_W 4
#define SR_MAX_LANES 8                       // streams a call spreads its layers over on small batches
#define SR_MAX_BLOCKS 32                     // blocks of per-layer hand-over buffers (layers whose buffers are alive at once)
#define SR_LANES_BUDGET_BYTES (1024ull << 20) // ... as long as their hand-over buffers together stay below this

struct sr_ctx {
  sr_model_desc desc;
  int n_k;        // H_k * d_k   (key columns of the projection)
  int n_v;        // H_v * d_v   (value columns)
  int n_gate;     // 2 * H_v     (decay and write-strength columns)
  int conv_ch;    // C = 2 H_k d_k + H_v d_v
  int64_t last_launches;
  bool kernels_cover;  // false: sizes can be queried but no kernel serves this geometry
  size_t wdec_bytes;   // workspace bytes for decoded e4m3 codes (0 for bf16 weights)
  bool fp16_stage;     // block-scaled weights on the fused path: weights dequantised and anchors converted to fp16
                       // once per layer, then the same tensor-core kernel as for bf16 weights (SR_DEBUG_FP8_EXACT
                       // selects fp32 promotion of bare-code partial sums instead)
  uint32_t debug_flags;  // desc.debug_flags (SR_DEBUG_*)
  bool w8a8;             // e4m3 weights x on-the-fly e4m3 activations on the 8-bit tensor-core path
  // optional per-kernel timing (sr_profile_*): events bracketing every launch of the last call
  bool profiling;
  std::vector<cudaEvent_t> ev_pool;   // created on demand, reused, destroyed with the context
  // small batches: layers are independent, so up to SR_MAX_LANES of them run side by side on streams of the
  // context (lane 0 is the caller's stream); created at the first call that uses them
  cudaStream_t lane_stream[SR_MAX_LANES - 1];
  cudaEvent_t lane_fork, lane_join[SR_MAX_LANES - 1];
  bool lanes_ready;
  // sr_replay_states_host only: two copy streams and their events, created at its first call
  cudaStream_t copy_in, copy_out;
  std::vector<cudaEvent_t> ev_copy;
  std::vector<int> ev_kind;           // kernel kind of bracket i (events 2i, 2i+1)
  size_t ev_used;
};

// Counts the kernel launches of one step and, when profiling is on, brackets them with two events on `stream`.
struct SrLaunchScope {
  sr_ctx* ctx;
  cudaStream_t stream;
  bool armed;
  SrLaunchScope(sr_ctx* c, cudaStream_t s, int kind, int kernels = 1) : ctx(c), stream(s), armed(false) {
    ctx->last_launches += kernels;
    if (!ctx->profiling) return;
    while (ctx->ev_pool.size() < ctx->ev_used + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return;
      ctx->ev_pool.push_back(e);
    }
    if (cudaEventRecord(ctx->ev_pool[ctx->ev_used], stream) != cudaSuccess) return;
    ctx->ev_kind.push_back(kind);
    armed = true;
  }
  ~SrLaunchScope() {
    if (!armed) return;
    cudaEventRecord(ctx->ev_pool[ctx->ev_used + 1], stream);
    ctx->ev_used += 2;
  }
};

// Per-device one-time set-up (kernel attributes are per device, and several host threads may make their first
// call at once): runs `setup` with the current device the first time `key` is seen on it, under a lock; later
// calls return cudaSuccess at once.  A failed set-up is retried by the next call.
enum SrOnceKey {
  SR_ONCE_PROJ_FUSED = 0, SR_ONCE_PROJ_FUSED2, SR_ONCE_CHUNK_LOCAL_64, SR_ONCE_CHUNK_LOCAL_96,
  SR_ONCE_CHUNK_LOCAL_128, SR_ONCE_CHAIN_UMMA, SR_ONCE_CONV_GEMM, SR_ONCE_ROWS_GEMM, SR_ONCE_GROUP_OUT_64, SR_ONCE_GROUP_OUT_96,
  SR_ONCE_GROUP_OUT_128, SR_ONCE_KEYS
};
cudaError_t sr_once_per_device(int key, cudaError_t (*setup)());
// SM count of the current device (looked up once per device)
cudaError_t sr_current_device_sms(int* sms);
// Creates the context's side streams and fork / join events at first use (outside any stream capture).
bool sr_ensure_lanes(sr_ctx* ctx);

// Scratch layout inside the caller's workspace (all offsets in bytes, 256-aligned).
struct sr_ctx;
size_t sr_scan_split_bytes(const sr_ctx* ctx, int64_t max_slots);
size_t sr_conv_tail_part_bytes(const sr_ctx* ctx);

struct SrWorkspace {
  size_t off_header;     // uint32 status, int32 n_slots, int32 total_rows
  size_t off_req_rows;   // int32 [B]   rows to replay (0 for skipped / sentinel requests)
  size_t off_req_slot0;  // int32 [B]   first page slot of the request in the packed row space
  size_t off_req_out;    // int32 [B]   destination state slot, -1 = write nothing
  size_t off_req_row0;   // int32 [B]   first packed row (no page padding) for the debug gather
  size_t off_req_order;  // int32 [B]   request indices, longest replay first (launch order of the state chains)
  size_t off_slot_page;  // int32 [max_slots] physical page of each page slot
  size_t off_slot_rows;  // int32 [max_slots] valid rows in the slot (1..64)
  size_t off_slot_first; // int32 [max_slots] request index + 1 where the slot opens its request, else 0
  size_t off_kv16;       // half [max_slots][ncb * 128][64] conv + SiLU outputs, one layer at a time
  size_t off_zraw;       // float [max_slots][6][n_k+n_v] raw projection rows 0,1,2 | last 3 valid
  size_t off_z;          // float [max_slots][2 H_v][64] raw gate pre-activations, one layer at a time
  size_t off_split;      // per (slot, head) T matrices (fp16) and row factors handed from the chunk-local
                         // kernel to the chain kernel
  size_t off_wdec;       // [n_k + n_v (+ 2 H_v)][d_model] 16-bit decoded weights of the current layer (0 bytes for bf16 weights)
  size_t off_hist;       // bf16 [n_requests][C][w-1] conv state each request continues from (current layer)
  size_t off_x16;        // fp16 staging: half [max_slots][64][d_model] anchors of the current layer, slot order;
                         // W8A8: uint8 [max_slots][64][d_model] activation codes
  size_t off_sx;         // W8A8: float [max_slots][d_model / 128][64] activation scales
  size_t off_qpart;      // float [4][256][channels] partial sums of the conv-state kernel's k quarters (small batches)
  size_t off_sched;      // tile counter and per-pair mailboxes of the projection's tile scheduler (SR_TILE_SCHED_BYTES)
  size_t lane_bytes;     // size of one lane's block of hand-over buffers (off_kv16 .. end)
  int lanes;             // lane blocks in `total`
  size_t total;
  int64_t max_slots;
};

// The persistent projection kernels hand out their tiles in index order at run time: one counter and, per CTA pair
// (per CTA in the 8-bit kernel), a ring of sixteen 8-byte mailboxes through which the producer thread that draws the
// tile tells every other role which tile comes next.
constexpr int SR_SCHED_MAX_PAIRS = 160, SR_SCHED_RING = 16;     // pairs, or single CTAs of the 8-bit projection
constexpr size_t SR_TILE_SCHED_BYTES = 256 + (size_t)SR_SCHED_MAX_PAIRS * SR_SCHED_RING * 8;

static inline size_t sr_align256(size_t x) { return (x + 255) & ~size_t(255); }

static inline SrWorkspace sr_workspace_layout(const sr_ctx* ctx, int32_t n_requests, int32_t max_pages,
                                              int64_t max_total_rows, int lanes = 1) {
  SrWorkspace w;
  int64_t by_rows = max_total_rows / SR_PAGE_ROWS + n_requests;
  int64_t by_table = (int64_t)n_requests * max_pages;
  w.max_slots = by_rows < by_table ? by_rows : by_table;
  if (w.max_slots < 1) w.max_slots = 1;
  w.max_slots = (w.max_slots + 3) & ~int64_t(3);  // the projection tiles up to four page slots at a time
  size_t at = 0;
  w.off_header = at;    at += 256;
  w.off_req_rows = at;  at = sr_align256(at + sizeof(int32_t) * (size_t)n_requests);
  w.off_req_slot0 = at; at = sr_align256(at + sizeof(int32_t) * (size_t)n_requests);
  w.off_req_out = at;   at = sr_align256(at + sizeof(int32_t) * (size_t)n_requests);
  w.off_req_row0 = at;  at = sr_align256(at + sizeof(int32_t) * (size_t)n_requests);
  w.off_req_order = at; at = sr_align256(at + sizeof(int32_t) * (size_t)n_requests);
  w.off_slot_page = at; at = sr_align256(at + sizeof(int32_t) * (size_t)w.max_slots);
  w.off_slot_rows = at; at = sr_align256(at + sizeof(int32_t) * (size_t)w.max_slots);
  w.off_slot_first = at; at = sr_align256(at + sizeof(int32_t) * (size_t)w.max_slots);
  // from here on: the per-layer hand-over buffers of lane 0; lane i sits lane_bytes * i further on
  at = (at + 1023) & ~size_t(1023);
  const size_t lane0 = at;
  const size_t n_kv = (size_t)ctx->n_k + ctx->n_v;
  const size_t kv_pitch = (n_kv + 127) / 128 * 128;     // channels per slot in the hand-over tiles (whole 128-channel tiles)
  w.off_kv16 = at;      at = sr_align256(at + sizeof(uint16_t) * (size_t)w.max_slots * SR_PAGE_ROWS * kv_pitch);
  w.off_zraw = at;      at = sr_align256(at + sizeof(float) * (size_t)w.max_slots * 6 * n_kv);
  w.off_z = at;         at = sr_align256(at + sizeof(float) * (size_t)w.max_slots * SR_PAGE_ROWS * (size_t)ctx->n_gate);
  w.off_split = at;     at = sr_align256(at + sr_scan_split_bytes(ctx, w.max_slots));
  w.off_wdec = at;      at = sr_align256(at + ctx->wdec_bytes);
  w.off_hist = at;      at = sr_align256(at + sizeof(uint16_t) * (size_t)n_requests * ctx->conv_ch * (SR_CONV_W - 1));
  w.off_x16 = at;       at = sr_align256(at + (ctx->fp16_stage || ctx->w8a8 ? (ctx->w8a8 ? 1 : 2) * (size_t)w.max_slots * SR_PAGE_ROWS *
                                                                                     (size_t)ctx->desc.d_model : 0));
  w.off_sx = at;        at = sr_align256(at + (ctx->w8a8 ? sizeof(float) * (size_t)w.max_slots * SR_PAGE_ROWS *
                                                               (size_t)(ctx->desc.d_model / 128) : 0));
  w.off_qpart = at;     at = sr_align256(at + ((int64_t)n_requests * (SR_CONV_W - 1) <= 256 ? sr_conv_tail_part_bytes(ctx) : 0));
  w.off_sched = at;     at = sr_align256(at + SR_TILE_SCHED_BYTES);
  at = (at + 1023) & ~size_t(1023);
  w.lane_bytes = at - lane0;
  w.lanes = lanes < 1 ? 1 : lanes;
  w.total = lane0 + w.lane_bytes * (size_t)w.lanes;
  return w;
}

// Blocks of hand-over buffers for a batch of these bounds (layers in flight at once): as many (up to SR_MAX_BLOCKS, and
// no more than the model has layers) as keep the blocks together within SR_LANES_BUDGET_BYTES; up to SR_MAX_LANES
// streams work on them; large batches fill the device with
// one layer and get one lane.  (Measured with a 24 GiB budget, i.e. two to four lanes on the 250 000-row
// configurations, in the same run as one lane: the chunk-local kernel does run in the shared memory the next
// layer's persistent projection leaves free, but the projection slows by as much -- steps 1.8 % and 1.0 % shorter
// on two configurations, 1.1 % longer on the third.)
// the block counts a call may use: 32, 24, 16, 8, 4, 2, 1 (all multiples of the stream count they are served by, so a
// block always meets the same stream)
static inline int sr_fewer_blocks(int blocks) { return blocks == 32 ? 24 : (blocks == 24 ? 16 : blocks >> 1); }
static inline int sr_policy_lanes(const sr_ctx* ctx, int32_t n_requests, int32_t max_pages, int64_t max_total_rows) {
  const size_t per_lane = sr_workspace_layout(ctx, n_requests, max_pages, max_total_rows, 1).lane_bytes;
  int lanes = SR_MAX_BLOCKS;
  while (lanes > 1 && ((size_t)lanes * per_lane > SR_LANES_BUDGET_BYTES || lanes > ctx->desc.n_layers)) lanes = sr_fewer_blocks(lanes);
  return lanes;
}

// Device views handed to the kernels.
struct SrSched {
  uint32_t* status;     // [0] status word, [1] n_slots, [2] total rows
  int32_t* req_rows;
  int32_t* req_slot0;
  int32_t* req_out;
  int32_t* req_row0;
  int32_t* req_order;
  int32_t* slot_page;
  int32_t* slot_rows;
  int32_t* slot_first;
  int32_t n_requests;
  int32_t max_slots;
  // SR_DEBUG_CHECK_BOUNDS: kernels test every table-driven index against these before using it
  int32_t check_bounds;   // 0 = off
  int32_t n_phys_pages;   // pool pages
  int32_t n_state_slots;  // slots in the output arrays (0 = not stated: not checked)
};

#ifdef __CUDACC__
// Range check used under SR_DEBUG_CHECK_BOUNDS: records the failure and tells the caller to skip the access.
__device__ __forceinline__ bool sr_check(const SrSched& s, bool in_range) {
  if (!s.check_bounds || in_range) return true;
  atomicOr(s.status, SR_DEV_BOUNDS_CHECK);
  return false;
}
__device__ __forceinline__ bool sr_check_slot(const SrSched& s, int slot) { return sr_check(s, slot >= 0 && slot < s.max_slots); }
__device__ __forceinline__ bool sr_check_page(const SrSched& s, int page) { return sr_check(s, page >= 0 && page < s.n_phys_pages); }
__device__ __forceinline__ bool sr_check_out(const SrSched& s, int out_slot) {
  return sr_check(s, out_slot >= 0 && (s.n_state_slots <= 0 || out_slot < s.n_state_slots));
}
#endif

static inline SrSched sr_sched_view(void* workspace, const SrWorkspace& w, int32_t n_requests) {
  char* b = (char*)workspace;
  SrSched s;
  s.status = (uint32_t*)(b + w.off_header);
  s.req_rows = (int32_t*)(b + w.off_req_rows);
  s.req_slot0 = (int32_t*)(b + w.off_req_slot0);
  s.req_out = (int32_t*)(b + w.off_req_out);
  s.req_row0 = (int32_t*)(b + w.off_req_row0);
  s.req_order = (int32_t*)(b + w.off_req_order);
  s.slot_page = (int32_t*)(b + w.off_slot_page);
  s.slot_rows = (int32_t*)(b + w.off_slot_rows);
  s.slot_first = (int32_t*)(b + w.off_slot_first);
  s.n_requests = n_requests;
  s.max_slots = (int32_t)w.max_slots;
  s.check_bounds = 0;
  s.n_phys_pages = 0;
  s.n_state_slots = 0;
  return s;
}

// The fused intermediate format between the projection epilogue and the chunk scan.  Tiles are channel-major:
// the k | v channels of one 64-row page slot are [ncb * 128 channels][64 rows] (the channel count rounded up to
// whole 128-channel projection tiles), so a head's keys (d_k channels) or values (d_v channels) of one slot
// are one contiguous [channels][64 rows] block.
struct SrFused {
  const __nv_bfloat16* hist;  // conv state the requests continue from, [request][C][w-1] (current layer), or null = zero
  const char* in_ssm_layer;   // recurrent states the requests continue from (current layer; slot stride below), or null
  int64_t in_ssm_slot_stride;
  const uint8_t* x8; // W8A8 only: the layer's activation codes in slot order [slot][64][d_model], else null
  const float* sx;   // W8A8 only: their scales [slot][d_model / 128][64]
  const __half* x16; // fp16 staging only: the layer's anchors in slot order [slot][64][d_model], else null
  const __half* w16; // fp16 staging only: dequantised k | v weight rows, then the 2 H_v gate rows, [.][d_model]
  __half* kv16;      // [slot][ncb * 128][64] = SiLU(conv(Z)) in fp16.  Rows 0..2 of a slot whose conv
                     // history lies in another projection tile (slot % fix_mod == 0 and not the first slot of
                     // its request) are placeholders: the scan recomputes them from zraw
  float* zraw;       // [slot][6][n_kv] raw fp32 projection rows: 0,1,2 (slots with slot % fix_mod == 0) |
                     // the slot's last three valid rows (every slot)
  float* gates;      // [slot][2 H_v][64] raw fp32 gate pre-activations: a_0.., b_0.. (channel-major)
  int32_t ncb;       // 128-channel blocks per slot: ceil((n_k + n_v) / 128)
  int32_t n_kv;
  int32_t n_gate;
  int32_t fix_mod;   // page slots per projection tile along the token axis
  // Group replay projects the query channels for every row too (the layer's outputs need them): the hand-over tiles
  // then hold q | k | v and the conv channel of projected channel c is c itself; otherwise they hold k | v and the
  // conv channel is n_k + c.
  int32_t x_slot_order;   // the projection's row operand (`pool` argument) is a packed bf16 buffer in slot order
  int32_t with_q;    // 0: k | v tiles (state-only replay), 1: q | k | v tiles
  int32_t k_ch0;     // first key channel inside a slot's tiles (0, or n_k with the query block in front)
  int32_t v_ch0;     // first value channel (n_k, or 2 n_k)
  // group replay only: what the state chain leaves for the output kernel, per (slot, value head)
  __half* dump_s;    // [slot][H_v][d_k][d_v] fp16: the state entering the chunk (not written for a request's first chunk)
  __half* dump_u;    // [slot][H_v][d_v][64] fp16: the chunk's pseudo-values U^T, before the row factors
  float* qpart;      // conv state of small batches: partial sums of the batched kernel's k quarters, or null
  void* tile_sched;  // the projection's tile scheduler state (SR_TILE_SCHED_BYTES; cleared by every launch)
};

struct SrPoolView {
  const char* base;
  int64_t page_stride, layer_stride, row_stride;
  int32_t n_phys_pages;
};

// ---- launch functions (one per kernel file) ----------------------------------------------------

// Packs the batch: validates each request on the device, assigns page slots, fills the tables.
cudaError_t sr_launch_schedule(const SrSched& s, const int32_t* pages, const int32_t* state_slots,
                               const int32_t* replay_lens, int32_t max_pages, int32_t max_replay_len,
                               int64_t max_total_rows, int32_t n_phys_pages, int32_t n_state_slots,
                               cudaStream_t stream);

// Copies the gathered rows of one pool layer into a packed [rows][d_model] bf16 array.
cudaError_t sr_launch_debug_gather(const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                   int32_t d_model, int32_t max_pages, void* out_rows,
                                   int64_t out_capacity_rows, cudaStream_t stream);

// block-scaled weights, exact form: the bare e4m3 codes of the k | v rows decoded (exactly) to bf16 into `decoded`
cudaError_t sr_launch_weight_decode(const sr_ctx* ctx, const sr_layer_weights& w, void* decoded, cudaStream_t stream);
// continuation: copies the layer's conv states of the batch from the caller's array (by state slot) into the
// workspace (by request), so that the kernels never read an array the same call writes (sr_conv_tail.cu)
cudaError_t sr_launch_hist_gather(const sr_ctx* ctx, const SrSched& s, const char* in_conv_layer, int64_t slot_stride,
                                  __nv_bfloat16* hist, cudaStream_t stream);
// the sidecar's write side (sr_anchor_write.cu)
cudaError_t sr_launch_anchor_write(const sr_anchor_pool& pool, const int32_t* pool_layers, int32_t n_layers,
                                   const void* hidden, int64_t hidden_layer_stride, int64_t hidden_row_stride,
                                   const int32_t* dest_page, const int32_t* dest_row, int32_t n_tokens, int32_t d_model,
                                   uint32_t* status, cudaStream_t stream);
// fp16 staging for block-scaled weights (sr_fp16_stage.cu)
cudaError_t sr_launch_stage_weights_fp16(const sr_ctx* ctx, const sr_layer_weights& w, __half* w16, cudaStream_t stream);
cudaError_t sr_launch_stage_anchors_fp16(const sr_ctx* ctx, const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                         __half* x16, cudaStream_t stream);
// W8A8: the activation quantiser (codes and scales in slot order) and, for tests, its output re-packed by request
cudaError_t sr_launch_quant_anchors_e4m3(const sr_ctx* ctx, const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                         uint8_t* x8, float* sx, cudaStream_t stream);
cudaError_t sr_launch_pack_quantised(const sr_ctx* ctx, const SrSched& s, int32_t max_pages, const uint8_t* x8,
                                     const float* sx, void* out_codes, float* out_scales, int64_t capacity_rows,
                                     cudaStream_t stream);

// The projection with channels on the MMA's M axis and tokens on its N axis, so that each epilogue
// thread owns one channel and walks its tokens in order: the causal conv and SiLU are applied in
// registers and the fused format (SrFused) is written instead of fp32 columns.
bool sr_proj_fused_supported(const sr_ctx* ctx);
bool sr_proj_fused_exact_fp8_supported(const sr_ctx* ctx);
cudaError_t sr_launch_proj_fused(const sr_ctx* ctx, const SrSched& s, const sr_anchor_pool& pool, int32_t pool_layer,
                                 const sr_layer_weights& w, const void* decoded, const SrFused& fused, int sm_count,
                                 cudaStream_t stream);
// the projections of several layers of a small batch in one launch (bf16 weights, at most one wave of tiles per layer)
bool sr_proj_fused_batchable(const sr_ctx* ctx, int64_t max_slots, int sm_count);
int sr_proj_fused_batch_max();
cudaError_t sr_launch_proj_fused_batch(const sr_ctx* ctx, const SrSched& s, const sr_anchor_pool& pool, int n,
                                       const int32_t* pool_layers, const sr_layer_weights* const* w, const SrFused* fused,
                                       int sm_count, cudaStream_t stream);

// group replay (sr_group_gemm.cu, sr_group_output.cu)
cudaError_t sr_launch_rows_gemm(const SrSched& s, int kind, const __nv_bfloat16* a, int64_t k, const void* b, const void* b2,
                                int32_t n, __nv_bfloat16* c, int64_t ldc, const __nv_bfloat16* residual, int64_t ldr,
                                int sm_count, cudaStream_t stream);
bool sr_group_output_supported(int d_k, int d_v);
cudaError_t sr_launch_group_output(const sr_ctx* ctx, const SrSched& s, const SrFused& fused, const void* split_buf,
                                   const __nv_bfloat16* zg, const __nv_bfloat16* o_norm_w, float norm_eps, __nv_bfloat16* y,
                                   cudaStream_t stream);
// conv state of every channel from the raw rows a q | k | v projection kept (group replay)
cudaError_t sr_launch_conv_tail_from_raw(const sr_ctx* ctx, const SrSched& s, const SrFused& fused, char* out_conv_layer,
                                         int64_t slot_stride, cudaStream_t stream);
cudaError_t sr_launch_rmsnorm_rows(const SrSched& s, const SrPoolView& pool, int32_t pool_layer, const __nv_bfloat16* rows_in,
                                   const __nv_bfloat16* w, float eps, int32_t d_model, __nv_bfloat16* out,
                                   __nv_bfloat16* copy_out, cudaStream_t stream);

// Conv state: last w-1 projection rows of every channel, rounded to bf16.
int sr_conv_tail_launches(const sr_ctx* ctx, int n_requests);
cudaError_t sr_launch_conv_tail(const sr_ctx* ctx, const SrSched& s, const SrPoolView& pool, int32_t pool_layer,
                                const sr_layer_weights& w, const SrFused& fused, char* out_conv_layer,
                                int64_t slot_stride, cudaStream_t stream);

// The chunked scan in two kernels for the fused format: everything local to a chunk (gates, K K^T, the
// inverse) for all chunks at once, then the state chain per (head, request).
bool sr_chunk_local_supported(int d_k, int d_v);
cudaError_t sr_launch_chunk_local(const sr_ctx* ctx, const SrSched& s, const sr_layer_weights& w, const SrFused& fused,
                                  void* split_buf, cudaStream_t stream);
// (tcgen05 tensor cores, the state in tensor memory)
bool sr_scan_chain_supported(int d_k, int d_v);
cudaError_t sr_launch_scan_chain_umma(const sr_ctx* ctx, const SrSched& s, const SrFused& fused, const void* split_buf,
                                      char* out_ssm_layer, int64_t slot_stride, int sm_count, cudaStream_t stream);
