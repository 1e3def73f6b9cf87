// The C boundary: argument checking and the per-layer launch sequence.  No arithmetic of the
// method lives here; every step runs in the kernels the launch functions enqueue.
#include <mutex>
#include <new>
#include <stdlib.h>
#include <string.h>

#include "sr_common.cuh"

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_device_mutex;
bool g_once_done[kMaxDevices][SR_ONCE_KEYS];
int g_sm_count[kMaxDevices];
}  // namespace

cudaError_t sr_once_per_device(int key, cudaError_t (*setup)()) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices || key < 0 || key >= SR_ONCE_KEYS) return cudaErrorInvalidValue;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (g_once_done[dev][key]) return cudaSuccess;
  e = setup();
  if (e == cudaSuccess) g_once_done[dev][key] = true;
  return e;
}

cudaError_t sr_current_device_sms(int* sms) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidValue;
  std::lock_guard<std::mutex> lock(g_device_mutex);
  if (g_sm_count[dev] <= 0) {
    int n = 0;
    e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    if (n <= 0) return cudaErrorInvalidValue;
    g_sm_count[dev] = n;
  }
  *sms = g_sm_count[dev];
  return cudaSuccess;
}

namespace {

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int check_batch(const sr_ctx* ctx, const sr_page_table* t) {
  if (!ctx || !t) return SR_ERR_INVALID_ARG;
  if (!ctx->kernels_cover) return SR_ERR_UNSUPPORTED_SHAPE;
  if (t->n_requests < 0 || t->max_pages < 0 || t->max_replay_len < 0 || t->max_total_rows < 0 || t->n_state_slots < 0)
    return SR_ERR_INVALID_ARG;
  if (t->n_requests > 65535) return SR_ERR_UNSUPPORTED_SHAPE;   // one grid row per request
  if ((int64_t)t->max_replay_len > (int64_t)t->max_pages * ctx->desc.page_rows) return SR_ERR_INVALID_ARG;
  if (t->max_total_rows > (int64_t)1 << 30) return SR_ERR_UNSUPPORTED_SHAPE;
  // the tensor-core kernels index page slots with one grid row (and one 32-bit tile coordinate) per slot
  if (sr_workspace_layout(ctx, t->n_requests, t->max_pages, t->max_total_rows).max_slots > 65535)
    return SR_ERR_UNSUPPORTED_SHAPE;
  return SR_OK;
}

int check_pool(const sr_ctx* ctx, const sr_anchor_pool* p) {
  if (!p || !p->base || !p->layer_to_pool) return SR_ERR_INVALID_ARG;
  if (p->n_phys_pages <= 0 || p->n_pool_layers <= 0) return SR_ERR_INVALID_ARG;
  const int64_t row_bytes = (int64_t)ctx->desc.d_model * 2;
  if (p->row_stride_bytes < row_bytes || p->row_stride_bytes % 16 || p->layer_stride_bytes % 16 ||
      p->page_stride_bytes % 16 || p->layer_stride_bytes < 0 || p->page_stride_bytes < 0)
    return SR_ERR_INVALID_ARG;
  if (!aligned(p->base, 16)) return SR_ERR_INVALID_ARG;
  for (int l = 0; l < ctx->desc.n_layers; ++l)
    if (p->layer_to_pool[l] < -1 || p->layer_to_pool[l] >= p->n_pool_layers) return SR_ERR_INVALID_ARG;
  return SR_OK;
}

SrPoolView pool_view(const sr_anchor_pool* p) {
  SrPoolView v;
  v.base = (const char*)p->base;
  v.page_stride = p->page_stride_bytes;
  v.layer_stride = p->layer_stride_bytes;
  v.row_stride = p->row_stride_bytes;
  v.n_phys_pages = p->n_phys_pages;
  return v;
}

}  // namespace

extern "C" {

const char* sr_version(void) { return "sr_replay 0.1 (sm_100a)"; }

const char* sr_status_string(int status) {
  switch (status) {
    case SR_OK: return "SR_OK";
    case SR_ERR_INVALID_ARG: return "SR_ERR_INVALID_ARG";
    case SR_ERR_UNSUPPORTED_SHAPE: return "SR_ERR_UNSUPPORTED_SHAPE";
    case SR_ERR_WORKSPACE: return "SR_ERR_WORKSPACE";
    case SR_ERR_CUDA: return "SR_ERR_CUDA";
    default: return "SR_ERR_UNKNOWN";
  }
}

int sr_create(const sr_model_desc* d, sr_ctx** out_ctx) {
  if (!d || !out_ctx) return SR_ERR_INVALID_ARG;
  *out_ctx = nullptr;
  if (d->n_layers <= 0 || d->d_model <= 0 || d->n_k_heads <= 0 || d->n_v_heads <= 0 || d->d_k <= 0 || d->d_v <= 0)
    return SR_ERR_INVALID_ARG;
  if (d->weight_format != SR_W_BF16 && d->weight_format != SR_W_E4M3_BLOCK128) return SR_ERR_INVALID_ARG;
  if (d->conv_activation != SR_CONV_SILU && d->conv_activation != SR_CONV_IDENTITY) return SR_ERR_INVALID_ARG;
  if (d->recurrence != SR_REC_GATED_DELTA && d->recurrence != SR_REC_DECAY_ONLY) return SR_ERR_INVALID_ARG;
  if (d->act_quant != SR_AQ_NONE && d->act_quant != SR_AQ_E4M3_1X128) return SR_ERR_INVALID_ARG;
  if (d->act_quant == SR_AQ_E4M3_1X128 && d->weight_format != SR_W_E4M3_BLOCK128) return SR_ERR_INVALID_ARG;
  if (!(d->l2_eps >= 0.f)) return SR_ERR_INVALID_ARG;
  if (d->conv_width < 2 || d->page_rows <= 0 || d->n_v_heads % d->n_k_heads != 0) return SR_ERR_INVALID_ARG;
  sr_ctx* c = new (std::nothrow) sr_ctx;
  if (!c) return SR_ERR_INVALID_ARG;
  c->desc = *d;
  c->n_k = d->n_k_heads * d->d_k;
  c->n_v = d->n_v_heads * d->d_v;
  c->n_gate = 2 * d->n_v_heads;
  c->conv_ch = 2 * c->n_k + c->n_v;
  c->last_launches = 0;
  c->profiling = false;
  c->ev_used = 0;
  c->copy_in = nullptr;
  c->copy_out = nullptr;
  c->lanes_ready = false;
  for (int i = 0; i < SR_MAX_LANES - 1; ++i) { c->lane_stream[i] = nullptr; c->lane_join[i] = nullptr; }
  c->lane_fork = nullptr;
  c->debug_flags = d->debug_flags;
  c->wdec_bytes = 0;
  c->kernels_cover = d->conv_width == SR_CONV_W && d->page_rows == SR_PAGE_ROWS && sr_proj_fused_supported(c) &&
                     sr_chunk_local_supported(d->d_k, d->d_v) && sr_scan_chain_supported(d->d_k, d->d_v);
  const bool e4m3 = d->weight_format == SR_W_E4M3_BLOCK128;
  c->w8a8 = e4m3 && d->act_quant == SR_AQ_E4M3_1X128;
  // 8-bit operands: channel tiles inside the scale blocks, and the batched conv-state kernel's tiling
  if (c->w8a8 && !(sr_proj_fused_exact_fp8_supported(c) && c->conv_ch % 64 == 0 && c->n_gate <= 256)) c->kernels_cover = false;
  // block-scaled weights: fp16 staging by default; fp32 promotion of bare-code partial sums on request, where the
  // channel tiles line up with the scale blocks
  c->fp16_stage = c->kernels_cover && e4m3 && !c->w8a8 &&
                  !((d->debug_flags & SR_DEBUG_FP8_EXACT) && sr_proj_fused_exact_fp8_supported(c));
  if (c->kernels_cover && e4m3 && !c->w8a8)
    c->wdec_bytes = (size_t)(c->n_k + c->n_v + (c->fp16_stage ? c->n_gate : 0)) * d->d_model * 2;
  *out_ctx = c;
  return SR_OK;
}

void sr_destroy(sr_ctx* ctx) {
  if (!ctx) return;
  for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : ctx->ev_copy) cudaEventDestroy(e);
  for (int i = 0; i < SR_MAX_LANES - 1; ++i) {
    if (ctx->lane_stream[i]) cudaStreamDestroy(ctx->lane_stream[i]);
    if (ctx->lane_join[i]) cudaEventDestroy(ctx->lane_join[i]);
  }
  if (ctx->lane_fork) cudaEventDestroy(ctx->lane_fork);
  if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
  if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
  delete ctx;
}

int sr_ssm_bytes_per_layer(const sr_ctx* ctx, size_t* out_bytes) {
  if (!ctx || !out_bytes) return SR_ERR_INVALID_ARG;
  *out_bytes = (size_t)ctx->desc.n_v_heads * ctx->desc.d_k * ctx->desc.d_v * sizeof(float);
  return SR_OK;
}

int sr_conv_bytes_per_layer(const sr_ctx* ctx, size_t* out_bytes) {
  if (!ctx || !out_bytes) return SR_ERR_INVALID_ARG;
  *out_bytes = (size_t)ctx->conv_ch * (ctx->desc.conv_width - 1) * 2;
  return SR_OK;
}

int sr_workspace_bytes(const sr_ctx* ctx, const sr_page_table* table, size_t* out_bytes) {
  if (!out_bytes) return SR_ERR_INVALID_ARG;
  int st = check_batch(ctx, table);
  if (st != SR_OK) return st;
  const int lanes = sr_policy_lanes(ctx, table->n_requests, table->max_pages, table->max_total_rows);
  *out_bytes = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows, lanes).total;
  return SR_OK;
}

int sr_workspace_bytes_min(const sr_ctx* ctx, const sr_page_table* table, size_t* out_bytes) {
  if (!out_bytes) return SR_ERR_INVALID_ARG;
  int st = check_batch(ctx, table);
  if (st != SR_OK) return st;
  *out_bytes = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows, 1).total;
  return SR_OK;
}

}  // extern "C"

namespace {
// Host-side callbacks around the launches of one layer (used by the host-buffer entry point to order its
// per-layer copies against the kernels); each returns false on a CUDA error.
struct LayerHooks {
  void* user;
  bool (*before)(void* user, int layer, int pool_layer, cudaStream_t stream);
  bool (*after)(void* user, int layer, cudaStream_t stream);
};

// Every check that needs no device: run before anything is enqueued.
int validate_call(const sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
                  const uint8_t* layer_mask, const sr_layer_weights* weights, const sr_out* out_ssm,
                  const sr_out* out_conv, const void* workspace, size_t workspace_bytes, const sr_out* in_ssm,
                  const sr_out* in_conv) {
  int st = check_batch(ctx, table);
  if (st != SR_OK) return st;
  if (in_ssm && (!in_ssm->base || !aligned(in_ssm->base, 16) || in_ssm->slot_stride_bytes % 16 ||
                 in_ssm->layer_stride_bytes % 16))
    return SR_ERR_INVALID_ARG;
  if (in_conv && (!in_conv->base || !aligned(in_conv->base, 2) || in_conv->slot_stride_bytes % 2 ||
                  in_conv->layer_stride_bytes % 2))
    return SR_ERR_INVALID_ARG;
  if (!replay_lens || !layer_mask || !weights || !out_ssm || !out_conv || !table->pages) return SR_ERR_INVALID_ARG;
  if (!out_ssm->base || !out_conv->base) return SR_ERR_INVALID_ARG;
  if (!aligned(out_ssm->base, 16) || out_ssm->slot_stride_bytes % 16 || out_ssm->layer_stride_bytes % 16)
    return SR_ERR_INVALID_ARG;
  if (!aligned(out_conv->base, 2) || out_conv->slot_stride_bytes % 2 || out_conv->layer_stride_bytes % 2)
    return SR_ERR_INVALID_ARG;
  st = check_pool(ctx, pool);
  if (st != SR_OK) return st;
  const sr_model_desc& d = ctx->desc;
  for (int l = 0; l < d.n_layers; ++l) {
    if (!layer_mask[l]) continue;
    const sr_layer_weights& w = weights[l];
    if (pool->layer_to_pool[l] < 0) return SR_ERR_INVALID_ARG;   // asked to rebuild a layer that has no anchors
    if (!w.w_qkv || !w.w_ab || !w.conv_w || !w.decay_scale || !w.dt_bias) return SR_ERR_INVALID_ARG;
    if (d.weight_format == SR_W_E4M3_BLOCK128 && !w.w_qkv_scale) return SR_ERR_INVALID_ARG;
    if (!aligned(w.w_qkv, 16) || !aligned(w.w_ab, 16) || !aligned(w.conv_w, 16)) return SR_ERR_INVALID_ARG;
  }
  // the smallest workspace that serves the call holds one lane
  const SrWorkspace lay = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows, 1);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < lay.total) return SR_ERR_WORKSPACE;
  return SR_OK;
}

}  // namespace

// the context's lane streams and their fork / join events, made once
bool sr_ensure_lanes(sr_ctx* ctx) {
  if (ctx->lanes_ready) return true;
  for (int i = 0; i < SR_MAX_LANES - 1; ++i) {
    if (cudaStreamCreateWithFlags(&ctx->lane_stream[i], cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaEventCreateWithFlags(&ctx->lane_join[i], cudaEventDisableTiming) != cudaSuccess) return false;
  }
  if (cudaEventCreateWithFlags(&ctx->lane_fork, cudaEventDisableTiming) != cudaSuccess) return false;
  ctx->lanes_ready = true;
  return true;
}

namespace {

int replay_impl(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
                const uint8_t* layer_mask, const sr_layer_weights* weights, const sr_out* out_ssm,
                const sr_out* out_conv, void* workspace, size_t workspace_bytes, void* stream_,
                const LayerHooks* hooks, const sr_out* in_ssm = nullptr, const sr_out* in_conv = nullptr) {
  int st = validate_call(ctx, pool, table, replay_lens, layer_mask, weights, out_ssm, out_conv, workspace,
                         workspace_bytes, in_ssm, in_conv);
  if (st != SR_OK) return st;
  const sr_model_desc& d = ctx->desc;
  cudaStream_t stream = (cudaStream_t)stream_;
  ctx->last_launches = 0;
  ctx->ev_used = 0;
  ctx->ev_kind.clear();
  if (table->n_requests == 0) return SR_OK;

  // Layers are independent units (each has its own anchors, weights and outputs), so a batch too small to fill
  // the device with one layer runs several layers side by side: layer j of the call goes to lane j % lanes, a
  // lane being a stream with its own block of hand-over buffers.  As many lanes as the policy gives and the
  // workspace holds; lane 0 is the caller's stream, the others fork from it after the packing kernel and join
  // it at the end, so the call stays one unit of work on `stream` (and one graph when captured).
  int n_active = 0;
  for (int l = 0; l < d.n_layers; ++l) n_active += layer_mask[l] ? 1 : 0;
  int lanes = sr_policy_lanes(ctx, table->n_requests, table->max_pages, table->max_total_rows);
  while (lanes > 1 && (lanes > n_active ||
                       sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows, lanes).total > workspace_bytes))
    lanes = sr_fewer_blocks(lanes);
  const SrWorkspace lay = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows, lanes);
  const int blocks = lanes;                                  // hand-over blocks; the streams that work on them:
  if (lanes > SR_MAX_LANES) lanes = SR_MAX_LANES;            // (the block count is a multiple: a block always meets the same stream)
  if (lanes > 1 && !sr_ensure_lanes(ctx)) return SR_ERR_CUDA;

  SrSched sched = sr_sched_view(workspace, lay, table->n_requests);
  sched.check_bounds = (ctx->debug_flags & SR_DEBUG_CHECK_BOUNDS) ? 1 : 0;
  sched.n_phys_pages = pool->n_phys_pages;
  sched.n_state_slots = table->n_state_slots;
  const SrPoolView pv = pool_view(pool);
  int sm_count = 0;
  if (sr_current_device_sms(&sm_count) != cudaSuccess) return SR_ERR_CUDA;

  {
    SrLaunchScope scope(ctx, stream, SR_KERNEL_SCHEDULE);
    if (sr_launch_schedule(sched, table->pages, table->state_slots, replay_lens, table->max_pages,
                           table->max_replay_len, table->max_total_rows, pool->n_phys_pages, table->n_state_slots,
                           stream) != cudaSuccess)
      return SR_ERR_CUDA;
  }
  // Small batches with plain bf16 weights: the projections of up to `blocks` layers go through ONE launch on the
  // caller's stream (a single hit would otherwise run its layers' one-wave projection launches one after the other);
  // the rest of each layer then runs on the lanes as before.
  const bool batched = blocks > 1 && !hooks && sr_proj_fused_batchable(ctx, lay.max_slots, sm_count);
  const int batch_max = blocks < sr_proj_fused_batch_max() ? blocks : sr_proj_fused_batch_max();
  auto fork = [&]() -> bool {
    if (lanes <= 1) return true;
    if (cudaEventRecord(ctx->lane_fork, stream) != cudaSuccess) return false;
    for (int i = 0; i < lanes - 1; ++i)
      if (cudaStreamWaitEvent(ctx->lane_stream[i], ctx->lane_fork, 0) != cudaSuccess) return false;
    return true;
  };
  auto join = [&]() -> bool {
    bool ok = true;
    for (int i = 0; i < lanes - 1; ++i)
      if (cudaEventRecord(ctx->lane_join[i], ctx->lane_stream[i]) != cudaSuccess ||
          cudaStreamWaitEvent(stream, ctx->lane_join[i], 0) != cudaSuccess)
        ok = false;
    return ok;
  };
  if (!batched && !fork()) return SR_ERR_CUDA;
  int status = SR_OK, j = 0;
  int projected_until = 0;            // batched: layers (by count j) whose projection has been launched
  for (int l = 0; l < d.n_layers && status == SR_OK; ++l) {
    if (!layer_mask[l]) continue;
    if (batched && j == projected_until) {
      // the next batch of projections: layers j .. j + n - 1 of the call, into blocks (j + i) % blocks
      if (j > 0 && !join()) { status = SR_ERR_CUDA; break; }        // their blocks are in use until the lanes are done
      const sr_layer_weights* bw[SR_MAX_BLOCKS];
      int32_t bpl[SR_MAX_BLOCKS];
      SrFused bf[SR_MAX_BLOCKS];
      int n = 0;
      status = SR_ERR_CUDA;
      bool ok = true;
      for (int l2 = l; l2 < d.n_layers && n < batch_max && ok; ++l2) {
        if (!layer_mask[l2]) continue;
        char* b2 = (char*)workspace + (size_t)((j + n) % blocks) * lay.lane_bytes;
        SrFused& f = bf[n];
        f = SrFused();
        f.kv16 = (__half*)(b2 + lay.off_kv16);
        f.zraw = (float*)(b2 + lay.off_zraw);
        f.gates = (float*)(b2 + lay.off_z);
        f.ncb = (ctx->n_k + ctx->n_v + 127) / 128;
        f.tile_sched = b2 + lay.off_sched;
        f.hist = nullptr;
        if (in_conv) {
          __nv_bfloat16* hist = (__nv_bfloat16*)(b2 + lay.off_hist);
          SrLaunchScope scope(ctx, stream, SR_KERNEL_CONV_TAIL);
          if (sr_launch_hist_gather(ctx, sched, (const char*)in_conv->base + (int64_t)l2 * in_conv->layer_stride_bytes,
                                    in_conv->slot_stride_bytes, hist, stream) != cudaSuccess)
            ok = false;
          f.hist = hist;
        }
        bw[n] = &weights[l2];
        bpl[n] = pool->layer_to_pool[l2];
        ++n;
      }
      if (!ok) break;
      {
        SrLaunchScope scope(ctx, stream, SR_KERNEL_PROJECTION);
        if (sr_launch_proj_fused_batch(ctx, sched, *pool, n, bpl, bw, bf, sm_count, stream) != cudaSuccess) break;
      }
      if (!fork()) break;
      projected_until = j + n;
      status = SR_OK;
    }
    const int lane = j % lanes;
    cudaStream_t ls = lane == 0 ? stream : ctx->lane_stream[lane - 1];
    char* base = (char*)workspace + (size_t)(j % blocks) * lay.lane_bytes;       // this layer's hand-over block
    ++j;
    SrFused fused;
    fused.kv16 = (__half*)(base + lay.off_kv16);
    fused.zraw = (float*)(base + lay.off_zraw);
    fused.gates = (float*)(base + lay.off_z);
    fused.ncb = (ctx->n_k + ctx->n_v + 127) / 128;
    fused.n_kv = ctx->n_k + ctx->n_v;
    fused.n_gate = ctx->n_gate;
    // page slots per run of the projection's conv epilogue (the first three rows of a run are finished by the scan)
    fused.fix_mod = ctx->w8a8 ? 1 : ((d.weight_format == SR_W_E4M3_BLOCK128 && !ctx->fp16_stage) ? 2 : 4);
    fused.x_slot_order = 0;
    fused.with_q = 0;
    fused.k_ch0 = 0;
    fused.v_ch0 = ctx->n_k;
    fused.dump_s = nullptr;
    fused.dump_u = nullptr;
    fused.qpart = (int64_t)table->n_requests * (SR_CONV_W - 1) <= 256 ? (float*)(base + lay.off_qpart) : nullptr;
    fused.tile_sched = base + lay.off_sched;
    fused.hist = nullptr;
    fused.in_ssm_layer = nullptr;
    fused.in_ssm_slot_stride = 0;
    fused.x8 = ctx->w8a8 ? (const uint8_t*)(base + lay.off_x16) : nullptr;
    fused.sx = ctx->w8a8 ? (const float*)(base + lay.off_sx) : nullptr;
    fused.x16 = ctx->fp16_stage ? (const __half*)(base + lay.off_x16) : nullptr;
    fused.w16 = ctx->fp16_stage ? (const __half*)(base + lay.off_wdec) : nullptr;
    const int pl = pool->layer_to_pool[l];
    char* ssm_l = (char*)out_ssm->base + (int64_t)l * out_ssm->layer_stride_bytes;
    char* conv_l = (char*)out_conv->base + (int64_t)l * out_conv->layer_stride_bytes;
    void* wdec = base + lay.off_wdec;
    void* split = base + lay.off_split;
    status = SR_ERR_CUDA;       // any early exit below is a failed CUDA call; the lanes are still joined
    do {
      if (hooks && !hooks->before(hooks->user, l, pl, ls)) break;
      if (in_conv && batched) fused.hist = (__nv_bfloat16*)(base + lay.off_hist);     // gathered before the batch
      if (in_conv && !batched) {
        __nv_bfloat16* hist = (__nv_bfloat16*)(base + lay.off_hist);
        SrLaunchScope scope(ctx, ls, SR_KERNEL_CONV_TAIL);
        if (sr_launch_hist_gather(ctx, sched, (const char*)in_conv->base + (int64_t)l * in_conv->layer_stride_bytes,
                                  in_conv->slot_stride_bytes, hist, ls) != cudaSuccess)
          break;
        fused.hist = hist;
      }
      if (in_ssm) {
        fused.in_ssm_layer = (const char*)in_ssm->base + (int64_t)l * in_ssm->layer_stride_bytes;
        fused.in_ssm_slot_stride = in_ssm->slot_stride_bytes;
      }
      if (ctx->fp16_stage) {
        {
          SrLaunchScope scope(ctx, ls, SR_KERNEL_WEIGHT_DECODE);
          if (sr_launch_stage_weights_fp16(ctx, weights[l], (__half*)wdec, ls) != cudaSuccess) break;
        }
        SrLaunchScope scope(ctx, ls, SR_KERNEL_ANCHOR_STAGE);
        if (sr_launch_stage_anchors_fp16(ctx, sched, pv, pl, (__half*)(base + lay.off_x16), ls) != cudaSuccess) break;
      } else if (ctx->w8a8) {
        SrLaunchScope scope(ctx, ls, SR_KERNEL_ANCHOR_STAGE);
        if (sr_launch_quant_anchors_e4m3(ctx, sched, pv, pl, (uint8_t*)(base + lay.off_x16), (float*)(base + lay.off_sx), ls) !=
            cudaSuccess)
          break;
      } else if (ctx->wdec_bytes) {
        SrLaunchScope scope(ctx, ls, SR_KERNEL_WEIGHT_DECODE);
        if (sr_launch_weight_decode(ctx, weights[l], wdec, ls) != cudaSuccess) break;
      }
      if (!batched) {
        SrLaunchScope scope(ctx, ls, SR_KERNEL_PROJECTION, ctx->w8a8 ? 2 : 1);
        if (sr_launch_proj_fused(ctx, sched, *pool, pl, weights[l], ctx->wdec_bytes ? wdec : nullptr, fused, sm_count,
                                 ls) != cudaSuccess)
          break;
      }
      {
        SrLaunchScope scope(ctx, ls, SR_KERNEL_CONV_TAIL, sr_conv_tail_launches(ctx, sched.n_requests));
        if (sr_launch_conv_tail(ctx, sched, pv, pl, weights[l], fused, conv_l, out_conv->slot_stride_bytes, ls) !=
            cudaSuccess)
          break;
      }
      {
        SrLaunchScope scope(ctx, ls, SR_KERNEL_CHUNK_LOCAL);
        if (sr_launch_chunk_local(ctx, sched, weights[l], fused, split, ls) != cudaSuccess) break;
      }
      {
        SrLaunchScope scope(ctx, ls, SR_KERNEL_SCAN);
        if (sr_launch_scan_chain_umma(ctx, sched, fused, split, ssm_l, out_ssm->slot_stride_bytes, sm_count, ls) != cudaSuccess)
          break;
      }
      if (hooks && !hooks->after(hooks->user, l, ls)) break;
      status = SR_OK;
    } while (false);
  }
  // join: whatever happened above, `stream` resumes only after every lane's work
  if (!join()) status = SR_ERR_CUDA;
  return status;
}
}  // namespace

extern "C" {

int sr_replay_states(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                     const int32_t* replay_lens, const uint8_t* layer_mask, const sr_layer_weights* weights,
                     const sr_out* out_ssm, const sr_out* out_conv, void* workspace, size_t workspace_bytes,
                     void* stream_) {
  return replay_impl(ctx, pool, table, replay_lens, layer_mask, weights, out_ssm, out_conv, workspace,
                     workspace_bytes, stream_, nullptr);
}

int sr_replay_states_from(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                          const int32_t* replay_lens, const uint8_t* layer_mask, const sr_layer_weights* weights,
                          const sr_out* in_ssm, const sr_out* in_conv, const sr_out* out_ssm, const sr_out* out_conv,
                          void* workspace, size_t workspace_bytes, void* stream_) {
  return replay_impl(ctx, pool, table, replay_lens, layer_mask, weights, out_ssm, out_conv, workspace,
                     workspace_bytes, stream_, nullptr, in_ssm, in_conv);
}

int sr_profile_enable(sr_ctx* ctx, int enable) {
  if (!ctx) return SR_ERR_INVALID_ARG;
  ctx->profiling = enable != 0;
  return SR_OK;
}

int sr_profile_read(sr_ctx* ctx, int kind, float* out_ms, int64_t* out_launches) {
  if (!ctx || !out_ms || !out_launches || kind < 0 || kind >= SR_KERNEL_KINDS) return SR_ERR_INVALID_ARG;
  float total = 0.f;
  int64_t n = 0;
  for (size_t b = 0; b * 2 + 1 < ctx->ev_used; ++b) {
    if (ctx->ev_kind[b] != kind) continue;
    if (cudaEventSynchronize(ctx->ev_pool[2 * b + 1]) != cudaSuccess) return SR_ERR_CUDA;
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, ctx->ev_pool[2 * b], ctx->ev_pool[2 * b + 1]) != cudaSuccess) return SR_ERR_CUDA;
    total += ms;
    ++n;
  }
  *out_ms = total;
  *out_launches = n;
  return SR_OK;
}

}  // extern "C"

namespace {
// State of one sr_replay_states_host call: the anchor pool goes up one pool layer at a time on its own stream
// and the outputs come back one layer at a time on another, so both directions overlap the kernels.
struct HostPipe {
  sr_ctx* ctx;
  const sr_out* out_ssm;
  const sr_out* out_conv;
  char* host_ssm;
  char* host_conv;
  size_t ssm_layer_bytes, conv_layer_bytes;
  size_t ssm_slots, conv_slots;
  std::vector<int> slab_event;      // per pool layer: index into ctx->ev_copy of "slab arrived", or -1
  size_t next_event;
};

cudaEvent_t pipe_event(sr_ctx* ctx, size_t i) {
  while (ctx->ev_copy.size() <= i) {
    cudaEvent_t e;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    ctx->ev_copy.push_back(e);
  }
  return ctx->ev_copy[i];
}

bool pipe_before(void* user, int, int pool_layer, cudaStream_t stream) {
  HostPipe* hp = (HostPipe*)user;
  const int ev = hp->slab_event[pool_layer];
  return ev >= 0 && cudaStreamWaitEvent(stream, hp->ctx->ev_copy[ev], 0) == cudaSuccess;
}

bool pipe_after(void* user, int layer, cudaStream_t stream) {
  HostPipe* hp = (HostPipe*)user;
  sr_ctx* ctx = hp->ctx;
  cudaEvent_t done = pipe_event(ctx, hp->next_event++);
  if (!done || cudaEventRecord(done, stream) != cudaSuccess) return false;
  if (cudaStreamWaitEvent(ctx->copy_out, done, 0) != cudaSuccess) return false;
  const int64_t so = (int64_t)layer * hp->out_ssm->layer_stride_bytes, co = (int64_t)layer * hp->out_conv->layer_stride_bytes;
  if (cudaMemcpy2DAsync(hp->host_ssm + so, (size_t)hp->out_ssm->slot_stride_bytes, (const char*)hp->out_ssm->base + so,
                        (size_t)hp->out_ssm->slot_stride_bytes, hp->ssm_layer_bytes, hp->ssm_slots, cudaMemcpyDeviceToHost,
                        ctx->copy_out) != cudaSuccess)
    return false;
  return cudaMemcpy2DAsync(hp->host_conv + co, (size_t)hp->out_conv->slot_stride_bytes,
                           (const char*)hp->out_conv->base + co, (size_t)hp->out_conv->slot_stride_bytes,
                           hp->conv_layer_bytes, hp->conv_slots, cudaMemcpyDeviceToHost, ctx->copy_out) == cudaSuccess;
}
}  // namespace

extern "C" {

int sr_replay_states_host(sr_ctx* ctx, const void* host_pool, size_t pool_bytes, const int32_t* host_pages,
                          const int32_t* host_state_slots, const int32_t* host_replay_lens,
                          int32_t* dev_replay_lens, const sr_anchor_pool* pool, const sr_page_table* table,
                          const uint8_t* layer_mask, const sr_layer_weights* weights, const sr_out* out_ssm,
                          size_t out_ssm_bytes, void* host_out_ssm, const sr_out* out_conv, size_t out_conv_bytes,
                          void* host_out_conv, void* workspace, size_t workspace_bytes, void* stream_) {
  int st = check_batch(ctx, table);
  if (st != SR_OK) return st;
  if (!host_pool || !host_pages || !host_replay_lens || !dev_replay_lens || !pool || !pool->base || !table->pages ||
      !out_ssm || !out_conv || !host_out_ssm || !host_out_conv || !layer_mask)
    return SR_ERR_INVALID_ARG;
  if ((host_state_slots == nullptr) != (table->state_slots == nullptr)) return SR_ERR_INVALID_ARG;
  // everything the host can check, before the first copy is enqueued
  st = validate_call(ctx, pool, table, dev_replay_lens, layer_mask, weights, out_ssm, out_conv, workspace, workspace_bytes,
                     nullptr, nullptr);
  if (st != SR_OK) return st;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (!ctx->copy_in && cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking) != cudaSuccess) return SR_ERR_CUDA;
  if (!ctx->copy_out && cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking) != cudaSuccess) return SR_ERR_CUDA;
  const size_t n = (size_t)table->n_requests;

  HostPipe hp;
  hp.ctx = ctx;
  hp.out_ssm = out_ssm;
  hp.out_conv = out_conv;
  hp.host_ssm = (char*)host_out_ssm;
  hp.host_conv = (char*)host_out_conv;
  hp.next_event = 0;
  size_t ssm_layer = 0, conv_layer = 0;
  sr_ssm_bytes_per_layer(ctx, &ssm_layer);
  sr_conv_bytes_per_layer(ctx, &conv_layer);
  hp.ssm_layer_bytes = ssm_layer;
  hp.conv_layer_bytes = conv_layer;
  // whole slots inside the byte counts given: the 2-D copies never leave [base, base + bytes)
  if (out_ssm->slot_stride_bytes <= 0 || out_conv->slot_stride_bytes <= 0) return SR_ERR_INVALID_ARG;
  hp.ssm_slots = out_ssm_bytes / (size_t)out_ssm->slot_stride_bytes;
  hp.conv_slots = out_conv_bytes / (size_t)out_conv->slot_stride_bytes;

  // the copies may start once everything already queued on `stream` (earlier readers of the staging buffers) is done
  cudaEvent_t start = pipe_event(ctx, hp.next_event++);
  if (!start || cudaEventRecord(start, stream) != cudaSuccess) return SR_ERR_CUDA;
  if (cudaStreamWaitEvent(ctx->copy_in, start, 0) != cudaSuccess) return SR_ERR_CUDA;
  if (cudaStreamWaitEvent(ctx->copy_out, start, 0) != cudaSuccess) return SR_ERR_CUDA;
  if (n) {
    if (cudaMemcpyAsync((void*)table->pages, host_pages, n * table->max_pages * sizeof(int32_t),
                        cudaMemcpyHostToDevice, stream) != cudaSuccess)
      return SR_ERR_CUDA;
    if (cudaMemcpyAsync(dev_replay_lens, host_replay_lens, n * sizeof(int32_t), cudaMemcpyHostToDevice, stream) !=
        cudaSuccess)
      return SR_ERR_CUDA;
    if (host_state_slots &&
        cudaMemcpyAsync((void*)table->state_slots, host_state_slots, n * sizeof(int32_t), cudaMemcpyHostToDevice,
                        stream) != cudaSuccess)
      return SR_ERR_CUDA;
  }
  // anchors: one strided copy per pool layer that a rebuilt layer reads, in the order the layers run; a layout
  // whose page blocks are not contiguous, or that does not fit the byte count given, goes up in one piece
  hp.slab_event.assign((size_t)pool->n_pool_layers, -1);
  const size_t block = (size_t)SR_PAGE_ROWS * (size_t)pool->row_stride_bytes;
  const size_t pitch = pool->n_phys_pages > 1 ? (size_t)pool->page_stride_bytes : block;
  bool sliced = block <= pitch;
  for (int pl = 0; pl < pool->n_pool_layers && sliced; ++pl)
    sliced = (size_t)pl * (size_t)pool->layer_stride_bytes + (size_t)(pool->n_phys_pages - 1) * pitch + block <= pool_bytes;
  if (!sliced) {
    cudaEvent_t all = pipe_event(ctx, hp.next_event);
    if (!all || cudaMemcpyAsync((void*)pool->base, host_pool, pool_bytes, cudaMemcpyHostToDevice, ctx->copy_in) != cudaSuccess ||
        cudaEventRecord(all, ctx->copy_in) != cudaSuccess)
      return SR_ERR_CUDA;
    hp.slab_event.assign((size_t)pool->n_pool_layers, (int)hp.next_event);
    hp.next_event++;
  } else {
    for (int l = 0; l < ctx->desc.n_layers; ++l) {
      if (!layer_mask[l]) continue;
      const int pl = pool->layer_to_pool[l];
      if (pl < 0 || pl >= pool->n_pool_layers) return SR_ERR_INVALID_ARG;
      if (hp.slab_event[pl] >= 0) continue;
      const size_t off = (size_t)pl * (size_t)pool->layer_stride_bytes;
      cudaEvent_t arrived = pipe_event(ctx, hp.next_event);
      if (!arrived ||
          cudaMemcpy2DAsync((char*)pool->base + off, pitch, (const char*)host_pool + off, pitch, block,
                            (size_t)pool->n_phys_pages, cudaMemcpyHostToDevice, ctx->copy_in) != cudaSuccess ||
          cudaEventRecord(arrived, ctx->copy_in) != cudaSuccess)
        return SR_ERR_CUDA;
      hp.slab_event[pl] = (int)hp.next_event++;
    }
  }
  LayerHooks hooks = {&hp, pipe_before, pipe_after};
  st = replay_impl(ctx, pool, table, dev_replay_lens, layer_mask, weights, out_ssm, out_conv, workspace, workspace_bytes,
                   stream_, &hooks);
  // layers that were not rebuilt are not copied back; `stream` resumes when both copy streams are done -- also
  // after a failed launch, so that no copy of this call is left running behind the caller's back
  cudaEvent_t in_done = pipe_event(ctx, hp.next_event++), out_done = pipe_event(ctx, hp.next_event++);
  if (!in_done || !out_done || cudaEventRecord(in_done, ctx->copy_in) != cudaSuccess ||
      cudaEventRecord(out_done, ctx->copy_out) != cudaSuccess || cudaStreamWaitEvent(stream, in_done, 0) != cudaSuccess ||
      cudaStreamWaitEvent(stream, out_done, 0) != cudaSuccess)
    return SR_ERR_CUDA;
  return st;
}

int sr_anchor_write(sr_ctx* ctx, const sr_anchor_pool* pool, const int32_t* pool_layers, int32_t n_layers,
                    const void* hidden, int64_t hidden_layer_stride_bytes, int64_t hidden_row_stride_bytes,
                    const int32_t* dest_page, const int32_t* dest_row, int32_t n_tokens, uint32_t* status,
                    void* stream_) {
  if (!ctx || !pool_layers || !dest_page || !dest_row || n_layers < 0 || n_tokens < 0) return SR_ERR_INVALID_ARG;
  int st = check_pool(ctx, pool);
  if (st != SR_OK) return st;
  if (n_layers == 0 || n_tokens == 0) return SR_OK;
  if (!hidden || !aligned(hidden, 16) || hidden_row_stride_bytes % 16 || hidden_layer_stride_bytes % 16 ||
      hidden_row_stride_bytes < (int64_t)ctx->desc.d_model * 2)
    return SR_ERR_INVALID_ARG;
  for (int32_t i = 0; i < n_layers; ++i)
    if (pool_layers[i] < 0 || pool_layers[i] >= pool->n_pool_layers) return SR_ERR_INVALID_ARG;
  if (sr_launch_anchor_write(*pool, pool_layers, n_layers, hidden, hidden_layer_stride_bytes, hidden_row_stride_bytes,
                             dest_page, dest_row, n_tokens, ctx->desc.d_model, status, (cudaStream_t)stream_) !=
      cudaSuccess)
    return SR_ERR_CUDA;
  return SR_OK;
}

int sr_debug_gather(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
                    int32_t layer, void* out_rows, int64_t out_capacity_rows, void* workspace,
                    size_t workspace_bytes, void* stream_) {
  int st = check_batch(ctx, table);
  if (st != SR_OK) return st;
  if (!replay_lens || !out_rows || !table->pages || out_capacity_rows < 0) return SR_ERR_INVALID_ARG;
  st = check_pool(ctx, pool);
  if (st != SR_OK) return st;
  if (layer < 0 || layer >= ctx->desc.n_layers || pool->layer_to_pool[layer] < 0) return SR_ERR_INVALID_ARG;
  if (!aligned(out_rows, 16)) return SR_ERR_INVALID_ARG;
  const SrWorkspace lay = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < lay.total) return SR_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)stream_;
  ctx->last_launches = 0;
  if (table->n_requests == 0 || table->max_pages == 0) return SR_OK;
  SrSched sched = sr_sched_view(workspace, lay, table->n_requests);
  sched.check_bounds = (ctx->debug_flags & SR_DEBUG_CHECK_BOUNDS) ? 1 : 0;
  sched.n_phys_pages = pool->n_phys_pages;
  ctx->ev_used = 0;
  ctx->ev_kind.clear();
  if (sr_launch_schedule(sched, table->pages, table->state_slots, replay_lens, table->max_pages,
                         table->max_replay_len, table->max_total_rows, pool->n_phys_pages, table->n_state_slots,
                           stream) != cudaSuccess)
    return SR_ERR_CUDA;
  if (sr_launch_debug_gather(sched, pool_view(pool), pool->layer_to_pool[layer], ctx->desc.d_model, table->max_pages,
                             out_rows, out_capacity_rows, stream) != cudaSuccess)
    return SR_ERR_CUDA;
  ctx->last_launches = 2;
  return SR_OK;
}

int sr_debug_quantise(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
                      int32_t layer, void* out_codes, float* out_scales, int64_t out_capacity_rows, void* workspace,
                      size_t workspace_bytes, void* stream_) {
  int st = check_batch(ctx, table);
  if (st != SR_OK) return st;
  if (!ctx->w8a8) return SR_ERR_UNSUPPORTED_SHAPE;
  if (!replay_lens || !out_codes || !out_scales || !table->pages || out_capacity_rows < 0) return SR_ERR_INVALID_ARG;
  st = check_pool(ctx, pool);
  if (st != SR_OK) return st;
  if (layer < 0 || layer >= ctx->desc.n_layers || pool->layer_to_pool[layer] < 0) return SR_ERR_INVALID_ARG;
  if (!aligned(out_codes, 16) || !aligned(out_scales, 4)) return SR_ERR_INVALID_ARG;
  const SrWorkspace lay = sr_workspace_layout(ctx, table->n_requests, table->max_pages, table->max_total_rows);
  if (!workspace || !aligned(workspace, 256) || workspace_bytes < lay.total) return SR_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)stream_;
  ctx->last_launches = 0;
  if (table->n_requests == 0 || table->max_pages == 0) return SR_OK;
  SrSched sched = sr_sched_view(workspace, lay, table->n_requests);
  sched.n_phys_pages = pool->n_phys_pages;
  ctx->ev_used = 0;
  ctx->ev_kind.clear();
  uint8_t* x8 = (uint8_t*)workspace + lay.off_x16;
  float* sx = (float*)((char*)workspace + lay.off_sx);
  if (sr_launch_schedule(sched, table->pages, table->state_slots, replay_lens, table->max_pages, table->max_replay_len,
                         table->max_total_rows, pool->n_phys_pages, table->n_state_slots, stream) != cudaSuccess ||
      sr_launch_quant_anchors_e4m3(ctx, sched, pool_view(pool), pool->layer_to_pool[layer], x8, sx, stream) != cudaSuccess ||
      sr_launch_pack_quantised(ctx, sched, table->max_pages, x8, sx, out_codes, out_scales, out_capacity_rows, stream) !=
          cudaSuccess)
    return SR_ERR_CUDA;
  ctx->last_launches = 3;
  return SR_OK;
}

int sr_device_status(sr_ctx* ctx, const void* workspace, void* stream_, uint32_t* out_flags) {
  if (!ctx || !workspace || !out_flags) return SR_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  uint32_t v = 0;
  if (cudaMemcpyAsync(&v, workspace, sizeof(v), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return SR_ERR_CUDA;
  if (cudaStreamSynchronize(stream) != cudaSuccess) return SR_ERR_CUDA;
  *out_flags = v;
  return SR_OK;
}

int sr_last_launch_count(const sr_ctx* ctx, int64_t* out_launches) {
  if (!ctx || !out_launches) return SR_ERR_INVALID_ARG;
  *out_launches = ctx->last_launches;
  return SR_OK;
}

}  // extern "C"
