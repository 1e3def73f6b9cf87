// Group-propagated replay (Section 4.1): the launch sequence that rebuilds the states of a group of consecutive
// linear-attention layers from the group-entry anchors.  Per layer: row norm -> q | k | v projection with the conv
// fused behind it -> conv state -> chunk-local -> state chain (which also leaves the state entering every chunk and
// the chunk's pseudo-values) and, for every layer but the last: output gate GEMM -> per-token outputs, head norm and
// gate -> output projection + residual [-> row norm -> gate/up GEMM with SwiGLU -> down projection + residual].
// No arithmetic lives here.
#include "sr_common.cuh"

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) % 16) == 0; }

struct GroupLayout {
  SrWorkspace base;      // header and tables as for sr_replay_states (its per-layer block is not used)
  // offsets inside one group's block of scratch; block i of a call sits at tables_end + i * block_bytes
  size_t off_qkv16, off_zraw, off_gates, off_split, off_dump_s, off_dump_u, off_x, off_r0, off_r1, off_zg, off_y, off_hid, off_sched;
  size_t tables_end, block_bytes;
  int ncb;
  size_t total(int blocks) const { return tables_end + block_bytes * (size_t)blocks; }
};

GroupLayout group_layout(const sr_ctx* ctx, const sr_page_table* t, int32_t max_d_ff) {
  GroupLayout g;
  g.base = sr_workspace_layout(ctx, t->n_requests, t->max_pages, t->max_total_rows, 1);
  const size_t slots = (size_t)g.base.max_slots, rows = slots * SR_PAGE_ROWS;
  const sr_model_desc& d = ctx->desc;
  g.ncb = (ctx->conv_ch + 127) / 128;
  const size_t hv = (size_t)d.n_v_heads * d.d_v;
  g.tables_end = g.base.off_kv16;
  size_t at = 0;
  auto take = [&](size_t bytes) { const size_t o = at; at = (at + bytes + 1023) & ~size_t(1023); return o; };
  g.off_qkv16 = take(rows * (size_t)g.ncb * 128 * 2);
  g.off_zraw = take(slots * 6 * (size_t)ctx->conv_ch * 4);
  g.off_gates = take(rows * (size_t)ctx->n_gate * 4);
  g.off_split = take(sr_scan_split_bytes(ctx, g.base.max_slots));
  g.off_dump_s = take(slots * d.n_v_heads * (size_t)d.d_k * d.d_v * 2);
  g.off_dump_u = take(slots * d.n_v_heads * (size_t)d.d_v * SR_PAGE_ROWS * 2);
  g.off_x = take(rows * (size_t)d.d_model * 2);
  g.off_r0 = take(rows * (size_t)d.d_model * 2);
  g.off_r1 = take(rows * (size_t)d.d_model * 2);
  g.off_zg = take(rows * hv * 2);
  g.off_y = take(rows * hv * 2);
  g.off_hid = take(rows * (size_t)(max_d_ff > 0 ? max_d_ff : 0) * 2);
  g.off_sched = take(SR_TILE_SCHED_BYTES);
  g.block_bytes = at;
  return g;
}

// Groups in flight at once (each on a stream of the context with its own block of scratch): as many, up to
// SR_MAX_LANES and the number of groups, as keep the blocks together within SR_LANES_BUDGET_BYTES.
int group_lanes(const GroupLayout& lay, int n_groups) {
  int lanes = SR_MAX_LANES;
  while (lanes > 1 && ((size_t)lanes * lay.block_bytes > SR_LANES_BUDGET_BYTES || lanes > n_groups)) lanes >>= 1;
  return lanes;
}

int check_group_ctx(const sr_ctx* ctx, const sr_page_table* t) {
  if (!ctx || !t) return SR_ERR_INVALID_ARG;
  if (!ctx->kernels_cover || ctx->desc.weight_format != SR_W_BF16 || !sr_group_output_supported(ctx->desc.d_k, ctx->desc.d_v) ||
      (ctx->desc.n_v_heads * ctx->desc.d_v) % 64 != 0 || ctx->desc.d_model % 64 != 0)
    return SR_ERR_UNSUPPORTED_SHAPE;
  if (t->n_requests < 0 || t->n_requests > 65535 || t->max_pages < 0 || t->max_replay_len < 0 || t->max_total_rows < 0 ||
      t->n_state_slots < 0 || (int64_t)t->max_replay_len > (int64_t)t->max_pages * SR_PAGE_ROWS)
    return SR_ERR_INVALID_ARG;
  if (sr_workspace_layout(ctx, t->n_requests, t->max_pages, t->max_total_rows, 1).max_slots > 65535) return SR_ERR_UNSUPPORTED_SHAPE;
  return SR_OK;
}

}  // namespace

extern "C" int sr_group_workspace_bytes(const sr_ctx* ctx, const sr_page_table* table, int32_t max_d_ff, size_t* out_bytes) {
  if (!out_bytes || max_d_ff < 0) return SR_ERR_INVALID_ARG;
  const int st = check_group_ctx(ctx, table);
  if (st != SR_OK) return st;
  *out_bytes = group_layout(ctx, table, max_d_ff).total(1);
  return SR_OK;
}

extern "C" int sr_groups_workspace_bytes(const sr_ctx* ctx, const sr_page_table* table, int32_t max_d_ff, int32_t n_groups,
                                         size_t* out_bytes) {
  if (!out_bytes || max_d_ff < 0 || n_groups < 1) return SR_ERR_INVALID_ARG;
  const int st = check_group_ctx(ctx, table);
  if (st != SR_OK) return st;
  const GroupLayout lay = group_layout(ctx, table, max_d_ff);
  *out_bytes = lay.total(group_lanes(lay, n_groups));
  return SR_OK;
}

namespace {

// host-side checks shared by the two entries (nothing is launched before they pass)
int check_call(const sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
               const sr_layer_weights* weights, const sr_block_weights* blocks, float norm_eps, const sr_out* out_ssm,
               const sr_out* out_conv) {
  const int st = check_group_ctx(ctx, table);
  if (st != SR_OK) return st;
  const sr_model_desc& d = ctx->desc;
  if (!pool || !pool->base || !pool->layer_to_pool || !replay_lens || !weights || !blocks || !out_ssm || !out_conv ||
      !table->pages || !out_ssm->base || !out_conv->base || !(norm_eps >= 0.f))
    return SR_ERR_INVALID_ARG;
  if (!aligned16(out_ssm->base) || out_ssm->slot_stride_bytes % 16 || out_ssm->layer_stride_bytes % 16 ||
      out_conv->slot_stride_bytes % 2 || out_conv->layer_stride_bytes % 2 || !aligned16(pool->base) ||
      pool->row_stride_bytes % 16 || pool->layer_stride_bytes % 16 || pool->page_stride_bytes % 16 ||
      pool->row_stride_bytes < (int64_t)d.d_model * 2 || pool->n_phys_pages <= 0 || pool->n_pool_layers <= 0)
    return SR_ERR_INVALID_ARG;
  return SR_OK;
}

// one group's layers and weights; *max_ff receives the widest MLP the group runs
int check_group(const sr_ctx* ctx, const sr_anchor_pool* pool, int32_t first_layer, int32_t n_group_layers,
                const sr_layer_weights* weights, const sr_block_weights* blocks, int32_t* max_ff) {
  if (first_layer < 0 || n_group_layers < 1 || first_layer + n_group_layers > ctx->desc.n_layers) return SR_ERR_INVALID_ARG;
  const int pl = pool->layer_to_pool[first_layer];
  if (pl < 0 || pl >= pool->n_pool_layers) return SR_ERR_INVALID_ARG;      // the group has no anchors
  for (int j = 0; j < n_group_layers; ++j) {
    const sr_layer_weights& w = weights[first_layer + j];
    const sr_block_weights& b = blocks[first_layer + j];
    if (!w.w_qkv || !w.w_ab || !w.conv_w || !w.decay_scale || !w.dt_bias || !b.norm_w) return SR_ERR_INVALID_ARG;
    if (!aligned16(w.w_qkv) || !aligned16(w.w_ab) || !aligned16(w.conv_w) || !aligned16(b.norm_w)) return SR_ERR_INVALID_ARG;
    if (j + 1 == n_group_layers) break;                   // the last layer's output is never formed
    if (!b.w_z || !b.o_norm_w || !b.w_o || !aligned16(b.w_z) || !aligned16(b.w_o)) return SR_ERR_INVALID_ARG;
    if (b.mlp_norm_w) {
      if (!b.w_gate || !b.w_up || !b.w_down || b.d_ff <= 0 || b.d_ff % 64 || !aligned16(b.w_gate) || !aligned16(b.w_up) ||
          !aligned16(b.w_down) || !aligned16(b.mlp_norm_w))
        return SR_ERR_INVALID_ARG;
      if (b.d_ff > *max_ff) *max_ff = b.d_ff;
    }
  }
  return SR_OK;
}

struct GroupCall {
  sr_ctx* ctx;
  const sr_anchor_pool* pool;
  SrSched sched;
  SrPoolView pv;
  const GroupLayout* lay;
  const sr_layer_weights* weights;
  const sr_block_weights* blocks;
  float norm_eps;
  const sr_out* out_ssm;
  const sr_out* out_conv;
  int sm_count;
};

// The launches of one group on `stream`, with the group's scratch at `ws` (one block of the layout).  `side`: a
// stream of the context for the output-gate GEMM (joined before the per-token outputs), or null = everything in order
// on `stream`; `fork` / `join`: the events of that detour.
int run_group(const GroupCall& c, char* ws, int32_t first_layer, int32_t n_group_layers, void* debug_rows,
              cudaStream_t stream, cudaStream_t side_stream, cudaEvent_t fork, cudaEvent_t join) {
  sr_ctx* ctx = c.ctx;
  const sr_model_desc& d = ctx->desc;
  const GroupLayout& lay = *c.lay;
  const SrSched& sched = c.sched;
  const SrPoolView& pv = c.pv;
  const sr_layer_weights* weights = c.weights;
  const sr_block_weights* blocks = c.blocks;
  const float norm_eps = c.norm_eps;
  const sr_out* out_ssm = c.out_ssm;
  const sr_out* out_conv = c.out_conv;
  const int sm_count = c.sm_count;
  const bool side = side_stream != nullptr && n_group_layers > 1;
  const int pl = c.pool->layer_to_pool[first_layer];

  SrFused fused;
  fused.hist = nullptr;
  fused.in_ssm_layer = nullptr;
  fused.in_ssm_slot_stride = 0;
  fused.x8 = nullptr; fused.sx = nullptr; fused.x16 = nullptr; fused.w16 = nullptr;
  fused.kv16 = (__half*)(ws + lay.off_qkv16);
  fused.zraw = (float*)(ws + lay.off_zraw);
  fused.gates = (float*)(ws + lay.off_gates);
  fused.tile_sched = ws + lay.off_sched;
  fused.ncb = lay.ncb;
  fused.n_kv = ctx->conv_ch;
  fused.n_gate = ctx->n_gate;
  fused.fix_mod = 4;
  fused.x_slot_order = 1;
  fused.with_q = 1;
  fused.k_ch0 = ctx->n_k;
  fused.v_ch0 = 2 * ctx->n_k;
  fused.dump_s = (__half*)(ws + lay.off_dump_s);
  fused.dump_u = (__half*)(ws + lay.off_dump_u);
  fused.qpart = nullptr;
  void* split = ws + lay.off_split;
  __nv_bfloat16* x = (__nv_bfloat16*)(ws + lay.off_x);
  __nv_bfloat16* r_cur = (__nv_bfloat16*)(ws + lay.off_r0);
  __nv_bfloat16* r_nxt = (__nv_bfloat16*)(ws + lay.off_r1);
  __nv_bfloat16* zg = (__nv_bfloat16*)(ws + lay.off_zg);
  __nv_bfloat16* y = (__nv_bfloat16*)(ws + lay.off_y);
  __nv_bfloat16* hid = (__nv_bfloat16*)(ws + lay.off_hid);
  const int64_t dm = d.d_model, hv = (int64_t)d.n_v_heads * d.d_v;
  const size_t row_bytes = (size_t)lay.base.max_slots * SR_PAGE_ROWS * dm * 2;

  // the packed rows x as the projection's "pool": one pool layer, page = slot
  sr_anchor_pool xpool;
  xpool.base = x;
  xpool.row_stride_bytes = dm * 2;
  xpool.layer_stride_bytes = (int64_t)SR_PAGE_ROWS * dm * 2;
  xpool.page_stride_bytes = (int64_t)SR_PAGE_ROWS * dm * 2;
  xpool.n_phys_pages = (int32_t)lay.base.max_slots;
  xpool.n_pool_layers = 1;
  xpool.layer_to_pool = c.pool->layer_to_pool;

  for (int j = 0; j < n_group_layers; ++j) {
    const int l = first_layer + j;
    const sr_layer_weights& w = weights[l];
    const sr_block_weights& b = blocks[l];
    const bool last = j + 1 == n_group_layers;
    char* ssm_l = (char*)out_ssm->base + (int64_t)l * out_ssm->layer_stride_bytes;
    char* conv_l = (char*)out_conv->base + (int64_t)l * out_conv->layer_stride_bytes;
    {
      // layer input x = RMSNorm(r); the first layer reads the anchors through the page table and also leaves the
      // residual rows in packed order for the residual add
      SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
      if (sr_launch_rmsnorm_rows(sched, pv, pl, j == 0 ? nullptr : r_cur, (const __nv_bfloat16*)b.norm_w, norm_eps, d.d_model, x,
                                 (j == 0 && !last) ? r_cur : nullptr, stream) != cudaSuccess)
        return SR_ERR_CUDA;
    }
    {
      SrLaunchScope scope(ctx, stream, SR_KERNEL_PROJECTION);
      if (sr_launch_proj_fused(ctx, sched, xpool, 0, w, nullptr, fused, sm_count, stream) != cudaSuccess) return SR_ERR_CUDA;
    }
    if (side && !last) {
      // The output gate SiLU(x W_z^T) needs only x: it runs on a side stream of the context next to the conv-state,
      // chunk-local and chain kernels, which leave most of the GPU idle on a serving-size batch; the caller's stream
      // waits for it before the per-token outputs.
      cudaStream_t ss = side_stream;
      if (cudaEventRecord(fork, stream) != cudaSuccess || cudaStreamWaitEvent(ss, fork, 0) != cudaSuccess)
        return SR_ERR_CUDA;
      cudaError_t e;
      {
        SrLaunchScope scope(ctx, ss, SR_KERNEL_GROUP_BLOCK);
        e = sr_launch_rows_gemm(sched, 1, x, dm, b.w_z, nullptr, (int32_t)hv, zg, hv, nullptr, 0, sm_count, ss);
      }
      // joined whatever happened, so the call stays one unit of work on `stream`
      if (cudaEventRecord(join, ss) != cudaSuccess || e != cudaSuccess) {
        cudaStreamWaitEvent(stream, join, 0);
        return SR_ERR_CUDA;
      }
    }
    {
      SrLaunchScope scope(ctx, stream, SR_KERNEL_CONV_TAIL);
      if (sr_launch_conv_tail_from_raw(ctx, sched, fused, conv_l, out_conv->slot_stride_bytes, stream) != cudaSuccess)
        return SR_ERR_CUDA;
    }
    {
      SrLaunchScope scope(ctx, stream, SR_KERNEL_CHUNK_LOCAL);
      if (sr_launch_chunk_local(ctx, sched, w, fused, split, stream) != cudaSuccess) return SR_ERR_CUDA;
    }
    {
      SrLaunchScope scope(ctx, stream, SR_KERNEL_SCAN);
      SrFused f2 = fused;
      if (last) { f2.dump_s = nullptr; f2.dump_u = nullptr; }
      if (sr_launch_scan_chain_umma(ctx, sched, f2, split, ssm_l, out_ssm->slot_stride_bytes, sm_count, stream) != cudaSuccess)
        return SR_ERR_CUDA;
    }
    if (last) break;
    if (side) {
      if (cudaStreamWaitEvent(stream, join, 0) != cudaSuccess) return SR_ERR_CUDA;
    } else {
      // output gate SiLU(x W_z^T)
      SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
      if (sr_launch_rows_gemm(sched, 1, x, dm, b.w_z, nullptr, (int32_t)hv, zg, hv, nullptr, 0, sm_count, stream) != cudaSuccess)
        return SR_ERR_CUDA;
    }
    // per-token outputs with head norm and gate, output projection + residual
    {
      SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
      if (sr_launch_group_output(ctx, sched, fused, split, zg, (const __nv_bfloat16*)b.o_norm_w, norm_eps, y, stream) != cudaSuccess)
        return SR_ERR_CUDA;
    }
    {
      SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
      if (sr_launch_rows_gemm(sched, 2, y, hv, b.w_o, nullptr, d.d_model, r_nxt, dm, r_cur, dm, sm_count, stream) != cudaSuccess)
        return SR_ERR_CUDA;
    }
    __nv_bfloat16* t = r_cur; r_cur = r_nxt; r_nxt = t;
    if (b.mlp_norm_w) {
      {
        SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
        if (sr_launch_rmsnorm_rows(sched, pv, 0, r_cur, (const __nv_bfloat16*)b.mlp_norm_w, norm_eps, d.d_model, x, nullptr, stream) !=
            cudaSuccess)
          return SR_ERR_CUDA;
      }
      {
        SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
        if (sr_launch_rows_gemm(sched, 3, x, dm, b.w_gate, b.w_up, b.d_ff, hid, b.d_ff, nullptr, 0, sm_count, stream) != cudaSuccess)
          return SR_ERR_CUDA;
      }
      {
        SrLaunchScope scope(ctx, stream, SR_KERNEL_GROUP_BLOCK);
        if (sr_launch_rows_gemm(sched, 2, hid, b.d_ff, b.w_down, nullptr, d.d_model, r_nxt, dm, r_cur, dm, sm_count, stream) != cudaSuccess)
          return SR_ERR_CUDA;
      }
      t = r_cur; r_cur = r_nxt; r_nxt = t;
    }
    if (debug_rows &&
        cudaMemcpyAsync((char*)debug_rows + (size_t)j * row_bytes, r_cur, row_bytes, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
      return SR_ERR_CUDA;
  }
  return SR_OK;
}

// what both entries do before the groups: counters, views, the packing kernel
int begin_call(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
               const GroupLayout& lay, void* workspace, cudaStream_t stream, GroupCall* c) {
  ctx->last_launches = 0;
  ctx->ev_used = 0;
  ctx->ev_kind.clear();
  if (sr_current_device_sms(&c->sm_count) != cudaSuccess) return SR_ERR_CUDA;
  c->ctx = ctx;
  c->pool = pool;
  c->lay = &lay;
  c->sched = sr_sched_view(workspace, lay.base, table->n_requests);
  c->sched.check_bounds = (ctx->debug_flags & SR_DEBUG_CHECK_BOUNDS) ? 1 : 0;
  c->sched.n_phys_pages = pool->n_phys_pages;
  c->sched.n_state_slots = table->n_state_slots;
  c->pv.base = (const char*)pool->base;
  c->pv.page_stride = pool->page_stride_bytes;
  c->pv.layer_stride = pool->layer_stride_bytes;
  c->pv.row_stride = pool->row_stride_bytes;
  c->pv.n_phys_pages = pool->n_phys_pages;
  SrLaunchScope scope(ctx, stream, SR_KERNEL_SCHEDULE);
  if (sr_launch_schedule(c->sched, table->pages, table->state_slots, replay_lens, table->max_pages, table->max_replay_len,
                         table->max_total_rows, pool->n_phys_pages, table->n_state_slots, stream) != cudaSuccess)
    return SR_ERR_CUDA;
  return SR_OK;
}

}  // namespace

extern "C" int sr_replay_group_states(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                                      const int32_t* replay_lens, int32_t first_layer, int32_t n_group_layers,
                                      const sr_layer_weights* weights, const sr_block_weights* blocks, float norm_eps,
                                      const sr_out* out_ssm, const sr_out* out_conv, void* debug_rows, void* workspace,
                                      size_t workspace_bytes, void* stream_) {
  int st = check_call(ctx, pool, table, replay_lens, weights, blocks, norm_eps, out_ssm, out_conv);
  if (st != SR_OK) return st;
  int32_t max_ff = 0;
  st = check_group(ctx, pool, first_layer, n_group_layers, weights, blocks, &max_ff);
  if (st != SR_OK) return st;
  const GroupLayout lay = group_layout(ctx, table, max_ff);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % 256) || workspace_bytes < lay.total(1)) return SR_ERR_WORKSPACE;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (table->n_requests == 0) { ctx->last_launches = 0; return SR_OK; }
  const bool side = n_group_layers > 1 && sr_ensure_lanes(ctx);
  GroupCall c;
  c.weights = weights; c.blocks = blocks; c.norm_eps = norm_eps; c.out_ssm = out_ssm; c.out_conv = out_conv;
  st = begin_call(ctx, pool, table, replay_lens, lay, workspace, stream, &c);
  if (st != SR_OK) return st;
  return run_group(c, (char*)workspace + lay.tables_end, first_layer, n_group_layers, debug_rows, stream,
                   side ? ctx->lane_stream[0] : nullptr, ctx->lane_fork, side ? ctx->lane_join[0] : nullptr);
}

extern "C" int sr_replay_groups_states(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                                       const int32_t* replay_lens, int32_t n_groups, const int32_t* first_layers,
                                       const int32_t* group_sizes, const sr_layer_weights* weights,
                                       const sr_block_weights* blocks, float norm_eps, const sr_out* out_ssm,
                                       const sr_out* out_conv, void* workspace, size_t workspace_bytes, void* stream_) {
  int st = check_call(ctx, pool, table, replay_lens, weights, blocks, norm_eps, out_ssm, out_conv);
  if (st != SR_OK) return st;
  if (n_groups < 1 || !first_layers || !group_sizes) return SR_ERR_INVALID_ARG;
  int32_t max_ff = 0;
  for (int g = 0; g < n_groups; ++g) {
    st = check_group(ctx, pool, first_layers[g], group_sizes[g], weights, blocks, &max_ff);
    if (st != SR_OK) return st;
    for (int h = 0; h < g; ++h)        // groups write disjoint layers
      if (first_layers[g] < first_layers[h] + group_sizes[h] && first_layers[h] < first_layers[g] + group_sizes[g])
        return SR_ERR_INVALID_ARG;
  }
  const GroupLayout lay = group_layout(ctx, table, max_ff);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) % 256) || workspace_bytes < lay.total(1)) return SR_ERR_WORKSPACE;
  // as many groups side by side as the policy gives and the workspace holds
  int lanes = group_lanes(lay, n_groups);
  while (lanes > 1 && lay.total(lanes) > workspace_bytes) lanes >>= 1;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (table->n_requests == 0) { ctx->last_launches = 0; return SR_OK; }
  if (lanes > 1 && !sr_ensure_lanes(ctx)) return SR_ERR_CUDA;
  GroupCall c;
  c.weights = weights; c.blocks = blocks; c.norm_eps = norm_eps; c.out_ssm = out_ssm; c.out_conv = out_conv;
  st = begin_call(ctx, pool, table, replay_lens, lay, workspace, stream, &c);
  if (st != SR_OK) return st;
  // The groups are independent (each starts from its own anchors): group g goes to lane g mod lanes, a lane being a
  // stream of the context with its own block of scratch; lane 0 is the caller's stream, the others fork from it after
  // the packing kernel and join it at the end, so the call stays one unit of work on `stream`.
  if (lanes > 1) {
    if (cudaEventRecord(ctx->lane_fork, stream) != cudaSuccess) return SR_ERR_CUDA;
    for (int i = 0; i < lanes - 1; ++i)
      if (cudaStreamWaitEvent(ctx->lane_stream[i], ctx->lane_fork, 0) != cudaSuccess) return SR_ERR_CUDA;
  }
  int status = SR_OK;
  for (int g = 0; g < n_groups && status == SR_OK; ++g) {
    const int lane = g % lanes;
    status = run_group(c, (char*)workspace + lay.tables_end + (size_t)lane * lay.block_bytes, first_layers[g], group_sizes[g],
                       nullptr, lane == 0 ? stream : ctx->lane_stream[lane - 1], nullptr, nullptr, nullptr);
  }
  for (int i = 0; i < lanes - 1; ++i)    // joined whatever happened above
    if (cudaEventRecord(ctx->lane_join[i], ctx->lane_stream[i]) != cudaSuccess ||
        cudaStreamWaitEvent(stream, ctx->lane_join[i], 0) != cudaSuccess)
      status = SR_ERR_CUDA;
  return status;
}
