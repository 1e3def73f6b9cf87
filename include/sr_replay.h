/*
 * sr_replay.h -- C boundary of the B200 suffix-replay state builder.
 *
 * The library rebuilds the recurrent state of gated-delta-rule linear-attention layers
 * at a matched prefix-cache page boundary by replaying only the retained anchor hidden
 * states of a recent suffix, from a zero state (paper Eq. 2, "S'_j = f(h_{j-k+1..j})"),
 * for a packed batch of cache hits with different replay lengths (Section 5.2,
 * "Batched replay").  It writes, per (request, rebuilt layer), the two pieces of state a
 * linear-attention layer carries across tokens (Appendix A, "Native cache"):
 *
 *   recurrent state : one d_k x d_v matrix per value head, FP32, row-major [d_k][d_v];
 *   conv state      : the last w-1 inputs of each of the C = 2 H_k d_k + H_v d_v
 *                     convolution channels, BF16, [C][w-1], oldest row first.
 *
 * The recurrence is Eq. 4, S_t = A_t(S_{t-1}) + B_t with S_0 = 0, in its gated-delta
 * form (decay plus rank-one erase, Section 2.1):
 *
 *   S_t = alpha_t (I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T ,  S in R^{d_k x d_v}
 *
 * (the key index is the ROW of S: the state's answer for key k is S^T k).  Keys, values
 * and gates are projections of the layer input h_t (Section 2.1): with X the replayed
 * anchor rows,
 *   Z = X W_qkv^T (channels q | k | v, head-major), G = X W_ab^T (rows a_0.., b_0..);
 *   y = SiLU(causal depthwise conv of width w over Z, zero history, tap w-1 = current row);
 *   k = y_k / sqrt(sum y_k^2 + l2_eps) per (token, key head);  v = y_v;
 *   alpha = exp(-decay_scale[h] * softplus(a + dt_bias[h]));  beta = sigmoid(b);
 *   value head h uses key head h / (H_v / H_k).
 * Per-token outputs of the layer are never computed by sr_replay_states; sr_replay_group_states forms them to feed
 * the next layer of a group.
 *
 * Conventions for every call
 *   - plain C types only; "DEVICE" marks pointers to GPU global memory, "HOST" host memory;
 *   - the caller owns every buffer; the library allocates no device memory, keeps no
 *     pointer after the work it enqueued on `stream` has run, and never frees caller memory;
 *   - calls that launch work are asynchronous on `stream` (a cudaStream_t passed as
 *     void*) and never synchronise the host, except where stated;
 *   - every call returns an sr_status; problems detectable on the host are reported
 *     before anything is launched.  Problems only visible on the device (a page id outside
 *     the pool, a replay length outside [0, max_replay_len]) follow the paper's fail-closed
 *     rule (Section 5.2: a hit that cannot be served is treated as a miss): that request is
 *     skipped, its outputs are left untouched, and a bit is set in a device status word
 *     readable with sr_device_status.  No kernel traps or spins without bound.
 */
#ifndef SR_REPLAY_H_
#define SR_REPLAY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sr_ctx sr_ctx;

typedef enum sr_status {
  SR_OK = 0,
  SR_ERR_INVALID_ARG = 1,       /* null pointer, negative size, inconsistent strides   */
  SR_ERR_UNSUPPORTED_SHAPE = 2, /* geometry outside what the kernels are built for     */
  SR_ERR_WORKSPACE = 3,         /* workspace pointer null, misaligned or too small     */
  SR_ERR_CUDA = 4               /* a CUDA runtime/driver call failed                   */
} sr_status;

/* bits of the device status word (sr_device_status) */
#define SR_DEV_BAD_REPLAY_LEN 0x1u /* some replay_lens[i] < 0 or > max_replay_len      */
#define SR_DEV_BAD_PAGE_ID 0x2u    /* some used page-table entry outside [0, n_phys)   */
#define SR_DEV_BAD_SLOT 0x4u       /* some state_slots[i] < -1, or >= n_state_slots      */
#define SR_DEV_ROWS_OVERFLOW 0x8u  /* sum of replay lengths above max_total_rows        */
#define SR_DEV_WAIT_EXPIRED 0x10u  /* a bounded in-kernel wait gave up (internal fault) */
#define SR_DEV_BOUNDS_CHECK 0x20u  /* SR_DEBUG_CHECK_BOUNDS only: an index left its array  */

enum { SR_W_BF16 = 0, SR_W_E4M3_BLOCK128 = 1 };   /* sr_model_desc.weight_format   */
enum { SR_CONV_SILU = 0, SR_CONV_IDENTITY = 1 };  /* sr_model_desc.conv_activation */
/* sr_model_desc.act_quant: what the q | k | v projection multiplies the e4m3 weights with (Section 7.1 serves the
 * 27B model with FP8 weights).  NONE (default): the bf16 anchors as they are (W8A16): the result is the exact
 * product up to fp32 summation and one 16-bit rounding of each weight.  E4M3_1X128 (W8A8, weight_format
 * SR_W_E4M3_BLOCK128 only): each anchor row is quantised on the fly, 128 channels at a time, s = max(amax, 1e-10)/448,
 * code = e4m3(x / s) (fp32, IEEE division, round to nearest even, saturating), and the products run on the 8-bit
 * tensor-core path; a 128-deep partial sum enters the result as weight scale x activation scale x partial sum in
 * fp32, outside the tensor core -- which is what bounds this mode: with these plain fp32 scales it runs at under
 * half of the 8-bit tensor rate, as fast as NONE on the benchmark configuration.  The gate projection (bf16
 * weights) keeps the bf16 rows.
 * W8A8 changes the VALUE computed (e4m3 keeps 4 significant bits of each activation): it is its own variant with
 * its own reference result, not an approximation of NONE held to the same tolerance. */
enum { SR_AQ_NONE = 0, SR_AQ_E4M3_1X128 = 1 };
/* sr_model_desc.recurrence: the transition A_t of Eq. 4 (Section 2.1 names both families).
 * GATED_DELTA: A_t(S) = alpha_t (I - beta_t k_t k_t^T) S.  DECAY_ONLY: A_t(S) = alpha_t S (per-head decay, no
 * erase).  The write B_t = beta_t k_t v_t^T and everything before the recurrence are the same. */
enum { SR_REC_GATED_DELTA = 0, SR_REC_DECAY_ONLY = 1 };

/* sr_model_desc.debug_flags: switches for tests and diagnostics.  They select a second form of one step (to
 * test it against the same oracle) or add checks; results stay within the documented tolerances. */
#define SR_DEBUG_DOT_CONV_STATE 0x1u /* conv state by per-channel dot products instead of the batched GEMM       */
#define SR_DEBUG_SINGLE_CTA_MMA 0x2u /* projection on one-CTA MMA tiles where CTA pairs would be used             */
#define SR_DEBUG_FP8_EXACT 0x4u      /* e4m3 weights: fp32 promotion of bare-code partial sums, no 16-bit staging */
#define SR_DEBUG_CHECK_BOUNDS 0x8u   /* kernels range-check every table-driven index before the access, skip the
                                        access and record SR_DEV_BOUNDS_CHECK instead of reading or writing       */
#define SR_DEBUG_EXPIRE_WAIT 0x10u   /* fault-injection for the bounded waits: the state chain's first in-kernel
                                        wait is given a limit of about a millisecond and the arrival it waits for
                                        is withheld, so the wait gives up, SR_DEV_WAIT_EXPIRED is raised, the
                                        affected outputs stay untouched and the kernel returns normally          */

/* Model geometry, HOST struct, fixed at sr_create.  Sizes follow Appendix A's notation. */
typedef struct sr_model_desc {
  int32_t n_layers;        /* linear-attention layers of the model (L_lin)              */
  int32_t d_model;         /* width d of an anchor row                                  */
  int32_t n_k_heads;       /* H_k                                                       */
  int32_t n_v_heads;       /* H_v                                                       */
  int32_t d_k;             /* key head width                                            */
  int32_t d_v;             /* value head width                                          */
  int32_t conv_width;      /* w (4 in all of the paper's models)                        */
  int32_t page_rows;       /* anchor rows per pool page (64: one block per KV page, Section 5.1) */
  int32_t weight_format;   /* SR_W_*                                                    */
  int32_t conv_activation; /* SR_CONV_*                                                 */
  float l2_eps;            /* epsilon inside the key normalisation (1e-6)               */
  int32_t recurrence;      /* SR_REC_* (0 = gated delta rule)                           */
  uint32_t debug_flags;    /* SR_DEBUG_* test and diagnostic switches; 0 in production  */
  int32_t act_quant;       /* SR_AQ_* (0 = none)                                        */
} sr_model_desc;

/* One layer's parameters: HOST struct holding DEVICE pointers.  The array handed to
 * sr_replay_states has n_layers entries; entries of masked-out layers are not read. */
typedef struct sr_layer_weights {
  const void* w_qkv;        /* [C][d_model], d_model contiguous; bf16, or e4m3 codes (1 byte each) */
  const float* w_qkv_scale; /* e4m3 only: [ceil(C/128)][d_model/128] fp32,
                               weight = decode(code) * scale[row/128][col/128]; else NULL */
  const void* w_ab;         /* [2*H_v][d_model] bf16: rows a_0..a_{H_v-1}, b_0..b_{H_v-1} */
  const void* conv_w;       /* [C][conv_width] bf16                                     */
  const float* decay_scale; /* [H_v] fp32                                               */
  const float* dt_bias;     /* [H_v] fp32                                               */
} sr_layer_weights;

/* The paged anchor sidecar (Section 5.1): HOST struct.  Anchor row r of physical page p
 * for pool layer q starts at base + p*page_stride + q*layer_stride + r*row_stride bytes
 * and holds d_model contiguous bf16 values.  Strides are multiples of 16 bytes.
 * The pool is only read; requests may share pages. */
typedef struct sr_anchor_pool {
  const void* base;              /* DEVICE */
  int64_t page_stride_bytes;
  int64_t layer_stride_bytes;
  int64_t row_stride_bytes;
  int32_t n_phys_pages;
  int32_t n_pool_layers;
  const int32_t* layer_to_pool;  /* HOST [n_layers]: pool layer of each model layer, -1 = none */
} sr_anchor_pool;

/* The batch of cache hits (Section 5.2: packed variable-length execution with
 * device-side boundaries and destination slots): HOST struct. */
typedef struct sr_page_table {
  const int32_t* pages;        /* DEVICE [n_requests][max_pages]: physical pages of each request's
                                  replay window, oldest first; row t of the window is row t%page_rows
                                  of pages[t/page_rows]; entries past the window are ignored */
  const int32_t* state_slots;  /* DEVICE [n_requests] or NULL (= request index).  Destination slot
                                  in the outputs; -1 is the sentinel of a padding segment: nothing is
                                  read or written for it and no status bit is set */
  int32_t n_requests;          /* at most 65535 (one grid row per request), else SR_ERR_UNSUPPORTED_SHAPE */
  int32_t max_pages;           /* second extent of `pages` */
  int32_t max_replay_len;      /* upper bound on every replay_lens[i] (<= max_pages*page_rows) */
  int64_t max_total_rows;      /* upper bound on the sum of replay_lens (sizes grid and workspace); at most
                                  65535 page slots per call (one grid row per slot), i.e.
                                  max_total_rows / 64 + n_requests <= 65535 (about 4.19 M rows), else
                                  SR_ERR_UNSUPPORTED_SHAPE */
  int32_t n_state_slots;       /* slots the output arrays hold, or 0 = not stated.  When stated, a destination
                                  slot >= n_state_slots is treated like any other invalid request (skipped,
                                  SR_DEV_BAD_SLOT) instead of being written through */
} sr_page_table;

/* An output array: slot s, layer l starts at base + s*slot_stride + l*layer_stride. */
typedef struct sr_out {
  void* base;                  /* DEVICE */
  int64_t slot_stride_bytes;
  int64_t layer_stride_bytes;
} sr_out;

/* Library version string, static storage. */
const char* sr_version(void);

/* Human-readable name of a status code, static storage. */
const char* sr_status_string(int status);

/* Checks the geometry and builds a context (host memory only; no CUDA call).
 * Any consistent geometry (n_v_heads a multiple of n_k_heads) gets a context, so the size
 * queries below work for every model of Appendix A.  The kernels (one tensor-core path for every case) cover
 * d_k in {64, 96, 128}, d_v a multiple of 8 with 2 d_k + d_v <= 512, any n_v_heads = g * n_k_heads with at most 128
 * value heads, d_model a multiple of 64 (of 128 with block-scaled weights; with quantised activations H_k d_k and
 * H_k d_k + H_v d_v must be multiples of 128 too), conv_width == 4, page_rows == 64; for anything else
 * sr_workspace_bytes, sr_replay_states and sr_debug_gather return SR_ERR_UNSUPPORTED_SHAPE (there is no fallback). */
int sr_create(const sr_model_desc* desc, sr_ctx** out_ctx);

/* Frees a context.  NULL is allowed. */
void sr_destroy(sr_ctx* ctx);

/* Bytes of one layer's recurrent state, H_v*d_k*d_v*4 (Appendix A, B_rec). */
int sr_ssm_bytes_per_layer(const sr_ctx* ctx, size_t* out_bytes);

/* Bytes of one layer's conv state, C*(w-1)*2 (Appendix A, B_conv). */
int sr_conv_bytes_per_layer(const sr_ctx* ctx, size_t* out_bytes);

/* Scratch bytes sr_replay_states should be given for any batch within the bounds in `table`
 * (n_requests, max_pages, max_total_rows; the pointers in `table` are not read).  The layers of one call are
 * independent of one another (every layer has its own anchors, Eq. 2), so for a batch too small to fill the GPU
 * with one layer the call keeps up to 32 layers in flight (on up to eight streams of the context), each with its own
 * block of scratch: this size includes those blocks (as many of 32, 24, 16, 8, 4, 2, 1 as stay within 1 GiB together
 * and the model has layers; one block for large batches, where keeping a second layer in flight under the first
 * one's projection measured within +-2 % of running them in turn).  With bf16 weights such a call also runs the
 * projections of all those layers as one launch. */
int sr_workspace_bytes(const sr_ctx* ctx, const sr_page_table* table, size_t* out_bytes);

/* The least scratch a call accepts for the same bounds: one block, layers one after the other.  A workspace
 * between the two sizes is used for as many blocks as fit. */
int sr_workspace_bytes_min(const sr_ctx* ctx, const sr_page_table* table, size_t* out_bytes);

/*
 * Rebuilds the recurrent and conv state of every layer l with layer_mask[l] != 0 for every
 * request of the batch (Eq. 2 and Eq. 4; Section 5.2 for the batch form).
 *
 *   replay_lens  DEVICE [n_requests] int32: rows to replay per request (any value >= 0;
 *                0 gives a zero state and a zero conv state)
 *   layer_mask   HOST   [n_layers] uint8
 *   weights      HOST   [n_layers]
 *   out_ssm      FP32, per (slot, layer): [H_v][d_k][d_v]
 *   out_conv     BF16, per (slot, layer): [C][w-1]
 *   workspace    DEVICE, 256-byte aligned, >= sr_workspace_bytes_min (sr_workspace_bytes for full speed on
 *                small batches); contents are scratch.  Its first word is the device status word, cleared
 *                by this call.
 *
 * The call is one unit of work on `stream`: where it runs layers side by side it does so on streams of the
 * context that fork from `stream` after the batch is packed and join it before the call's work ends (the first
 * such call creates those streams: make it outside any stream capture).
 *
 * Outputs of masked-out layers, of sentinel requests and of skipped (invalid) requests are
 * not touched.  Results are bit-reproducible from run to run.
 */
int sr_replay_states(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                     const int32_t* replay_lens, const uint8_t* layer_mask,
                     const sr_layer_weights* weights, const sr_out* out_ssm, const sr_out* out_conv,
                     void* workspace, size_t workspace_bytes, void* stream);

/*
 * sr_replay_states for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry exists for the library's users, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc -- or a framework allocator that may call it -- is
 * off limits at the moment a batch of hits arrives: inside an engine whose device memory was carved
 * up and frozen at start-up, in a plugin whose host forbids allocation on the serving path, or in a
 * step that is set up once and re-issued many times and so must see the same addresses every time.
 * Such a caller cannot produce the `workspace` that sr_replay_states asks for.  Here the workspace is
 * a fixed array inside the library's device image, SR_NOALLOC_SCRATCH_BYTES long.  Every GPU that
 * loads the library holds that much memory from load until the process exits.
 *
 * Arguments, results and error behaviour are those of sr_replay_states, minus `workspace`, with
 * these differences:
 *   - if the bounds in `table` need more than SR_NOALLOC_SCRATCH_BYTES of scratch (compare
 *     sr_workspace_bytes) the call returns SR_ERR_WORKSPACE and launches nothing.  128 MiB covers,
 *     for example, 4096 packed rows in 8 requests at d_k = d_v = 128 with 16 key / 32 value heads;
 *   - the first call on each device looks up the array's device address (with that device
 *     current).  With CUDA's lazy module loading that look-up is also the moment the array is
 *     materialised on the device: make one call at start-up, outside any stream capture and before the
 *     process freezes or fills its device memory; later calls leave the device's free memory unchanged;
 *   - the call allocates nothing: no cudaMalloc, no cudaFree, no allocating library routine;
 *   - all calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing in it needs to start at zero (each call rewrites what it reads), but two calls whose
 *     GPU work overlaps -- different streams, or different host threads -- race on it: issue them
 *     on one stream, or order them with events;
 *   - the device status word sits inside the array and is not exposed; invalid requests are
 *     still skipped with their outputs untouched.
 */
#define SR_NOALLOC_SCRATCH_BYTES (128u * 1024u * 1024u)
int sr_replay_states_noalloc(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                             const int32_t* replay_lens, const uint8_t* layer_mask,
                             const sr_layer_weights* weights, const sr_out* out_ssm, const sr_out* out_conv,
                             void* stream);

/*
 * Replay that continues earlier states instead of starting from zero.  Eq. 5 splits a state
 * into the transported earlier state plus the window's own term; sr_replay_states computes
 * only the second (S_0 = 0, Eq. 4), this call both: for every request the recurrence starts
 * from in_ssm[slot][layer] and the convolution sees in_conv[slot][layer] (Appendix A: the
 * last w-1 inputs of each channel) as the rows before row 0.  The paper's replay always
 * starts from zero; this variant makes replay composable -- a long window in pieces, or a
 * live state advanced by newly retained anchors (Section 5.3, live-state path).
 *
 * `in_ssm`, `in_conv`: HOST structs describing DEVICE arrays with the layout and slot
 * addressing of the outputs (slot = state_slots[i] or i); either may be NULL (= zero).
 * Each may be the corresponding output array itself (states updated in place).  Requests
 * with replay length 0 hand their states through.  Served for every geometry sr_replay_states serves.
 * Everything else as sr_replay_states.
 */
int sr_replay_states_from(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                          const int32_t* replay_lens, const uint8_t* layer_mask,
                          const sr_layer_weights* weights, const sr_out* in_ssm, const sr_out* in_conv,
                          const sr_out* out_ssm, const sr_out* out_conv, void* workspace,
                          size_t workspace_bytes, void* stream);

/*
 * The same call for a caller whose anchors live in a host pool (Section 5.2: anchors are
 * fetched with asynchronous host-to-device copies before replay): copies the HOST
 * anchor pool, page table, slots and replay lengths into the caller's DEVICE staging
 * buffers, runs sr_replay_states on them, and copies both outputs back to HOST memory;
 * returns without synchronising.  The anchors go up one pool layer at a time (only the
 * pool layers that a rebuilt layer reads) and the outputs come back one rebuilt layer at
 * a time (entries of other layers in the host arrays are left as they are), on two copy
 * streams of the context, so both directions overlap the kernels; all of it starts after
 * the work already queued on `stream`, and `stream` resumes only when all of it is done,
 * so synchronising `stream` is enough before reading the host outputs.  Calls on one
 * context must not overlap.  The `pool` and `table` structs
 * describe the DEVICE staging buffers (`pool->base`, `table->pages`, `table->state_slots`);
 * host sources are byte-for-byte images of them (`pool_bytes`, and the table extents).
 * Host buffers should be pinned for the copies to be asynchronous.
 * `out_ssm_bytes` / `out_conv_bytes` are the sizes of the device output arrays copied back.
 */
int sr_replay_states_host(sr_ctx* ctx, const void* host_pool, size_t pool_bytes,
                          const int32_t* host_pages, const int32_t* host_state_slots,
                          const int32_t* host_replay_lens, int32_t* dev_replay_lens,
                          const sr_anchor_pool* pool, const sr_page_table* table,
                          const uint8_t* layer_mask, const sr_layer_weights* weights,
                          const sr_out* out_ssm, size_t out_ssm_bytes, void* host_out_ssm,
                          const sr_out* out_conv, size_t out_conv_bytes, void* host_out_conv,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Group-propagated replay (Section 4.1, "Layer-wise Sparse Anchors": the hidden state is stored only at the entry
 * of each group of consecutive linear-attention layers; replay rebuilds the states of all the group's layers from
 * that one anchor, running the linear-attention layers of the group in sequence and never a full-attention layer).
 *
 * To feed layer j + 1 of a group the call has to produce layer j's OUTPUT for every replayed row, which single-layer
 * replay never computes.  The paper does not spell the block out; this library takes a pre-norm residual block
 * around the gated-delta mixer (the shape hybrid models of this family use), with r the residual-stream row:
 *
 *   x = RMSNorm(r; norm_w)                    the layer input: q, k, v, alpha, beta and both states as in sr_replay_states
 *   q^ = q / sqrt(|q|^2 + l2_eps) / sqrt(d_k);   o[h] = S_t[h]^T q^[key head of h]     (state after the update at t)
 *   y  = RMSNorm(o[h]; o_norm_w) * SiLU(x W_z^T)                                       (per value head)
 *   r' = bf16(r + y W_o^T)
 *   r''= bf16(r' + (SiLU(n W_gate^T) * (n W_up^T)) W_down^T),  n = RMSNorm(r'; mlp_norm_w)    if an MLP is given
 *
 * and the next layer of the group takes r'' (or r') as its residual-stream row.  RMSNorm(v; w) = v / sqrt(mean(v^2) +
 * norm_eps) * w.  The anchors of the group are the residual-stream rows entering its FIRST layer: pool layer
 * layer_to_pool[first_layer].
 *
 * One layer of a group: HOST struct holding DEVICE pointers, all bf16, K (input width) contiguous.
 */
typedef struct sr_block_weights {
  const void* norm_w;      /* [d_model]                                              */
  const void* w_z;         /* [H_v*d_v][d_model] output gate                         */
  const void* o_norm_w;    /* [d_v]                                                  */
  const void* w_o;         /* [d_model][H_v*d_v] output projection                   */
  const void* mlp_norm_w;  /* [d_model], or NULL: the block has no MLP               */
  const void* w_gate;      /* [d_ff][d_model]                                        */
  const void* w_up;        /* [d_ff][d_model]                                        */
  const void* w_down;      /* [d_model][d_ff]                                        */
  int32_t d_ff;            /* a multiple of 64; 0 without an MLP                     */
} sr_block_weights;

/* Scratch bytes sr_replay_group_states needs for the bounds in `table` and MLPs up to `max_d_ff` wide. */
int sr_group_workspace_bytes(const sr_ctx* ctx, const sr_page_table* table, int32_t max_d_ff, size_t* out_bytes);

/*
 * Rebuilds the recurrent and conv state of layers first_layer .. first_layer + n_group_layers - 1 for every request
 * from the group-entry anchors alone.  `weights` and `blocks`: HOST arrays with n_layers entries (the group's are
 * read; the last layer's block needs only norm_w: its output is never formed).  Outputs, addressing, the batch
 * table, device-side validation and status bits as in sr_replay_states; every layer of the group is written.
 * bf16 weights (SR_W_BF16) and (d_k, d_v) in {(64, 64), (128, 128)}, d_model and H_v*d_v multiples of 64;
 * else SR_ERR_UNSUPPORTED_SHAPE.  `debug_rows`: NULL, or DEVICE bf16 [n_group_layers - 1][max_slots * 64][d_model]
 * receiving the rows handed from each layer to the next in packed page-slot order (request i's rows start at page
 * slot sum_{i' < i} ceil(R_i' / 64)); a test aid.  Asynchronous on `stream`, no allocation, no host sync.  One
 * kernel per layer (the output gate) runs on a stream of the context that forks from `stream` and joins it again, so
 * the call stays one unit of work on `stream`; the first call creates that stream: make it outside any stream capture.
 */
int sr_replay_group_states(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                           const int32_t* replay_lens, int32_t first_layer, int32_t n_group_layers,
                           const sr_layer_weights* weights, const sr_block_weights* blocks, float norm_eps,
                           const sr_out* out_ssm, const sr_out* out_conv, void* debug_rows, void* workspace,
                           size_t workspace_bytes, void* stream);

/*
 * Several groups in one call: group g covers layers first_layers[g] .. first_layers[g] + group_sizes[g] - 1 (HOST arrays
 * of n_groups entries; the groups must not overlap), each replayed from its own group-entry anchors exactly as
 * sr_replay_group_states does it -- same kernels, same bits.  The groups are independent (Section 4.1: each group
 * restarts from its own anchor), so the call keeps several of them in flight, each on a stream of the context with
 * its own block of scratch: as many as sr_groups_workspace_bytes made room for (up to eight, within 1 GiB together), or
 * as fit the workspace given (at least sr_group_workspace_bytes: then one group after the other).  The streams fork
 * from `stream` after the batch is packed and join it before the call's work ends (the first call creates them: make
 * it outside any stream capture).  This is the form a cache hit on a hybrid model takes: all its linear-attention
 * groups at once.
 */
int sr_groups_workspace_bytes(const sr_ctx* ctx, const sr_page_table* table, int32_t max_d_ff, int32_t n_groups,
                              size_t* out_bytes);
int sr_replay_groups_states(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                            const int32_t* replay_lens, int32_t n_groups, const int32_t* first_layers,
                            const int32_t* group_sizes, const sr_layer_weights* weights, const sr_block_weights* blocks,
                            float norm_eps, const sr_out* out_ssm, const sr_out* out_conv, void* workspace,
                            size_t workspace_bytes, void* stream);

/*
 * The write side of the sidecar (Section 5.1, "Writing anchors": the host precomputes a
 * destination table for the step; indexed copies inside the step's graph write the selected
 * hidden states directly to their sidecar locations; unsampled positions receive a scratch
 * address and are ignored).  For every token t with dest_page[t] >= 0 and every i < n_layers:
 *
 *   pool[dest_page[t]][pool_layers[i]][dest_row[t]][0:d_model] = hidden[i][t][0:d_model]
 *
 * `pool`: HOST struct, `base` DEVICE and written by this call (layout as for replay).
 * `pool_layers`: HOST [n_layers], the pool layer each written layer goes to.
 * `hidden`: DEVICE bf16, layer i token t at hidden + i*layer_stride + t*row_stride (16-byte
 * aligned strides).  `dest_page`, `dest_row`: DEVICE int32 [n_tokens], shared by the layers;
 * a negative page is the scratch address (the token is not sampled: nothing is read or
 * written for it).  Two sampled tokens of one call must not share a destination.
 * `status`: DEVICE uint32 or NULL; a destination outside the pool (page >= n_phys_pages, row
 * outside 0..63) is skipped and SR_DEV_BAD_PAGE_ID is OR-ed into *status.
 * Asynchronous on `stream`, no allocation, no synchronisation; graph-capturable.
 */
int sr_anchor_write(sr_ctx* ctx, const sr_anchor_pool* pool, const int32_t* pool_layers, int32_t n_layers,
                    const void* hidden, int64_t hidden_layer_stride_bytes, int64_t hidden_row_stride_bytes,
                    const int32_t* dest_page, const int32_t* dest_row, int32_t n_tokens, uint32_t* status,
                    void* stream);

/*
 * Materialises the gathered anchor rows of one layer (Section 5.1: the anchors of a page
 * live in that page's block): out_rows is DEVICE bf16 [sum of replay_lens][d_model],
 * requests packed in order, skipped requests contributing no rows.  A test and
 * diagnostic entry: the replay call itself never writes the gathered rows to memory.
 * `out_capacity_rows` bounds the rows written.
 */
int sr_debug_gather(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table,
                    const int32_t* replay_lens, int32_t layer, void* out_rows,
                    int64_t out_capacity_rows, void* workspace, size_t workspace_bytes, void* stream);

/*
 * W8A8 only (act_quant = SR_AQ_E4M3_1X128): materialises what the activation quantiser produces for one layer, for
 * the bit-exact check of codes and scales: out_codes DEVICE uint8 [sum of replay_lens][d_model], out_scales DEVICE
 * fp32 [sum of replay_lens][d_model / 128], requests packed in order like sr_debug_gather.  A test and diagnostic
 * entry; the replay call keeps the codes in its workspace.
 */
int sr_debug_quantise(sr_ctx* ctx, const sr_anchor_pool* pool, const sr_page_table* table, const int32_t* replay_lens,
                      int32_t layer, void* out_codes, float* out_scales, int64_t out_capacity_rows, void* workspace,
                      size_t workspace_bytes, void* stream);

/* Waits for `stream` and returns the device status word the last call on this
 * workspace left (SR_DEV_* bits).  Synchronising; for tests and diagnostics. */
int sr_device_status(sr_ctx* ctx, const void* workspace, void* stream, uint32_t* out_flags);

/* Number of kernels the last sr_replay_states / sr_debug_gather call on `ctx` launched. */
int sr_last_launch_count(const sr_ctx* ctx, int64_t* out_launches);

/* Kernel kinds of the replay path, in launch order per layer (Section 5.2's replay executes
 * "the computation needed to reconstruct each group"; these are its parts). */
enum {
  SR_KERNEL_SCHEDULE = 0,   /* batch packing, once per call                          */
  SR_KERNEL_PROJECTION = 1, /* anchor gather + in-projection                          */
  SR_KERNEL_CONV_TAIL = 2,  /* conv state                                             */
  SR_KERNEL_SCAN = 3,       /* conv + SiLU + norm + gates + gated-delta state scan    */
  SR_KERNEL_WEIGHT_DECODE = 4, /* e4m3 weights only: codes -> 16-bit weights before the projection */
  SR_KERNEL_CHUNK_LOCAL = 5,   /* gates, K K^T and the chunk inverse for all chunks at once (then SCAN is the chain) */
  SR_KERNEL_ANCHOR_STAGE = 6,  /* e4m3 weights only: the layer's anchors copied to fp16 (W8A16) or quantised to e4m3 (W8A8), slot order */
  SR_KERNEL_GROUP_BLOCK = 7,   /* group replay only: row norms, gate / output / MLP GEMMs and the per-token outputs */
  SR_KERNEL_KINDS = 8
};

/* Measurement aid: while enabled, sr_replay_states brackets each of its kernel launches with
 * a pair of CUDA events on the caller's stream (events are host resources created on first
 * use and freed by sr_destroy; no device memory).  Off by default. */
int sr_profile_enable(sr_ctx* ctx, int enable);

/* Waits for the last profiled sr_replay_states call and returns the summed device time (ms)
 * and the number of launches of kernels of `kind` in that call. */
int sr_profile_read(sr_ctx* ctx, int kind, float* out_ms, int64_t* out_launches);

#ifdef __cplusplus
}
#endif
#endif /* SR_REPLAY_H_ */
