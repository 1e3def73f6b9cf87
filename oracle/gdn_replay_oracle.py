"""CPU oracle for suffix-replay state reconstruction -- TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the replay hot path computes, written from
the paper's definitions and sharing no code with the CUDA path.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it; the product never does.

What it computes (per request, per rebuilt layer):

    S'_j = f(h_{j-k+1}, ..., h_j)                       (Eq. 2: replay of a suffix
                                                         from a zero state)
    S_t  = A_t(S_{t-1}) + B_t,  S_0 = 0                 (Eq. 4: the recurrence; keys,
                                                         values and gates are projections
                                                         of the layer input h_t)

with the gated-delta-rule instance of Eq. 4 (decay plus rank-one erase, Section 2.1):

    A_t(S) = alpha_t (I - beta_t k_t k_t^T) S ,   B_t = beta_t k_t v_t^T ,
    S in R^{d_k x d_v}  (one matrix per value head, Appendix A "Native cache")

evaluated one token at a time, exactly as the definition reads.  The layer's
convolution state (the last w-1 inputs of each of the C = 2 H_k d_k + H_v d_v
convolution channels, in bf16; Appendix A) is emitted next to it.  Optionally the same rows
continue an earlier state: the recurrence starts from a given S (the carried term of Eq. 5)
and the convolution takes a given conv state as the rows before row 0.

Readings of points the paper leaves open (all fixed by this build, none by the paper;
the functions below are pinned by tests, the *choices* are "parity unpinned"):
  * orientation: the key index is the ROW of S, so the read-out for key k is S^T k;
  * decay is applied first, the erase term reads the decayed state;
  * the short convolution is depthwise and causal with zero history before the first
    replayed row, tap w-1 multiplies the current row, no bias; SiLU follows it;
  * keys are L2-normalised per (token, head) as x / sqrt(sum x^2 + eps), eps = 1e-6;
  * alpha = exp(-c_h * softplus(a + delta_h)), beta = sigmoid(b) with a, b the gate
    projections; value head h uses key head h // (H_v / H_k);
  * the conv state lists, per channel, the last w-1 projection rows oldest first.

The sidecar's write side (anchor_write: destination-table indexed stores, Section 5.1) is restated too, and so is
group-propagated replay (Section 4.1: one anchor per group of consecutive linear-attention layers; block_forward,
gated_delta_outputs, group_replay) -- the latter as this build's reading of a block the paper does not spell out.

Pins (tests/test_oracle_pins.py): exact rational arithmetic on tiny projections, the
unrolled sum of Eq. 5 by explicit matrix products, closed forms for one-hot and
orthonormal keys, single-row and overwrite cases (the single-row closed form and a marker-channel
test also at H_v != H_k and d_k != d_v, which pin the q | k | v channel split), continuation from a cut (of the
recurrence, of the convolution with its history, and of a whole layer replayed in two
pieces against one pass), the contraction bound of the replay error, library convolution /
activation routines, all 256 e4m3 codes, the e4m3 activation quantiser (codes and scales bit for bit
against a library cast, every representable value as a fixed point, ties and saturation, the half-step
error bound), the state sizes printed in the paper's Appendix A table, a write / gather round trip; for group
replay: per-token outputs against the unrolled state of Eq. 5, the causal-linear-attention limit as one masked
matrix product, the block against a library composition, and the layer-to-layer feeding of a group.
"""

from __future__ import annotations

import numpy as np

PAGE_ROWS = 64


# ---------------------------------------------------------------------------------------
# storage formats

def bf16_bits_to_f64(bits) -> np.ndarray:
    """bfloat16 bit patterns (uint16) -> their exact values in fp64."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x) -> np.ndarray:
    """Round fp64 values to the nearest bfloat16 (ties to even); returns uint16 bits.
    Finite inputs inside the bf16 normal range only (all this oracle needs)."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                       # x = m * 2^e, 0.5 <= |m| < 1
    q = np.rint(m * 256.0) / 256.0           # keep 8 significant bits, round half to even
    y = np.ldexp(q, e).astype(np.float32)    # exact: y is a bf16 value
    return (y.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def e4m3_decode(codes) -> np.ndarray:
    """OCP FP8 E4M3 ("fn": bias 7, no infinities, S.1111.111 = NaN) codes -> fp64."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    expo = (c >> 3) & 0xF
    mant = (c & 0x7).astype(np.float64)
    normal = np.ldexp(1.0 + mant / 8.0, expo - 7)
    subnormal = np.ldexp(mant / 8.0, -6)
    val = sign * np.where(expo == 0, subnormal, normal)
    return np.where((expo == 0xF) & ((c & 0x7) == 0x7), np.nan, val)


def dequant_block_scaled(codes, scales, block: int = 128) -> np.ndarray:
    """w[c][j] = decode_e4m3(codes[c][j]) * scales[c // block][j // block], in fp64."""
    w = e4m3_decode(codes)
    C, d = w.shape
    rows = np.arange(C) // block
    cols = np.arange(d) // block
    return w * np.asarray(scales, dtype=np.float64)[rows[:, None], cols[None, :]]


def f32_to_e4m3_codes(y) -> np.ndarray:
    """fp32 values -> e4m3 codes, round to nearest even, magnitudes above 448 saturate to 448 (never NaN)."""
    y = np.asarray(y, dtype=np.float32).astype(np.float64)
    sign = np.where(np.signbit(y), 0x80, 0).astype(np.int64)
    a = np.minimum(np.abs(y), 448.0)
    m, e = np.frexp(a)                                   # a = m * 2^e, m in [0.5, 1)
    e = e - 1                                            # a = (2m) * 2^e, 2m in [1, 2)
    sub = a < 2.0 ** -6                                  # below the smallest normal: steps of 2^-9
    q_sub = np.rint(a / 2.0 ** -9).astype(np.int64)      # 0..8 (8 = the smallest normal, code 0x08)
    frac = np.rint((2.0 * m - 1.0) * 8.0).astype(np.int64)      # 0..8, ties to even
    e_n = np.where(frac == 8, e + 1, e)
    frac = np.where(frac == 8, 0, frac)
    q_norm = ((e_n + 7) << 3) | frac
    code = np.where(sub, q_sub, q_norm)
    return (sign | code).astype(np.uint8)


def quantise_e4m3_1x128(X, group: int = 128):
    """Activation quantiser of the W8A8 variant: each row is cut into groups of 128 consecutive channels; per
    group s = max(amax, 1e-10) / 448 and code = e4m3(x / s), both in fp32 with IEEE division and
    round-to-nearest-even.  X [R, d] (values exactly representable in fp32) -> (codes uint8 [R, d], scales
    float32 [R, d / group])."""
    X32 = np.asarray(X, dtype=np.float32)
    R, d = X32.shape
    g = X32.reshape(R, d // group, group)
    amax = np.max(np.abs(g), axis=-1)
    scale = (np.maximum(amax, np.float32(1e-10)) / np.float32(448.0)).astype(np.float32)
    codes = f32_to_e4m3_codes((g / scale[:, :, None]).astype(np.float32)).reshape(R, d)
    return codes, scale


def dequantise_1x128(codes, scales, group: int = 128) -> np.ndarray:
    """decode(code) * scale of its (row, group), exact in fp64."""
    R, d = codes.shape
    return (e4m3_decode(codes).reshape(R, d // group, group) *
            np.asarray(scales, dtype=np.float64)[:, :, None]).reshape(R, d)


# ---------------------------------------------------------------------------------------
# step 1: anchor gather through the page table (Section 5.1: one anchor block per KV page)

def gather_anchor_rows(pool, pages, n_rows: int, pool_layer: int, page_rows: int = PAGE_ROWS) -> np.ndarray:
    """Rows 0..n_rows-1 of one request's replay window for one layer.

    ``pool`` is indexable as ``pool[phys_page, pool_layer]`` -> uint16 [page_rows, d]
    (a 4-D array ``[n_phys][L_pool][page_rows][d]`` or a dict keyed that way);
    ``pages`` lists the request's physical pages, oldest first.  Row t lives on
    ``pages[t // page_rows]`` at row ``t % page_rows``.
    """
    rows = []
    for t in range(int(n_rows)):
        page = int(pages[t // page_rows])
        rows.append(np.asarray(pool[page, pool_layer])[t % page_rows])
    if not rows:
        return np.zeros((0, 0), dtype=np.float64)
    return bf16_bits_to_f64(np.stack(rows))


def anchor_write(pool, hidden_bits, dest_page, dest_row, pool_layer: int) -> None:
    """The write side of the sidecar (Section 5.1, "Writing anchors"): token t of a step stores its hidden state
    at row dest_row[t] of page dest_page[t]; a negative page is the scratch address -- the token is not sampled
    and nothing is stored.  `pool` is a uint16 array [n_phys, L_pool, page_rows, d], updated in place;
    `hidden_bits` uint16 [n_tokens, d]."""
    hidden_bits = np.asarray(hidden_bits, dtype=np.uint16)
    for t in range(hidden_bits.shape[0]):
        page = int(dest_page[t])
        if page >= 0:
            pool[page, pool_layer, int(dest_row[t])] = hidden_bits[t]


# ---------------------------------------------------------------------------------------
# step 2: in-projection (Section 2.1: keys, values and gates are projections of h_t)

def in_projection(X, w_qkv, w_ab):
    """Z = X W_qkv^T  [R, C]  and  G = X W_ab^T  [R, 2 H_v], all fp64."""
    X = np.asarray(X, dtype=np.float64)
    return X @ np.asarray(w_qkv, dtype=np.float64).T, X @ np.asarray(w_ab, dtype=np.float64).T


# ---------------------------------------------------------------------------------------
# step 3: convolution state (Appendix A: last w-1 inputs of each of the C channels, bf16)

def conv_tail_bits(Z, conv_width: int, history=None) -> np.ndarray:
    """[C, w-1] uint16: entry [c][j] = bf16(Z[R-(w-1)+j][c]).

    Rows before the window are 0, or, when replay continues an earlier state, the rows of `history`
    ([w-1, C] fp64, oldest first: the inputs that preceded row 0)."""
    Z = np.asarray(Z, dtype=np.float64)
    R, C = Z.shape
    out = np.zeros((C, conv_width - 1), dtype=np.uint16)
    for j in range(conv_width - 1):
        t = R - (conv_width - 1) + j
        if t >= 0:
            out[:, j] = f64_to_bf16_bits(Z[t])
        elif history is not None:
            out[:, j] = f64_to_bf16_bits(np.asarray(history, dtype=np.float64)[conv_width - 1 + t])
    return out


# ---------------------------------------------------------------------------------------
# step 4: short causal depthwise convolution + SiLU

def causal_conv_silu(Z, conv_w, activation: str = "silu", history=None) -> np.ndarray:
    """Y[t][c] = act( sum_j conv_w[c][j] * Z[t-(w-1)+j][c] ); Z[<0] = 0, or the rows of `history`
    ([w-1, C], oldest first; history[w-1+s] stands for Z[s], s < 0) when replay continues a state."""
    Z = np.asarray(Z, dtype=np.float64)
    cw = np.asarray(conv_w, dtype=np.float64)
    R, C = Z.shape
    w = cw.shape[1]
    hist = None if history is None else np.asarray(history, dtype=np.float64)
    pre = np.zeros((R, C), dtype=np.float64)
    for t in range(R):
        for j in range(w):
            s = t - (w - 1) + j
            if s >= 0:
                pre[t] += cw[:, j] * Z[s]
            elif hist is not None:
                pre[t] += cw[:, j] * hist[w - 1 + s]
    if activation == "identity":
        return pre
    return pre / (1.0 + np.exp(-pre))


def split_qkv(Y, n_k_heads: int, n_v_heads: int, d_k: int, d_v: int):
    """Channel order q | k | v, head-major inside each block."""
    R = Y.shape[0]
    nq = n_k_heads * d_k
    q = Y[:, :nq].reshape(R, n_k_heads, d_k)
    k = Y[:, nq:2 * nq].reshape(R, n_k_heads, d_k)
    v = Y[:, 2 * nq:].reshape(R, n_v_heads, d_v)
    return q, k, v


# ---------------------------------------------------------------------------------------
# step 5: L2 normalisation of the keys

def l2_normalise(x, eps: float = 1e-6) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.sum(x * x, axis=-1, keepdims=True) + eps)


# ---------------------------------------------------------------------------------------
# step 6: gates

def gates(G, decay_scale, dt_bias):
    """alpha[t][h] = exp(-c_h softplus(a + delta_h)),  beta[t][h] = sigmoid(b)."""
    G = np.asarray(G, dtype=np.float64)
    H = G.shape[1] // 2
    a = G[:, :H] + np.asarray(dt_bias, dtype=np.float64)[None, :]
    softplus = np.maximum(a, 0.0) + np.log1p(np.exp(-np.abs(a)))
    alpha = np.exp(-np.asarray(decay_scale, dtype=np.float64)[None, :] * softplus)
    beta = 1.0 / (1.0 + np.exp(-G[:, H:]))
    return alpha, beta


# ---------------------------------------------------------------------------------------
# step 7: the recurrence, one token at a time (Eq. 4)

def gated_delta_recurrence(k_hat, v, alpha, beta, S0=None, erase: bool = True) -> np.ndarray:
    """S_t = alpha_t (I - beta_t k_t k_t^T) S_{t-1} + beta_t k_t v_t^T per value head.

    k_hat [R, H_k, d_k], v [R, H_v, d_v], alpha/beta [R, H_v]; returns S [H_v, d_k, d_v].
    `erase=False` drops the rank-one erase: A_t(S) = alpha_t S, the per-head-decay family that
    Section 2.1 names next to the gated delta rule (same write B_t = beta_t k_t v_t^T).
    """
    k_hat = np.asarray(k_hat, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    alpha = np.asarray(alpha, dtype=np.float64)
    beta = np.asarray(beta, dtype=np.float64)
    R, H_k, d_k = k_hat.shape
    _, H_v, d_v = v.shape
    group = H_v // H_k
    S = np.zeros((H_v, d_k, d_v)) if S0 is None else np.array(S0, dtype=np.float64)
    for t in range(R):
        k_t = np.repeat(k_hat[t], group, axis=0)             # [H_v, d_k]
        S = alpha[t][:, None, None] * S                       # decay
        r = np.einsum("hkv,hk->hv", S, k_t) if erase else 0.0    # what the state returns for k_t
        S = S + beta[t][:, None, None] * k_t[:, :, None] * (v[t] - r)[:, None, :]
    return S


# ---------------------------------------------------------------------------------------
# the whole path for one (request, layer)

def replay_layer(X, w_qkv, w_ab, conv_w, decay_scale, dt_bias, *, n_k_heads, n_v_heads, d_k, d_v,
                 eps: float = 1e-6, activation: str = "silu", S0=None, conv_state_bits=None, erase: bool = True,
                 act_quant: str = "none"):
    """Anchor rows X [R, d] (fp64) -> (S fp32 [H_v, d_k, d_v], conv state uint16 [C, w-1]).

    Replay from a zero state (Eq. 4, S_0 = 0) by default.  With `S0` ([H_v, d_k, d_v]) and `conv_state_bits`
    ([C, w-1] uint16, the layout this function returns) the same rows continue an earlier state instead: the
    recurrence starts from S0 (Eq. 5 with a non-zero carried term) and the convolution sees the stored inputs
    as the rows before row 0 (Appendix A: the conv state is the last w-1 inputs of each channel).

    `act_quant="e4m3_1x128"` is the W8A8 variant of the block-scaled projection (Section 7.1 runs the 27B model
    with FP8 weights): the rows that enter the q | k | v projection are first quantised to e4m3 with one scale
    per row and 128 channels and the projection uses the dequantised values.  The gate projection, whose weights
    stay bf16, keeps the unquantised rows."""
    conv_w = np.asarray(conv_w, dtype=np.float64)
    width = conv_w.shape[1]
    C = 2 * n_k_heads * d_k + n_v_heads * d_v
    R = X.shape[0]
    history = None if conv_state_bits is None else bf16_bits_to_f64(np.asarray(conv_state_bits, dtype=np.uint16)).T
    if R == 0:
        S_out = np.zeros((n_v_heads, d_k, d_v), dtype=np.float32) if S0 is None else np.asarray(S0, dtype=np.float32)
        tail_out = (np.zeros((C, width - 1), dtype=np.uint16) if conv_state_bits is None
                    else np.array(conv_state_bits, dtype=np.uint16))
        return S_out, tail_out
    Z, G = in_projection(X, w_qkv, w_ab)
    if act_quant == "e4m3_1x128":
        Z, _ = in_projection(dequantise_1x128(*quantise_e4m3_1x128(X)), w_qkv, w_ab)
    elif act_quant != "none":
        raise ValueError(act_quant)
    tail = conv_tail_bits(Z, width, history)
    Y = causal_conv_silu(Z, conv_w, activation, history)
    _q, k, v = split_qkv(Y, n_k_heads, n_v_heads, d_k, d_v)
    k_hat = l2_normalise(k, eps)
    alpha, beta = gates(G, decay_scale, dt_bias)
    S = gated_delta_recurrence(k_hat, v, alpha, beta, S0, erase)
    return S.astype(np.float32), tail


def layer_weights_f64(arrays: dict):
    """Raw storage of one layer's parameters -> fp64 matrices (bf16 bits or e4m3 codes x scales)."""
    if "w_qkv_bits" in arrays:
        w_qkv = bf16_bits_to_f64(arrays["w_qkv_bits"])
    else:
        w_qkv = dequant_block_scaled(arrays["w_qkv_codes"], arrays["w_qkv_scale"])
    return (w_qkv, bf16_bits_to_f64(arrays["w_ab_bits"]), bf16_bits_to_f64(arrays["conv_w_bits"]),
            np.asarray(arrays["decay_scale"], dtype=np.float64), np.asarray(arrays["dt_bias"], dtype=np.float64))


def replay_request_layer(pool, pages, n_rows, pool_layer, arrays: dict, *, n_k_heads, n_v_heads, d_k, d_v,
                         eps: float = 1e-6, activation: str = "silu", S0=None, conv_state_bits=None,
                         erase: bool = True, act_quant: str = "none"):
    """Gather + replay for one (request, layer) from raw storage."""
    w_qkv, w_ab, conv_w, c, delta = layer_weights_f64(arrays)
    X = gather_anchor_rows(pool, pages, n_rows, pool_layer)
    if n_rows == 0:
        X = np.zeros((0, w_qkv.shape[1]))
    return replay_layer(X, w_qkv, w_ab, conv_w, c, delta, n_k_heads=n_k_heads, n_v_heads=n_v_heads,
                        d_k=d_k, d_v=d_v, eps=eps, activation=activation, S0=S0, conv_state_bits=conv_state_bits,
                        erase=erase, act_quant=act_quant)


# ---------------------------------------------------------------------------------------
# Group-propagated replay (Section 4.1, "Layer-wise Sparse Anchors"): one anchor per GROUP of consecutive
# linear-attention layers.  Only the hidden state entering the group's first layer is stored; replay rebuilds the
# first layer's state from it and, to feed the next layer of the group, also has to produce that layer's OUTPUT
# for every replayed row -- the per-token half of the layer that single-layer replay never computes.
#
# The paper describes the scheme, not the block, so the block below is this build's reading (a pre-norm residual
# block around a gated-delta mixer, the shape hybrid models of this family use; every choice "parity unpinned"):
#
#   x_t  = RMSNorm(r_t; norm_w)                               layer input, from the residual stream r_t
#   q, k, v, alpha, beta from x_t as in replay_layer; q is L2-normalised like k and scaled by d_k^-1/2
#   o_t[h] = S_t[h]^T q_t[kh]                                  read-out of the state AFTER the update at t
#   g_t  = x_t W_z^T                                           output gate, H_v d_v wide
#   y_t  = RMSNorm_per_head(o_t; o_norm_w) * SiLU(g_t)
#   r'_t = bf16(r_t + y_t W_o^T)                               residual add, stored in bf16
#   r''_t = bf16(r'_t + (SiLU(n W_gate^T) * (n W_up^T)) W_down^T),  n = RMSNorm(r'_t; mlp_norm_w)    (optional MLP)
#
# The group's anchors are rows of the residual stream entering its first layer.

def rms_norm(x, w, eps: float = 1e-6) -> np.ndarray:
    x = np.asarray(x, dtype=np.float64)
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * np.asarray(w, dtype=np.float64)


def gated_delta_outputs(q, k_hat, v, alpha, beta, S0=None, erase: bool = True):
    """The recurrence of gated_delta_recurrence with the per-token read-out o_t = S_t^T q_t (the state after the
    update at t).  q [R, H_k, d_k]; returns (O [R, H_v, d_v], S [H_v, d_k, d_v])."""
    q = np.asarray(q, dtype=np.float64)
    k_hat = np.asarray(k_hat, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    R, H_k, d_k = k_hat.shape
    _, H_v, d_v = v.shape
    group = H_v // H_k
    S = np.zeros((H_v, d_k, d_v)) if S0 is None else np.array(S0, dtype=np.float64)
    O = np.zeros((R, H_v, d_v))
    for t in range(R):
        k_t = np.repeat(k_hat[t], group, axis=0)
        q_t = np.repeat(q[t], group, axis=0)
        S = alpha[t][:, None, None] * S
        r = np.einsum("hkv,hk->hv", S, k_t) if erase else 0.0
        S = S + beta[t][:, None, None] * k_t[:, :, None] * (v[t] - r)[:, None, :]
        O[t] = np.einsum("hkv,hk->hv", S, q_t)
    return O, S


def block_forward(r_rows, layer: dict, *, n_k_heads, n_v_heads, d_k, d_v, eps: float = 1e-6, norm_eps: float = 1e-6,
                  erase: bool = True):
    """One block of a group on the residual-stream rows r [R, d] (fp64 values of bf16 storage).

    `layer`: fp64 arrays norm_w [d], w_qkv [C, d], w_ab [2 H_v, d], conv_w [C, w], decay_scale, dt_bias [H_v],
    w_z [H_v d_v, d], o_norm_w [d_v], w_o [d, H_v d_v] and optionally mlp_norm_w [d], w_gate, w_up [f, d],
    w_down [d, f].  Returns (next residual rows as bf16 bits [R, d], S fp32 [H_v, d_k, d_v], conv state bits)."""
    r_rows = np.asarray(r_rows, dtype=np.float64)
    R = r_rows.shape[0]
    # the layer input stands where a stored anchor stands in single-layer replay: a bf16 hidden state
    x = bf16_bits_to_f64(f64_to_bf16_bits(rms_norm(r_rows, layer["norm_w"], norm_eps)))
    Z, G = in_projection(x, layer["w_qkv"], layer["w_ab"])
    width = np.asarray(layer["conv_w"]).shape[1]
    tail = conv_tail_bits(Z, width)
    Y = causal_conv_silu(Z, layer["conv_w"])
    q, k, v = split_qkv(Y, n_k_heads, n_v_heads, d_k, d_v)
    alpha, beta = gates(G, layer["decay_scale"], layer["dt_bias"])
    O, S = gated_delta_outputs(l2_normalise(q, eps) * d_k ** -0.5, l2_normalise(k, eps), v, alpha, beta, erase=erase)
    gate = x @ np.asarray(layer["w_z"], dtype=np.float64).T
    y = (rms_norm(O, layer["o_norm_w"], norm_eps).reshape(R, n_v_heads * d_v)) * (gate / (1.0 + np.exp(-gate)))
    r1 = bf16_bits_to_f64(f64_to_bf16_bits(r_rows + y @ np.asarray(layer["w_o"], dtype=np.float64).T))
    if "w_gate" in layer:
        n = bf16_bits_to_f64(f64_to_bf16_bits(rms_norm(r1, layer["mlp_norm_w"], norm_eps)))
        a = n @ np.asarray(layer["w_gate"], dtype=np.float64).T
        hidden = (a / (1.0 + np.exp(-a))) * (n @ np.asarray(layer["w_up"], dtype=np.float64).T)
        r1 = bf16_bits_to_f64(f64_to_bf16_bits(r1 + hidden @ np.asarray(layer["w_down"], dtype=np.float64).T))
    return f64_to_bf16_bits(r1), S.astype(np.float32), tail


def group_replay(anchor_rows, layers, return_rows: bool = False, **geometry):
    """States of every layer of one group from the group-entry anchors alone (Section 4.1): layer j is replayed on
    the rows that layers 0..j-1 of the group produced.  anchor_rows [R, d] fp64 (residual stream entering the
    group); returns [(S fp32, conv state bits)] per layer.  The last layer's output is never formed.  With
    return_rows also the bf16 bits of the rows handed from each layer to the next ([R, d] per hand-over)."""
    r = np.asarray(anchor_rows, dtype=np.float64)
    out, handed = [], []
    for j, layer in enumerate(layers):
        bits, S, tail = block_forward(r, layer, **geometry)
        out.append((S, tail))
        if j + 1 < len(layers):
            handed.append(bits)
            r = bf16_bits_to_f64(bits)
    return (out, handed) if return_rows else out


# ---------------------------------------------------------------------------------------
# extents of the two outputs (Appendix A)

def state_extents(n_k_heads: int, n_v_heads: int, d_k: int, d_v: int, conv_width: int):
    """((H_v, d_k, d_v) fp32, (C, w-1) bf16) per linear layer."""
    C = 2 * n_k_heads * d_k + n_v_heads * d_v
    return (n_v_heads, d_k, d_v), (C, conv_width - 1)
