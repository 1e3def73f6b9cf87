"""Pins for the CPU oracle: each check compares it with something other than itself --
exact rational arithmetic, explicit matrix products of the unrolled form (Eq. 5),
closed forms, library routines, or numbers the paper prints."""

import math
import os
import struct
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import gdn_replay_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def _bf16_bits(x: torch.Tensor) -> np.ndarray:
    return x.to(torch.bfloat16).contiguous().view(torch.int16).numpy().view(np.uint16)


def _rng(seed):
    return np.random.RandomState(seed)


def _unit_rows(x):
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


# ----------------------------------------------------------------------------- formats

def test_bf16_decode_matches_torch_for_every_finite_pattern():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    ours = orc.bf16_bits_to_f64(bits)
    finite = np.isfinite(t)
    assert np.array_equal(ours[finite], t[finite])


def test_bf16_rounding_matches_torch_including_ties():
    r = _rng(1)
    x = np.concatenate([r.standard_normal(20000) * 10.0 ** r.uniform(-6, 6, 20000),
                        # exact ties between neighbouring bf16 values
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7), 0.0, 0.5, -3.0])])
    # torch rounds fp32 -> bf16; use values exactly representable in fp32 so both see the same number
    x = x.astype(np.float32).astype(np.float64)
    want = _bf16_bits(torch.from_numpy(x.astype(np.float32)))
    assert np.array_equal(orc.f64_to_bf16_bits(x), want)


def test_e4m3_decode_all_256_codes_against_torch_and_closed_form():
    codes = np.arange(256, dtype=np.uint8)
    ours = orc.e4m3_decode(codes)
    lib = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(ours), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(ours[ok], lib[ok])
    # spot values fixed by the format definition
    assert ours[0x7E] == 448.0 and ours[0x01] == 2.0 ** -9 and ours[0x08] == 2.0 ** -6
    assert ours[0x38] == 1.0 and ours[0xB8] == -1.0 and np.isnan(ours[0x7F]) and np.isnan(ours[0xFF])


def test_e4m3_rounding_every_code_is_a_fixed_point_and_ties_go_to_even():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    vals = orc.e4m3_decode(codes)
    back = orc.f32_to_e4m3_codes(vals.astype(np.float32))
    assert np.array_equal(back & 0x7F, codes & 0x7F)                       # every value maps to its own code
    assert np.array_equal(back[vals != 0] & 0x80, codes[vals != 0] & 0x80)
    # midpoints between neighbours go to the even code; a hair to either side goes to the nearer one
    pos = np.sort(vals[codes < 0x80])                                      # the non-negative values, +0 once
    lo, hi = pos[:-1], pos[1:]
    mid = ((lo + hi) / 2).astype(np.float32)                              # exact in fp32
    c_lo, c_hi = orc.f32_to_e4m3_codes(lo.astype(np.float32)), orc.f32_to_e4m3_codes(hi.astype(np.float32))
    want = np.where(c_lo % 2 == 0, c_lo, c_hi)
    assert np.array_equal(orc.f32_to_e4m3_codes(mid), want)
    assert np.array_equal(orc.f32_to_e4m3_codes(np.nextafter(mid, np.float32(0))), c_lo)
    assert np.array_equal(orc.f32_to_e4m3_codes(np.nextafter(mid, np.float32(1e9))), c_hi)
    # saturation instead of NaN, signs kept
    assert orc.f32_to_e4m3_codes(np.float32([449.0, 1e9, -1e9, 464.0, -0.0])).tolist() == [0x7E, 0x7E, 0xFE, 0x7E, 0x80]


def test_e4m3_rounding_matches_the_library_cast_inside_the_range():
    r = _rng(61)
    y = np.concatenate([r.standard_normal(50000) * 10.0 ** r.uniform(-4, 2.6, 50000), r.uniform(-448, 448, 20000)])
    y = y[np.abs(y) <= 448].astype(np.float32)
    lib = torch.from_numpy(y).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(orc.f32_to_e4m3_codes(y), lib)


def test_activation_quantiser_scales_codes_and_error_bound():
    r = _rng(62)
    X = torch.from_numpy(r.standard_normal((9, 384)) * 10.0 ** r.uniform(-3, 3, (9, 1))).to(torch.bfloat16)
    X[3, 128:256] = 0                                           # an all-zero group: scale floor, codes zero
    Xf = X.float().numpy()
    codes, scales = orc.quantise_e4m3_1x128(Xf)
    assert codes.shape == (9, 384) and scales.shape == (9, 3) and scales.dtype == np.float32
    # the same arithmetic through torch: fp32 amax, fp32 divisions, library cast
    g = X.float().reshape(9, 3, 128)
    s_t = torch.clamp(g.abs().amax(-1), min=1e-10) / 448.0
    c_t = (g / s_t[:, :, None]).to(torch.float8_e4m3fn).view(torch.uint8).reshape(9, 384).numpy()
    assert np.array_equal(scales, s_t.numpy()) and np.array_equal(codes, c_t)
    assert not codes[3, 128:256].any() and scales[3, 1] == np.float32(1e-10) / np.float32(448)
    # the largest magnitude of every group lands on +-448, and nothing is off by more than half a step of its binade
    deq = orc.dequantise_1x128(codes, scales)
    y = Xf.astype(np.float64).reshape(9, 3, 128) / scales.astype(np.float64)[:, :, None]
    step = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -6))) - 3), 2.0 ** -9)
    err = np.abs(deq.reshape(9, 3, 128) / scales.astype(np.float64)[:, :, None] - y)
    assert np.all(err <= step / 2 * (1 + 1e-6) + 448 * 2.0 ** -23)
    nz = [(i, j) for i in range(9) for j in range(3) if not (i == 3 and j == 1)]
    assert all(np.abs(orc.e4m3_decode(codes.reshape(9, 3, 128)[i, j])).max() == 448.0 for i, j in nz)


def test_w8a8_layer_is_the_layer_on_dequantised_rows_with_exact_gates():
    """act_quant: the q | k | v projection sees decode(code) * scale, the gate projection the original rows."""
    r = _rng(63)
    R, d, H, dk = 11, 256, 2, 4
    C = 3 * H * dk
    X = torch.from_numpy(r.standard_normal((R, d))).to(torch.bfloat16).double().numpy()
    W = r.standard_normal((C, d)) / math.sqrt(d)
    Wab = r.standard_normal((2 * H, d)) / math.sqrt(d)
    cw = r.standard_normal((C, 4)) / 2
    c, delta = np.array([0.1, 0.2]), np.zeros(2)
    kw = dict(n_k_heads=H, n_v_heads=H, d_k=dk, d_v=dk)
    S_q, tail_q = orc.replay_layer(X, W, Wab, cw, c, delta, act_quant="e4m3_1x128", **kw)
    Xd = orc.dequantise_1x128(*orc.quantise_e4m3_1x128(X))
    assert 1e-3 < np.abs(Xd - X).max() / np.abs(X).max() < 0.07          # really quantised: e4m3 keeps 4 bits
    # the same thing spelled out with the step functions: Z from the dequantised rows, G from the original ones
    Z = Xd @ W.T
    G = X @ Wab.T
    Y = orc.causal_conv_silu(Z, cw)
    _, k, v = orc.split_qkv(Y, H, H, dk, dk)
    alpha, beta = orc.gates(G, c, delta)
    S_want = orc.gated_delta_recurrence(orc.l2_normalise(k), v, alpha, beta)
    assert np.allclose(S_q, S_want.astype(np.float32), rtol=1e-6, atol=1e-9)
    assert np.array_equal(tail_q, orc.conv_tail_bits(Z, 4))
    S_plain, _ = orc.replay_layer(X, W, Wab, cw, c, delta, **kw)
    assert not np.allclose(S_q, S_plain, rtol=1e-3)                        # and it differs from the exact-activation layer


def test_block_scaled_dequant_brute_force():
    r = _rng(2)
    C, d = 200, 384
    codes = r.randint(0, 256, size=(C, d)).astype(np.uint8)
    codes[(codes & 0x7F) == 0x7F] = 0x10
    scales = np.exp(r.standard_normal((2, 3))).astype(np.float32)
    got = orc.dequant_block_scaled(codes, scales)
    for (c, j) in [(0, 0), (127, 127), (128, 127), (199, 383), (5, 256), (130, 255)]:
        want = float(torch.tensor([codes[c, j]], dtype=torch.uint8).view(torch.float8_e4m3fn).double()) \
            * float(scales[c // 128, j // 128])
        assert got[c, j] == want


# ------------------------------------------------------------------------------ gather

def test_gather_brute_force_and_dict_pool():
    r = _rng(3)
    n_phys, L_pool, P, d = 7, 2, 64, 8
    pool = r.randint(0, 0x4000, size=(n_phys, L_pool, P, d)).astype(np.uint16)
    pages = [5, 0, 3]
    R = 2 * P + 9
    X = orc.gather_anchor_rows(pool, pages, R, 1)
    assert X.shape == (R, d)
    for t in (0, 1, 63, 64, 127, 128, R - 1):
        bits = pool[pages[t // P], 1, t % P]
        want = [struct.unpack("<f", struct.pack("<I", int(b) << 16))[0] for b in bits]
        assert list(X[t]) == want
    as_dict = {(p, 1): pool[p, 1] for p in pages}
    assert np.array_equal(orc.gather_anchor_rows(as_dict, pages, R, 1), X)


# -------------------------------------------------------------------------- projection

def test_projection_exact_rational_arithmetic():
    r = _rng(4)
    R, d, C, H = 3, 16, 5, 1
    X = torch.from_numpy(r.standard_normal((R, d))).to(torch.bfloat16)
    W = torch.from_numpy(r.standard_normal((C, d)) / 4).to(torch.bfloat16)
    Wab = torch.from_numpy(r.standard_normal((2 * H, d)) / 4).to(torch.bfloat16)
    Z, G = orc.in_projection(orc.bf16_bits_to_f64(_bf16_bits(X)), orc.bf16_bits_to_f64(_bf16_bits(W)),
                             orc.bf16_bits_to_f64(_bf16_bits(Wab)))
    Xf = [[Fraction(float(v)) for v in row] for row in X.double().tolist()]
    for Wm, out in ((W, Z), (Wab, G)):
        Wf = [[Fraction(float(v)) for v in row] for row in Wm.double().tolist()]
        for t in range(R):
            for c in range(len(Wf)):
                exact = sum(Xf[t][j] * Wf[c][j] for j in range(d))
                assert abs(Fraction(float(out[t, c])) - exact) <= abs(exact) * Fraction(1, 10 ** 13) + Fraction(1, 10 ** 15)


# --------------------------------------------------------------- conv, SiLU, norm, gates

def test_conv_matches_library_conv1d_and_silu():
    r = _rng(5)
    R, C, w = 37, 6, 4
    Z = r.standard_normal((R, C))
    cw = r.standard_normal((C, w))
    got = orc.causal_conv_silu(Z, cw)
    zt = torch.from_numpy(Z.T.copy())[None]                       # [1, C, R]
    lib = torch.nn.functional.conv1d(torch.nn.functional.pad(zt, (w - 1, 0)),
                                     torch.from_numpy(cw)[:, None, :], groups=C)
    lib = torch.nn.functional.silu(lib)[0].T.numpy()
    assert np.allclose(got, lib, rtol=1e-13, atol=1e-14)
    assert np.allclose(orc.causal_conv_silu(Z, cw, "identity")[:, 0],
                       np.convolve(Z[:, 0], cw[0, ::-1])[:R], rtol=1e-13, atol=1e-14)


def test_conv_tap_order_and_zero_history():
    Z = np.arange(1, 11, dtype=np.float64)[:, None]
    cur = orc.causal_conv_silu(Z, np.array([[0.0, 0, 0, 1]]), "identity")[:, 0]
    old = orc.causal_conv_silu(Z, np.array([[1.0, 0, 0, 0]]), "identity")[:, 0]
    assert list(cur) == list(range(1, 11))                        # last tap = current row
    assert list(old) == [0, 0, 0, 1, 2, 3, 4, 5, 6, 7]            # first tap = row t-3, zeros before row 0


def test_conv_tail_is_last_rows_oldest_first_with_zero_fill():
    Z = np.array([[1.0, -2.0], [3.0, 0.5], [5.0, 1.0 + 2.0 ** -9], [7.0, 8.0]])
    tail = orc.conv_tail_bits(Z, 4)
    vals = orc.bf16_bits_to_f64(tail)
    assert vals.tolist() == [[3.0, 5.0, 7.0], [0.5, 1.0, 8.0]]    # 1 + 2^-9 rounds to 1 in bf16
    short = orc.bf16_bits_to_f64(orc.conv_tail_bits(Z[:2], 4))
    assert short.tolist() == [[0.0, 1.0, 3.0], [0.0, -2.0, 0.5]]
    assert tail.shape == (2, 3) and tail.dtype == np.uint16


def test_l2_normalise_and_gates_against_library():
    r = _rng(6)
    x = r.standard_normal((5, 3, 16))
    lib = (torch.from_numpy(x) / torch.sqrt((torch.from_numpy(x) ** 2).sum(-1, keepdim=True) + 1e-6)).numpy()
    assert np.allclose(orc.l2_normalise(x), lib, rtol=1e-14)
    assert np.all(np.linalg.norm(orc.l2_normalise(x), axis=-1) <= 1.0)
    G = r.standard_normal((11, 6)) * 4
    c = np.array([0.1, 0.03, 1.0]); delta = np.array([0.0, 0.5, -1.0])
    alpha, beta = orc.gates(G, c, delta)
    want_a = torch.exp(-torch.from_numpy(c) * torch.nn.functional.softplus(torch.from_numpy(G[:, :3] + delta))).numpy()
    want_b = torch.sigmoid(torch.from_numpy(G[:, 3:])).numpy()
    assert np.allclose(alpha, want_a, rtol=1e-13) and np.allclose(beta, want_b, rtol=1e-13)
    assert np.all((alpha > 0) & (alpha <= 1)) and np.all((beta > 0) & (beta < 1))


# ---------------------------------------------------------------------- the recurrence

def _random_tokens(r, R, H, dk, dv, unit=True):
    k = r.standard_normal((R, H, dk))
    if unit:
        k = _unit_rows(k)
    v = r.standard_normal((R, H, dv))
    alpha = np.exp(-0.1 * np.log1p(np.exp(r.standard_normal((R, H)))))
    beta = 1 / (1 + np.exp(-r.standard_normal((R, H))))
    return k, v, alpha, beta


def test_unrolled_sum_of_transition_products():
    """Eq. 5: S_n = sum_i Phi_{n,i}(B_i), Phi = A_n o ... o A_{i+1}, by explicit matrices."""
    r = _rng(7)
    R, H, dk, dv = 9, 2, 5, 3
    k, v, alpha, beta = _random_tokens(r, R, H, dk, dv, unit=False)
    S = orc.gated_delta_recurrence(k, v, alpha, beta)
    for h in range(H):
        total = np.zeros((dk, dv))
        for i in range(R):
            term = beta[i, h] * np.outer(k[i, h], v[i, h])                  # B_i
            for t in range(i + 1, R):                                        # apply A_{i+1} .. A_n
                M = alpha[t, h] * (np.eye(dk) - beta[t, h] * np.outer(k[t, h], k[t, h]))
                term = M @ term
            total += term
        assert np.allclose(S[h], total, rtol=1e-12, atol=1e-14)


def test_zero_write_strength_and_empty_replay_give_zero_state():
    r = _rng(8)
    k, v, alpha, _ = _random_tokens(r, 20, 2, 4, 4)
    S = orc.gated_delta_recurrence(k, v, np.ones_like(alpha), np.zeros_like(alpha))
    assert np.all(S == 0.0)
    S = orc.gated_delta_recurrence(k[:0], v[:0], alpha[:0], alpha[:0])
    assert S.shape == (2, 4, 4) and np.all(S == 0.0)


def test_single_token_is_rank_one_with_key_as_row_index():
    k = np.zeros((1, 1, 3)); k[0, 0] = [0.6, 0.0, 0.8]
    v = np.array([[[1.0, 2.0]]])
    S = orc.gated_delta_recurrence(k, v, np.array([[0.5]]), np.array([[0.25]]))
    assert np.allclose(S[0], 0.25 * np.outer([0.6, 0.0, 0.8], [1.0, 2.0]), rtol=1e-15)
    assert S.shape == (1, 3, 2)


def test_same_key_full_write_overwrites():
    r = _rng(9)
    dk, dv = 6, 4
    key = _unit_rows(r.standard_normal((1, dk)))[0]
    k = np.stack([key, key])[:, None, :]
    v = r.standard_normal((2, 1, dv))
    S = orc.gated_delta_recurrence(k, v, np.array([[0.9], [0.37]]), np.array([[0.7], [1.0]]))
    assert np.allclose(S[0], np.outer(key, v[1, 0]), rtol=1e-13, atol=1e-15)


def test_one_hot_keys_rows_decouple():
    r = _rng(10)
    R, dk, dv = 12, 4, 3
    slot = r.randint(0, dk, size=R)
    k = np.zeros((R, 1, dk)); k[np.arange(R), 0, slot] = 1.0
    _, v, alpha, beta = _random_tokens(r, R, 1, dk, dv)
    S = orc.gated_delta_recurrence(k, v, alpha, beta)[0]
    for i in range(dk):
        row = np.zeros(dv)
        for t in range(R):
            if slot[t] != i:
                continue
            wgt = beta[t, 0]
            for s in range(t + 1, R):
                wgt *= alpha[s, 0] * ((1 - beta[s, 0]) if slot[s] == i else 1.0)
            row += wgt * v[t, 0]
        assert np.allclose(S[i], row, rtol=1e-12, atol=1e-15)


def test_orthonormal_keys_no_decay_is_an_associative_memory():
    r = _rng(11)
    R, dk, dv = 6, 8, 5
    Q, _ = np.linalg.qr(r.standard_normal((dk, dk)))
    K = Q[:R]
    V = r.standard_normal((R, dv))
    beta = r.uniform(0.1, 1.0, size=R)
    S = orc.gated_delta_recurrence(K[:, None, :], V[:, None, :], np.ones((R, 1)), beta[:, None])[0]
    assert np.allclose(S, K.T @ np.diag(beta) @ V, rtol=1e-12, atol=1e-14)
    S1 = orc.gated_delta_recurrence(K[:, None, :], V[:, None, :], np.ones((R, 1)), np.ones((R, 1)))[0]
    assert np.allclose(S1.T @ K.T, V.T, rtol=1e-12, atol=1e-13)      # exact recall S^T k_t = v_t


def test_continuation_from_a_cut_equals_one_pass():
    r = _rng(12)
    k, v, alpha, beta = _random_tokens(r, 50, 3, 8, 8)
    full = orc.gated_delta_recurrence(k, v, alpha, beta)
    c = 17
    head = orc.gated_delta_recurrence(k[:c], v[:c], alpha[:c], beta[:c])
    both = orc.gated_delta_recurrence(k[c:], v[c:], alpha[c:], beta[c:], S0=head)
    assert np.allclose(full, both, rtol=1e-13, atol=1e-15)


def test_replay_error_is_the_transported_cut_state_and_obeys_the_contraction_bound():
    """S_full - S_replay = Phi_{n,c}(S_c) (Eq. 5); with |k| <= 1 and beta in [0,1] every
    A_t has spectral norm <= alpha_t, so the error is at most prod(alpha over the replayed
    window) * |S_c|_F."""
    r = _rng(13)
    n, c, H, dk, dv = 80, 30, 2, 8, 6
    k, v, alpha, beta = _random_tokens(r, n, H, dk, dv)
    full = orc.gated_delta_recurrence(k, v, alpha, beta)
    cut = orc.gated_delta_recurrence(k[:c], v[:c], alpha[:c], beta[:c])
    replay = orc.gated_delta_recurrence(k[c:], v[c:], alpha[c:], beta[c:])
    for h in range(H):
        moved = cut[h].copy()
        for t in range(c, n):
            moved = alpha[t, h] * (np.eye(dk) - beta[t, h] * np.outer(k[t, h], k[t, h])) @ moved
        assert np.allclose(full[h] - replay[h], moved, rtol=1e-11, atol=1e-14)
        bound = np.prod(alpha[c:, h]) * np.linalg.norm(cut[h])
        assert np.linalg.norm(full[h] - replay[h]) <= bound * (1 + 1e-12)
    whole = orc.gated_delta_recurrence(k[0:], v[0:], alpha[0:], beta[0:])
    assert np.array_equal(whole, full)                              # replay of the whole prefix = full prefill


def test_decay_only_family_is_the_discounted_sum_of_writes():
    """Without the erase, Eq. 5 has scalar transitions: S_n = sum_i (prod_{t>i} alpha_t) beta_i k_i v_i^T (+ the
    carried state times the whole product) -- written here with cumulative products, no loop over the state."""
    r = _rng(41)
    R, H, dk, dv = 29, 3, 5, 4
    k = _unit_rows(r.standard_normal((R, H, dk)))
    v = r.standard_normal((R, H, dv))
    alpha = r.uniform(0.5, 1.0, size=(R, H))
    beta = r.uniform(0.0, 1.0, size=(R, H))
    S0 = r.standard_normal((H, dk, dv))
    got = orc.gated_delta_recurrence(k, v, alpha, beta, S0, erase=False)
    tail = np.cumprod(alpha[::-1], axis=0)[::-1]                     # prod_{t >= i} alpha_t
    disc = np.concatenate([tail[1:], np.ones((1, H))], axis=0)       # prod_{t > i} alpha_t
    want = np.einsum("th,thk,thv->hkv", disc * beta, k, v) + tail[0][:, None, None] * S0
    assert np.allclose(got, want, rtol=1e-12, atol=1e-13)
    with_erase = orc.gated_delta_recurrence(k, v, alpha, beta, S0)
    assert not np.allclose(with_erase, want, rtol=1e-3)              # and the erase term is not a no-op


def test_state_is_linear_in_values_and_carried_state_and_equivariant_in_value_columns():
    """Eq. 5: with keys and gates fixed, S_n is a linear map of (S_0, v_1..v_n); the value columns never mix."""
    r = _rng(43)
    R, H, dk, dv = 17, 2, 6, 5
    k = _unit_rows(r.standard_normal((R, H, dk)))
    alpha = r.uniform(0.6, 1.0, size=(R, H))
    beta = r.uniform(0.0, 1.0, size=(R, H))
    v1, v2 = r.standard_normal((R, H, dv)), r.standard_normal((R, H, dv))
    A0, B0 = r.standard_normal((H, dk, dv)), r.standard_normal((H, dk, dv))
    f = lambda v, S0: orc.gated_delta_recurrence(k, v, alpha, beta, S0)
    assert np.allclose(f(2.5 * v1 - v2, 2.5 * A0 - B0), 2.5 * f(v1, A0) - f(v2, B0), rtol=1e-11, atol=1e-12)
    perm = r.permutation(dv)
    assert np.allclose(f(v1[:, :, perm], A0[:, :, perm]), f(v1, A0)[:, :, perm], rtol=0, atol=1e-14)
    # rotating all keys by one orthogonal matrix rotates the key index of the state
    Q, _ = np.linalg.qr(r.standard_normal((dk, dk)))
    rot = orc.gated_delta_recurrence(k @ Q.T, v1, alpha, beta, np.einsum("ij,hjv->hiv", Q, A0))
    assert np.allclose(rot, np.einsum("ij,hjv->hiv", Q, f(v1, A0)), rtol=1e-11, atol=1e-12)


def test_grouped_value_heads_share_their_key_head():
    r = _rng(14)
    R, Hk, Hv, dk, dv = 7, 2, 4, 4, 3
    k = _unit_rows(r.standard_normal((R, Hk, dk)))
    v = r.standard_normal((R, Hv, dv))
    alpha = r.uniform(0.5, 1, (R, Hv)); beta = r.uniform(0, 1, (R, Hv))
    S = orc.gated_delta_recurrence(k, v, alpha, beta)
    for h in range(Hv):
        single = orc.gated_delta_recurrence(k[:, h // 2:h // 2 + 1], v[:, h:h + 1], alpha[:, h:h + 1], beta[:, h:h + 1])
        assert np.allclose(S[h], single[0], rtol=1e-14)


# ------------------------------------------------------------------- the whole pipeline

def test_single_row_end_to_end_closed_form():
    r = _rng(15)
    d, H, dk, dv = 32, 2, 4, 4
    C = 3 * H * dk
    x = torch.from_numpy(r.standard_normal((1, d))).to(torch.bfloat16).double().numpy()
    W = r.standard_normal((C, d)) / math.sqrt(d)
    Wab = r.standard_normal((2 * H, d)) / math.sqrt(d)
    cw = r.standard_normal((C, 4))
    c = np.array([0.1, 0.2]); delta = np.array([0.3, -0.2])
    S, tail = orc.replay_layer(x, W, Wab, cw, c, delta, n_k_heads=H, n_v_heads=H, d_k=dk, d_v=dv)
    z = [sum(x[0, j] * W[ch, j] for j in range(d)) for ch in range(C)]
    y = [cw[ch, 3] * z[ch] for ch in range(C)]
    y = [val / (1 + math.exp(-val)) for val in y]
    for h in range(H):
        kk = y[H * dk + h * dk: H * dk + (h + 1) * dk]
        vv = y[2 * H * dk + h * dv: 2 * H * dk + (h + 1) * dv]
        nrm = math.sqrt(sum(t * t for t in kk) + 1e-6)
        a = sum(x[0, j] * Wab[h, j] for j in range(d)) + delta[h]
        b = sum(x[0, j] * Wab[H + h, j] for j in range(d))
        beta = 1 / (1 + math.exp(-b))
        assert 0 < math.exp(-c[h] * math.log1p(math.exp(a))) <= 1
        want = np.array([[beta * (ki / nrm) * vj for vj in vv] for ki in kk])
        assert np.allclose(S[h], want.astype(np.float32), rtol=2e-7, atol=1e-12)
    assert S.dtype == np.float32
    got_tail = orc.bf16_bits_to_f64(tail)
    assert np.all(got_tail[:, :2] == 0.0)
    assert np.allclose(got_tail[:, 2], z, rtol=2 ** -8)


GEOMETRIES_UNEQUAL = [(2, 4, 4, 4), (2, 6, 4, 4), (2, 2, 3, 6), (2, 4, 3, 5)]   # (H_k, H_v, d_k, d_v)


@pytest.mark.parametrize("Hk,Hv,dk,dv", GEOMETRIES_UNEQUAL)
def test_single_row_closed_form_with_unequal_head_counts_and_widths(Hk, Hv, dk, dv):
    """The one-row closed form with H_v != H_k and d_k != d_v (Appendix A's table: 16/32 and 16/48 heads,
    widths 96/192): channel offsets are written out here with scalars -- q block H_k d_k wide, k block H_k d_k
    wide, v block H_v d_v wide, C = 2 H_k d_k + H_v d_v -- and value head h reads key head h // (H_v / H_k)."""
    r = _rng(150 + Hv * 10 + dv)
    d = 24
    C = 2 * Hk * dk + Hv * dv
    x = torch.from_numpy(r.standard_normal((1, d))).to(torch.bfloat16).double().numpy()
    W = r.standard_normal((C, d)) / math.sqrt(d)
    Wab = r.standard_normal((2 * Hv, d)) / math.sqrt(d)
    cw = r.standard_normal((C, 4))
    c = r.uniform(0.05, 0.3, Hv); delta = r.uniform(-0.3, 0.3, Hv)
    S, tail = orc.replay_layer(x, W, Wab, cw, c, delta, n_k_heads=Hk, n_v_heads=Hv, d_k=dk, d_v=dv)
    assert S.shape == (Hv, dk, dv) and tail.shape == (C, 3)
    z = [sum(x[0, j] * W[ch, j] for j in range(d)) for ch in range(C)]
    y = [cw[ch, 3] * z[ch] for ch in range(C)]
    y = [val / (1 + math.exp(-val)) for val in y]
    k_block, v_block = Hk * dk, 2 * Hk * dk
    for h in range(Hv):
        kh = h // (Hv // Hk)
        kk = [y[k_block + kh * dk + i] for i in range(dk)]
        vv = [y[v_block + h * dv + j] for j in range(dv)]
        nrm = math.sqrt(sum(t * t for t in kk) + 1e-6)
        b = sum(x[0, j] * Wab[Hv + h, j] for j in range(d))
        beta = 1 / (1 + math.exp(-b))
        want = np.array([[beta * (ki / nrm) * vj for vj in vv] for ki in kk])
        assert np.allclose(S[h], want.astype(np.float32), rtol=2e-7, atol=1e-12), h
    assert np.allclose(orc.bf16_bits_to_f64(tail)[:, 2], z, rtol=2 ** -8)


@pytest.mark.parametrize("Hk,Hv,dk,dv", GEOMETRIES_UNEQUAL)
def test_marker_channels_land_in_the_right_state_entry(Hk, Hv, dk, dv):
    """Weights that light up exactly one key channel (key head a, index i) and one value channel (value head h,
    index j): after one row the only non-zero state entries are S[h'][i][j'] with h' sharing key head a and
    (h', j') = (h, j).  A key or value offset wrong by one head, or d_v used for d_k, moves or kills the entry."""
    d = 8
    C = 2 * Hk * dk + Hv * dv
    x = np.zeros((1, d)); x[0, 0] = 1.0
    cw = np.zeros((C, 4)); cw[:, 3] = 1.0
    Wab = np.zeros((2 * Hv, d))
    group = Hv // Hk
    for a in range(Hk):
        for i in (0, dk - 1):
            for h in range(Hv):
                for j in (0, dv - 1):
                    W = np.zeros((C, d))
                    W[Hk * dk + a * dk + i, 0] = 2.0              # key channel (a, i)
                    W[2 * Hk * dk + h * dv + j, 0] = 3.0          # value channel (h, j)
                    W[a * dk + i, 0] = 5.0                        # the q channel of the same index must not matter
                    S, tail = orc.replay_layer(x, W, Wab, cw, np.full(Hv, 0.1), np.zeros(Hv), n_k_heads=Hk,
                                               n_v_heads=Hv, d_k=dk, d_v=dv, activation="identity")
                    nz = {tuple(idx) for idx in np.argwhere(S != 0)}
                    want = {(h, i, j)} if h // group == a else set()
                    assert nz == want, (a, i, h, j, nz)
                    if want:
                        assert np.isclose(S[h, i, j], 0.5 * 3.0 * 2.0 / math.sqrt(4.0 + 1e-6), rtol=1e-6)
                    t = orc.bf16_bits_to_f64(tail)[:, 2]
                    assert set(np.flatnonzero(t)) == {a * dk + i, Hk * dk + a * dk + i, 2 * Hk * dk + h * dv + j}


def test_pipeline_against_library_composition():
    """Whole layer on a small case against torch fp64 library ops (conv1d, silu, normalise)
    feeding a directly written rank-one update loop on torch tensors."""
    r = _rng(16)
    R, d, H, dk, dv = 23, 48, 2, 8, 8
    C = 3 * H * dk
    X = torch.from_numpy(r.standard_normal((R, d))).to(torch.bfloat16).double()
    W = torch.from_numpy(r.standard_normal((C, d)) / math.sqrt(d)).to(torch.bfloat16).double()
    Wab = torch.from_numpy(r.standard_normal((2 * H, d)) / math.sqrt(d)).to(torch.bfloat16).double()
    cw = torch.from_numpy(r.standard_normal((C, 4)) / 2).to(torch.bfloat16).double()
    c = np.array([0.1, 0.1]); delta = np.zeros(2)
    S, tail = orc.replay_layer(X.numpy(), W.numpy(), Wab.numpy(), cw.numpy(), c, delta,
                               n_k_heads=H, n_v_heads=H, d_k=dk, d_v=dv)
    Z = torch.nn.functional.linear(X, W)
    G = torch.nn.functional.linear(X, Wab)
    Y = torch.nn.functional.silu(torch.nn.functional.conv1d(
        torch.nn.functional.pad(Z.T[None], (3, 0)), cw[:, None, :], groups=C))[0].T
    k = Y[:, H * dk:2 * H * dk].reshape(R, H, dk)
    v = Y[:, 2 * H * dk:].reshape(R, H, dv)
    k = k / torch.sqrt((k * k).sum(-1, keepdim=True) + 1e-6)
    alpha = torch.exp(-0.1 * torch.nn.functional.softplus(G[:, :H]))
    beta = torch.sigmoid(G[:, H:])
    St = torch.zeros(H, dk, dv, dtype=torch.float64)
    for t in range(R):
        for h in range(H):
            M = alpha[t, h] * (torch.eye(dk, dtype=torch.float64) - beta[t, h] * torch.outer(k[t, h], k[t, h]))
            St[h] = M @ St[h] + beta[t, h] * torch.outer(k[t, h], v[t, h])
    assert np.allclose(S, St.numpy().astype(np.float32), rtol=1e-6, atol=1e-9)
    assert np.array_equal(tail, _bf16_bits(Z[-3:].T.float()))


def test_conv_with_history_equals_conv_of_the_concatenated_rows():
    r = _rng(21)
    R, C, w = 19, 5, 4
    Z = r.standard_normal((R, C))
    cw = r.standard_normal((C, w))
    whole = orc.causal_conv_silu(Z, cw)
    zt = torch.from_numpy(Z.T.copy())[None]
    lib = torch.nn.functional.silu(torch.nn.functional.conv1d(torch.nn.functional.pad(zt, (w - 1, 0)),
                                                              torch.from_numpy(cw)[:, None, :], groups=C))[0].T.numpy()
    for cut in (3, 4, 11, 18):
        got = orc.causal_conv_silu(Z[cut:], cw, history=Z[cut - 3:cut])
        assert np.allclose(got, whole[cut:], rtol=0, atol=1e-15)
        assert np.allclose(got, lib[cut:], rtol=1e-13, atol=1e-14)
    # unit taps: history row w-1+s stands for row s < 0 (oldest first)
    hist = np.array([[10.0], [20.0], [30.0]])
    Zs = np.array([[1.0], [2.0]])
    assert orc.causal_conv_silu(Zs, np.array([[1.0, 0, 0, 0]]), "identity", hist)[:, 0].tolist() == [10.0, 20.0]
    assert orc.causal_conv_silu(Zs, np.array([[0.0, 0, 1, 0]]), "identity", hist)[:, 0].tolist() == [30.0, 1.0]
    # conv state of a window shorter than w-1: the tail of (history | window)
    assert orc.bf16_bits_to_f64(orc.conv_tail_bits(Zs, 4, hist)).tolist() == [[30.0, 1.0, 2.0]]
    assert orc.bf16_bits_to_f64(orc.conv_tail_bits(Zs[:1], 4, hist)).tolist() == [[20.0, 30.0, 1.0]]


def test_layer_continuation_equals_one_pass_when_the_carried_state_is_exact():
    """Replaying rows [0, n) at once against replaying [0, c) and continuing with [c, n) from the state and
    conv state of the first piece.  Inputs are small integers, so the bf16 conv state carries the projected
    rows exactly; the recurrent state is carried in fp32."""
    r = _rng(22)
    n, d, H, dk, dv = 21, 16, 2, 4, 4
    C = 3 * H * dk
    X = r.randint(-1, 2, size=(n, d)).astype(np.float64)
    W = r.randint(-1, 2, size=(C, d)).astype(np.float64)
    Wab = r.randint(-1, 2, size=(2 * H, d)).astype(np.float64) / 4
    cw = r.randint(-2, 3, size=(C, 4)).astype(np.float64) / 4
    kw = dict(n_k_heads=H, n_v_heads=H, d_k=dk, d_v=dv)
    c, delta = np.array([0.1, 0.3]), np.array([0.0, 0.5])
    S_all, tail_all = orc.replay_layer(X, W, Wab, cw, c, delta, **kw)
    for cut in (1, 2, 3, 8, 19, 20):
        S1, tail1 = orc.replay_layer(X[:cut], W, Wab, cw, c, delta, **kw)
        S2, tail2 = orc.replay_layer(X[cut:], W, Wab, cw, c, delta, S0=S1, conv_state_bits=tail1, **kw)
        assert np.array_equal(tail2, tail_all), cut
        assert np.allclose(S2, S_all, rtol=2e-6, atol=1e-7), cut
    # an empty continuation hands the carried state through
    S3, tail3 = orc.replay_layer(X[:0], W, Wab, cw, c, delta, S0=S_all, conv_state_bits=tail_all, **kw)
    assert np.array_equal(S3, S_all) and np.array_equal(tail3, tail_all)


def test_anchor_write_then_gather_returns_the_sampled_rows():
    """A decode-like step stream: every 4th token is sampled and lands on consecutive rows of the pages of a
    table; gathering through that table must return exactly the sampled hidden states, other layers and pages
    untouched (the gather is pinned on its own above)."""
    r = _rng(31)
    n_phys, L_pool, d, T = 7, 3, 8, 600
    pool = r.randint(0, 2 ** 16, size=(n_phys, L_pool, 64, d)).astype(np.uint16)
    before = pool.copy()
    hidden = r.randint(0, 0x7F80, size=(T, d)).astype(np.uint16)          # finite bf16 patterns
    pages = [5, 0, 3]
    dest_page = np.full(T, -1, dtype=np.int32)
    dest_row = np.zeros(T, dtype=np.int32)
    sampled = np.arange(0, T, 4)
    for n, t in enumerate(sampled):
        dest_page[t], dest_row[t] = pages[n // 64], n % 64
    orc.anchor_write(pool, hidden, dest_page, dest_row, 1)
    got = orc.gather_anchor_rows(pool, pages, len(sampled), 1)
    assert np.array_equal(got, orc.bf16_bits_to_f64(hidden[sampled]))
    untouched = np.ones(pool.shape[:3], dtype=bool)
    for n in range(len(sampled)):
        untouched[pages[n // 64], 1, n % 64] = False
    assert np.array_equal(pool[untouched], before[untouched])


def test_replay_request_layer_reads_pages_through_the_table():
    r = _rng(17)
    n_phys, P, d, H, dk = 5, 64, 32, 1, 4
    C = 3 * H * dk
    pool = _bf16_bits(torch.from_numpy(r.standard_normal((n_phys, 1, P, d))))
    arrays = {
        "w_qkv_bits": _bf16_bits(torch.from_numpy(r.standard_normal((C, d)) / math.sqrt(d))),
        "w_ab_bits": _bf16_bits(torch.from_numpy(r.standard_normal((2 * H, d)) / math.sqrt(d))),
        "conv_w_bits": _bf16_bits(torch.from_numpy(r.standard_normal((C, 4)) / 2)),
        "decay_scale": np.array([0.1], dtype=np.float32), "dt_bias": np.zeros(1, dtype=np.float32),
    }
    kw = dict(n_k_heads=H, n_v_heads=H, d_k=dk, d_v=dk)
    S, tail = orc.replay_request_layer(pool, [3, 1], 70, 0, arrays, **kw)
    X = np.concatenate([orc.bf16_bits_to_f64(pool[3, 0]), orc.bf16_bits_to_f64(pool[1, 0][:6])])
    S2, tail2 = orc.replay_layer(X, *orc.layer_weights_f64(arrays), **kw)
    assert np.array_equal(S, S2) and np.array_equal(tail, tail2)
    S0, tail0 = orc.replay_request_layer(pool, [], 0, 0, arrays, **kw)
    assert np.all(S0 == 0) and np.all(tail0 == 0) and tail0.shape == (C, 3)


# ----------------------------------------------------------------- group-propagated replay (Section 4.1)

def _group_layer(r, d, Hk, Hv, dk, dv, mlp=0):
    C = 2 * Hk * dk + Hv * dv
    L = dict(norm_w=r.uniform(0.5, 1.5, d), w_qkv=r.standard_normal((C, d)) / math.sqrt(d),
             w_ab=r.standard_normal((2 * Hv, d)) / math.sqrt(d), conv_w=r.standard_normal((C, 4)) / 2,
             decay_scale=np.full(Hv, 0.1), dt_bias=np.zeros(Hv), w_z=r.standard_normal((Hv * dv, d)) / math.sqrt(d),
             o_norm_w=r.uniform(0.5, 1.5, dv), w_o=r.standard_normal((d, Hv * dv)) / math.sqrt(Hv * dv))
    if mlp:
        L.update(mlp_norm_w=r.uniform(0.5, 1.5, d), w_gate=r.standard_normal((mlp, d)) / math.sqrt(d),
                 w_up=r.standard_normal((mlp, d)) / math.sqrt(d), w_down=r.standard_normal((d, mlp)) / math.sqrt(mlp))
    return L


def test_rms_norm_matches_the_library():
    r = _rng(70)
    x, w = r.standard_normal((5, 3, 16)), r.uniform(0.5, 2, 16)
    lib = torch.nn.functional.rms_norm(torch.from_numpy(x), (16,), torch.from_numpy(w), eps=1e-6).numpy()
    assert np.allclose(orc.rms_norm(x, w), lib, rtol=1e-13, atol=1e-15)


def test_per_token_outputs_are_the_read_out_of_the_unrolled_state():
    """o_t = S_t^T q_t with S_t from Eq. 5 by explicit transition products; and the final state is the recurrence's."""
    r = _rng(71)
    R, Hk, Hv, dk, dv = 9, 2, 4, 5, 3
    q = r.standard_normal((R, Hk, dk))
    k = _unit_rows(r.standard_normal((R, Hk, dk)))
    v = r.standard_normal((R, Hv, dv))
    alpha, beta = r.uniform(0.5, 1, (R, Hv)), r.uniform(0, 1, (R, Hv))
    O, S = orc.gated_delta_outputs(q, k, v, alpha, beta)
    assert np.allclose(S, orc.gated_delta_recurrence(k, v, alpha, beta), rtol=0, atol=1e-15)
    for h in range(Hv):
        kh = h // 2
        for t in range(R):
            St = np.zeros((dk, dv))
            for i in range(t + 1):
                B = beta[i, h] * np.outer(k[i, kh], v[i, h])
                for j in range(i + 1, t + 1):
                    B = alpha[j, h] * (np.eye(dk) - beta[j, h] * np.outer(k[j, kh], k[j, kh])) @ B
                St += B
            assert np.allclose(O[t, h], St.T @ q[t, kh], rtol=1e-11, atol=1e-13)


def test_outputs_without_erase_and_decay_are_causal_linear_attention():
    """erase off, alpha = 1: o_t = sum_{s <= t} beta_s (k_s . q_t) v_s, one masked matrix product."""
    r = _rng(72)
    R, dk, dv = 12, 6, 4
    q, k, v = r.standard_normal((R, 1, dk)), r.standard_normal((R, 1, dk)), r.standard_normal((R, 1, dv))
    beta = r.uniform(0, 1, (R, 1))
    O, _ = orc.gated_delta_outputs(q, k, v, np.ones((R, 1)), beta, erase=False)
    want = np.tril(q[:, 0] @ k[:, 0].T) @ (beta * v[:, 0])
    assert np.allclose(O[:, 0], want, rtol=1e-12, atol=1e-13)


def test_block_against_a_library_composition_and_single_row_closed_form():
    r = _rng(73)
    R, d, Hk, Hv, dk, dv = 13, 32, 2, 4, 4, 6
    geo = dict(n_k_heads=Hk, n_v_heads=Hv, d_k=dk, d_v=dv)
    L = _group_layer(r, d, Hk, Hv, dk, dv, mlp=24)
    rows = torch.from_numpy(r.standard_normal((R, d))).to(torch.bfloat16).double()
    bits, S, tail = orc.block_forward(rows.numpy(), L, **geo)
    T = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    F = torch.nn.functional
    x = F.rms_norm(rows, (d,), T(L["norm_w"]), eps=1e-6).to(torch.bfloat16).double()   # layer inputs are bf16, like anchors
    Z = F.linear(x, T(L["w_qkv"]))
    C = Z.shape[1]
    Y = F.silu(F.conv1d(F.pad(Z.T[None], (3, 0)), T(L["conv_w"])[:, None, :], groups=C))[0].T
    nq = Hk * dk
    q, k, v = Y[:, :nq].reshape(R, Hk, dk), Y[:, nq:2 * nq].reshape(R, Hk, dk), Y[:, 2 * nq:].reshape(R, Hv, dv)
    q = q / torch.sqrt((q * q).sum(-1, keepdim=True) + 1e-6) * dk ** -0.5
    k = k / torch.sqrt((k * k).sum(-1, keepdim=True) + 1e-6)
    G = F.linear(x, T(L["w_ab"]))
    alpha, beta = torch.exp(-0.1 * F.softplus(G[:, :Hv])), torch.sigmoid(G[:, Hv:])
    St = torch.zeros(Hv, dk, dv, dtype=torch.float64)
    O = torch.zeros(R, Hv, dv, dtype=torch.float64)
    for t in range(R):
        for h in range(Hv):
            kk = k[t, h // 2]
            St[h] = alpha[t, h] * (torch.eye(dk, dtype=torch.float64) - beta[t, h] * torch.outer(kk, kk)) @ St[h] \
                + beta[t, h] * torch.outer(kk, v[t, h])
            O[t, h] = St[h].T @ q[t, h // 2]
    y = (F.rms_norm(O, (dv,), T(L["o_norm_w"]), eps=1e-6).reshape(R, Hv * dv)) * F.silu(F.linear(x, T(L["w_z"])))
    r1 = (rows + F.linear(y, T(L["w_o"]))).to(torch.bfloat16).double()
    n = F.rms_norm(r1, (d,), T(L["mlp_norm_w"]), eps=1e-6).to(torch.bfloat16).double()
    r2 = (r1 + F.linear(F.silu(F.linear(n, T(L["w_gate"]))) * F.linear(n, T(L["w_up"])), T(L["w_down"]))).to(torch.bfloat16)
    got = orc.bf16_bits_to_f64(bits)
    dist = np.abs(got - r2.double().numpy())
    assert (dist == 0).mean() > 0.99 and np.all(dist <= np.abs(got) * 2.0 ** -7 + 1e-30)   # bf16 ties may flip a bit
    assert np.allclose(S, St.numpy().astype(np.float32), rtol=1e-6, atol=1e-9)
    assert np.array_equal(tail, _bf16_bits(Z[-3:].T.float()))
    # the state and conv state are those of single-layer replay on the normed rows
    S1, tail1 = orc.replay_layer(x.numpy(), L["w_qkv"], L["w_ab"], L["conv_w"], L["decay_scale"], L["dt_bias"], **geo)
    assert np.array_equal(S, S1) and np.array_equal(tail, tail1)


def test_group_replay_feeds_each_layer_with_the_previous_block_output():
    r = _rng(74)
    R, d, Hk, Hv, dk, dv = 10, 32, 2, 2, 4, 4
    geo = dict(n_k_heads=Hk, n_v_heads=Hv, d_k=dk, d_v=dv)
    layers = [_group_layer(r, d, Hk, Hv, dk, dv, mlp=(16 if j == 1 else 0)) for j in range(3)]
    anchors = torch.from_numpy(r.standard_normal((R, d))).to(torch.bfloat16).double().numpy()
    res = orc.group_replay(anchors, layers, **geo)
    assert len(res) == 3
    rows = anchors
    for j, L in enumerate(layers):
        bits, S, tail = orc.block_forward(rows, L, **geo)
        assert np.array_equal(res[j][0], S) and np.array_equal(res[j][1], tail)
        rows = orc.bf16_bits_to_f64(bits)
    # layers of a group are coupled only through the rows: changing layer 0's output projection changes the states of
    # layers 1 and 2 but not layer 0's
    layers2 = [dict(layers[0], w_o=layers[0]["w_o"] * 1.5)] + layers[1:]
    res2 = orc.group_replay(anchors, layers2, **geo)
    assert np.array_equal(res2[0][0], res[0][0])
    assert not np.allclose(res2[1][0], res[1][0]) and not np.allclose(res2[2][0], res[2][0])
    # a single-layer group is single-layer replay of the normed anchors
    one = orc.group_replay(anchors, layers[:1], **geo)
    assert np.array_equal(one[0][0], res[0][0])


# ----------------------------------------------------------------- sizes the paper prints

def test_state_extents_reproduce_appendix_a_table():
    rows = [ln.split() for ln in open(os.path.join(HERE, "golden", "appendix_a_state_sizes.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for name, L, d, Hk, Hv, dk, dv, C, B_rec, B_conv, B_ckpt in rows:
        L, Hk, Hv, dk, dv, C, B_rec, B_conv, B_ckpt = map(int, (L, Hk, Hv, dk, dv, C, B_rec, B_conv, B_ckpt))
        ssm, conv = orc.state_extents(Hk, Hv, dk, dv, 4)
        assert conv[0] == C
        assert int(np.prod(ssm)) * 4 == B_rec            # fp32
        assert int(np.prod(conv)) * 2 == B_conv          # bf16
        assert L * (B_rec + B_conv) == B_ckpt
