"""Helpers shared by the GPU parity tests: run the oracle on the raw bytes of a workload and
compare the CUDA path's outputs with it."""

import numpy as np
import torch

from oracle import gdn_replay_oracle as orc
from paper_2609_33477_b200 import synth

REL_FROB_TOL = 2e-3   # per head, relative Frobenius error of the fp32 state (bf16 in, fp32 accumulate)


def oracle_request_layer(wl, request, layer, activation="silu", eps=1e-6, S0=None, conv_state_bits=None):
    """Oracle state and conv tail for one (request, layer), from bytes copied off the workload."""
    s = wl.spec
    R = int(wl.replay_lens[request].item())
    n_pages = -(-R // synth.PAGE_ROWS)
    pages = wl.page_table[request, :n_pages].cpu().tolist()
    pl = wl.layer_to_pool[layer]
    pool = synth.fetch_pages(wl, pages, pl)
    arrays = synth.layer_arrays(wl.layers[layer])
    return orc.replay_request_layer(pool, pages, R, pl, arrays, n_k_heads=s.n_k_heads, n_v_heads=s.n_v_heads,
                                    d_k=s.d_k, d_v=s.d_v, eps=eps, activation=activation, S0=S0,
                                    conv_state_bits=conv_state_bits, erase=s.recurrence != "decay_only",
                                    act_quant=getattr(s, "act_quant", "none"))


def rel_frob_per_head(S_gpu, S_ref):
    """max over heads of |S_gpu - S_ref|_F / |S_ref|_F; a zero reference demands an exactly zero result."""
    worst = 0.0
    for h in range(S_ref.shape[0]):
        ref = S_ref[h].astype(np.float64)
        got = S_gpu[h].astype(np.float64)
        den = np.linalg.norm(ref)
        if den == 0.0:
            assert np.all(got == 0.0), f"head {h}: reference state is zero but the result is not"
            continue
        worst = max(worst, float(np.linalg.norm(got - ref) / den))
    return worst


def bf16_ulp_distance(bits_a, bits_b):
    """Distance in bf16 steps between two uint16 bit arrays (sign-magnitude -> ordered ints)."""
    def ordered(b):
        b = b.astype(np.int32)
        return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)
    return np.abs(ordered(bits_a) - ordered(bits_b))


def check_request_layer(rep, wl, request, layer, slot=None, activation="silu", tol=REL_FROB_TOL, S0=None,
                        conv_state_bits=None):
    """Compare one (request, layer) of a finished replay call with the oracle; returns the error.
    `S0` / `conv_state_bits`: the states the call continued from (zero when None)."""
    slot = request if slot is None else slot
    S_ref, tail_ref = oracle_request_layer(wl, request, layer, activation, S0=S0, conv_state_bits=conv_state_bits)
    S_gpu = rep.out_ssm[slot, layer].cpu().numpy()
    tail_gpu = rep.out_conv[slot, layer].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    err = rel_frob_per_head(S_gpu, S_ref)
    assert np.all(np.isfinite(S_gpu))
    assert err <= tol, f"request {request} layer {layer}: rel Frobenius {err:.3e} > {tol}"
    # The conv state is the fp32 projection rounded once to bf16.  It may differ from the fp64
    # oracle's rounding by one bf16 step where the fp32 sum lands on the other side of a rounding
    # boundary (plus the fp32 sum's own ~1e-5 absolute error for entries near zero); that must be rare.
    dist = bf16_ulp_distance(tail_gpu, tail_ref)
    a, b = orc.bf16_bits_to_f64(tail_gpu), orc.bf16_bits_to_f64(tail_ref)
    slack, differ_max = np.full(a.shape, 1e-5), 0.02
    step = np.where(b != 0, 2.0 ** (np.floor(np.log2(np.abs(np.where(b != 0, b, 1.0)))) - 7), 0.0)
    ok = (dist <= 1) | (np.abs(a - b) <= slack + step)
    assert ok.all(), f"request {request} layer {layer}: conv state off by {dist[~ok].max()} bf16 steps"
    assert (dist > 0).mean() <= differ_max, f"conv state: {(dist > 0).mean():.3%} of entries differ"
    return err
