"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

The oracle cannot replay millions of layer-tokens, but every (request, layer) unit is independent
(zero initial state, read-only inputs, disjoint outputs), so checking a sample of units one by one is
a sound check of the whole call: longest and shortest request, first / middle / last rebuilt layer,
and, where pages are shared, requests that share them."""

import gc

import numpy as np
import pytest
import torch

from paper_2609_33477_b200 import binding as B
from paper_2609_33477_b200 import build as sr_build
from paper_2609_33477_b200 import synth
import parity_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module", autouse=True)
def _built():
    sr_build.build()
    B.load()


def _free():
    gc.collect()
    torch.cuda.empty_cache()


def _run_full(name):
    wl = synth.build_workload(name, device=DEV)
    rep = B.Replayer(wl)
    rep.out_ssm.fill_(float("nan"))          # every rebuilt unit must be overwritten
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    return wl, rep


def _check_units(wl, rep, units):
    worst = 0.0
    for req, layer in units:
        worst = max(worst, U.check_request_layer(rep, wl, req, layer))
    return worst


def _all_rebuilt_outputs_are_finite(wl, rep):
    active = [l for l, m in enumerate(wl.layer_mask) if m]
    assert bool(torch.isfinite(rep.out_ssm[:, active]).all())
    masked = [l for l, m in enumerate(wl.layer_mask) if not m]
    if masked:
        assert bool(torch.isnan(rep.out_ssm[:, masked]).all())     # masked layers were left alone


def test_cfg2_whole_model_replay_sampled_units():
    wl, rep = _run_full("cfg2")
    _all_rebuilt_outputs_are_finite(wl, rep)
    worst = _check_units(wl, rep, [(0, 0), (7, 23), (15, 47), (3, 30)])
    print(f"cfg2: worst rel Frobenius error per head over the sample {worst:.3e}")
    del wl, rep
    _free()


def test_cfg3_ragged_branching_batch_sampled_units():
    wl, rep = _run_full("cfg3")
    _all_rebuilt_outputs_are_finite(wl, rep)
    lens = wl.replay_lens.cpu().tolist()
    longest = max(range(len(lens)), key=lambda i: lens[i])
    shortest = min(range(len(lens)), key=lambda i: lens[i])
    # two requests of one trunk whose windows overlap on physical pages
    table = wl.page_table.cpu().numpy()
    pair = None
    for i in range(len(lens)):
        for j in range(i + 1, len(lens)):
            a = set(table[i, : lens[i] // 64].tolist())
            b = set(table[j, : lens[j] // 64].tolist())
            if a & b and lens[i] + lens[j] <= 6000:
                pair = (i, j)
                break
        if pair:
            break
    assert pair is not None, "the generator must produce windows that share pages"
    active = [l for l, m in enumerate(wl.layer_mask) if m]
    units = [(longest, active[0]), (shortest, active[-1]), (pair[0], active[len(active) // 2]),
             (pair[1], active[len(active) // 2]), (shortest, active[0])]
    worst = _check_units(wl, rep, units)
    print(f"cfg3: worst rel Frobenius error per head over the sample {worst:.3e}")
    del wl, rep
    _free()


def test_cfg4_fp8_block_scaled_weights_sampled_units():
    wl, rep = _run_full("cfg4")
    _all_rebuilt_outputs_are_finite(wl, rep)
    worst = _check_units(wl, rep, [(0, 0), (31, 23), (17, 11)])
    print(f"cfg4: worst rel Frobenius error per head over the sample {worst:.3e}")
    del wl, rep
    _free()


def test_cfg4_shorter_replay_lengths_of_the_sweep():
    for name in ("cfg4_R1024", "cfg4_R2048"):
        wl, rep = _run_full(name)
        worst = _check_units(wl, rep, [(5, 7)])
        print(f"{name}: worst rel Frobenius error per head {worst:.3e}")
        del wl, rep
        _free()


def test_cfg4_w8a8_at_full_width_sampled_units():
    """The 8-bit projection (quantised activations) at the benchmark's width and tile schedule: config 4 with 2048-row
    windows (32 requests, 24 layers, d = 5120), two (request, layer) units against the W8A8 oracle."""
    import dataclasses
    spec = dataclasses.replace(synth.SPECS["cfg4_R2048"], name="cfg4_w8a8_R2048", act_quant="e4m3_1x128")
    wl, rep = _run_full(spec)
    _all_rebuilt_outputs_are_finite(wl, rep)
    worst = _check_units(wl, rep, [(9, 3), (30, 22)])
    print(f"cfg4_w8a8_R2048: worst rel Frobenius error per head over the sample {worst:.3e}")
    del wl, rep
    _free()
