"""Replay that continues earlier states (sr_replay_states_from) against the oracle and against one-pass replay."""

import numpy as np
import pytest
import torch

import parity_util as U
from paper_2609_33477_b200 import binding, synth
from paper_2609_33477_b200 import build as sr_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    sr_build.build()
    binding.load()


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _random_states(rep, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    in_ssm = 0.05 * torch.randn(rep.out_ssm.shape, generator=g, device="cuda", dtype=torch.float32)
    in_conv = torch.randn(rep.out_conv.shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    return in_ssm, in_conv


@pytest.mark.parametrize("name", ["ragged_small", "fp8_small", "grouped_small", "decay_only_small",
                                  "ragged_d64", "wide_v_small", "grouped3_small"])
def test_continuation_matches_oracle(name):
    wl = synth.build_workload(name, device="cuda")
    rep = binding.Replayer(wl)
    in_ssm, in_conv = _random_states(rep, 7)
    rep.out_ssm.fill_(float("nan"))
    rep.replay_states_from(in_ssm, in_conv)
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    for l in range(wl.spec.n_layers):
        if not wl.layer_mask[l]:
            continue
        for i in range(wl.spec.n_requests):
            U.check_request_layer(rep, wl, i, l, S0=in_ssm[i, l].cpu().numpy().astype(np.float64),
                                  conv_state_bits=_bits(in_conv[i, l]))


def test_only_one_of_the_two_states_given():
    wl = synth.build_workload("ragged_small", device="cuda")
    rep = binding.Replayer(wl)
    in_ssm, in_conv = _random_states(rep, 8)
    rep.replay_states_from(in_ssm, None)
    torch.cuda.synchronize()
    U.check_request_layer(rep, wl, 5, 0, S0=in_ssm[5, 0].cpu().numpy().astype(np.float64))
    U.check_request_layer(rep, wl, 1, 2, S0=in_ssm[1, 2].cpu().numpy().astype(np.float64))
    rep.replay_states_from(None, in_conv)
    torch.cuda.synchronize()
    U.check_request_layer(rep, wl, 5, 0, conv_state_bits=_bits(in_conv[5, 0]))
    U.check_request_layer(rep, wl, 2, 0, conv_state_bits=_bits(in_conv[2, 0]))     # 3 rows: window = whole conv state


def test_two_pieces_in_place_equal_one_pass():
    """Rows [0, 512) at once against rows [0, 192) followed, in place, by rows [192, 512)."""
    wl = synth.build_workload("cfg1_narrow", device="cuda")
    rep = binding.Replayer(wl)
    rep.replay_states()
    torch.cuda.synchronize()
    one_ssm, one_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    pages = wl.page_table.clone()
    wl.replay_lens.fill_(192)
    rep.replay_states()
    wl.page_table[:, :5] = pages[:, 3:8]
    wl.replay_lens.fill_(320)
    rep.replay_states_from(rep.out_ssm, rep.out_conv)          # the outputs are also the states to continue
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    assert torch.equal(rep.out_conv, one_conv)                  # the same last three rows
    for i in range(wl.spec.n_requests):
        err = U.rel_frob_per_head(rep.out_ssm[i, 0].cpu().numpy(), one_ssm[i, 0].cpu().numpy())
        assert err <= U.REL_FROB_TOL, err
    # and against the oracle's one pass
    wl.page_table.copy_(pages)
    wl.replay_lens.fill_(512)
    U.check_request_layer(rep, wl, 1, 0)


def test_zero_length_continuation_hands_the_states_through():
    wl = synth.build_workload("ragged_small", device="cuda")
    rep = binding.Replayer(wl)
    in_ssm, in_conv = _random_states(rep, 9)
    wl.replay_lens.zero_()
    rep.replay_states_from(in_ssm, in_conv)
    torch.cuda.synchronize()
    for l in range(wl.spec.n_layers):
        if wl.layer_mask[l]:
            assert torch.equal(rep.out_ssm[:, l], in_ssm[:, l]) and torch.equal(rep.out_conv[:, l], in_conv[:, l])
