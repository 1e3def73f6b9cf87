"""Replay graphs per bucket with static buffers and sentinel padding (Section 5.2, Section 6) against the direct call
(a comparison of the CUDA path with itself: the direct call is compared with the CPU oracle on the same workload in
test_parity_gpu.py)."""

import pytest
import torch

import parity_util as U
from paper_2609_33477_b200 import binding, graphs, synth
from paper_2609_33477_b200 import build as sr_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    sr_build.build()
    binding.load()


def test_bucketed_graphs_match_the_direct_call_and_pad_with_sentinels():
    wl = synth.build_workload("trunks_small", device="cuda")
    B = wl.spec.n_requests
    rep = binding.Replayer(wl)
    rep.replay_states()
    torch.cuda.synchronize()
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    total = int(wl.replay_lens.sum().item())
    runner = graphs.BucketedGraphReplayer(wl, buckets=[(2, 512), (4, 1024), (B + 3, total + 64)], n_slots=B)
    # the whole batch: only the largest bucket holds it; three padding segments ride along
    host_lens = wl.replay_lens.cpu()
    used = runner.replay(wl.page_table, host_lens, torch.arange(B, dtype=torch.int32))
    torch.cuda.synchronize()
    assert used == 2 and runner.device_status(used) == 0
    for l in range(wl.spec.n_layers):
        if wl.layer_mask[l]:
            assert torch.equal(runner.out_ssm[:, l], ref_ssm[:, l]) and torch.equal(runner.out_conv[:, l], ref_conv[:, l])
    # two requests, written to other slots, through the smallest bucket that fits
    runner.out_ssm.zero_()
    runner.out_conv.zero_()
    pick = [5, 1]
    lens = host_lens[pick]
    used = runner.replay(wl.page_table[pick], lens, torch.tensor([0, 3], dtype=torch.int32))
    torch.cuda.synchronize()
    assert used == runner.pick(2, int(lens.sum().item())) and runner.device_status(used) == 0
    for l in range(wl.spec.n_layers):
        if wl.layer_mask[l]:
            assert torch.equal(runner.out_ssm[0, l], ref_ssm[5, l]) and torch.equal(runner.out_ssm[3, l], ref_ssm[1, l])
            assert torch.equal(runner.out_conv[0, l], ref_conv[5, l])
            assert not runner.out_ssm[[1, 2, 4], l].any()          # no other slot was touched
    with pytest.raises(ValueError):
        runner.pick(B + 4, 10)
    with pytest.raises(ValueError):                                # device-side lengths would force a host sync
        runner.replay(wl.page_table, wl.replay_lens, torch.arange(B, dtype=torch.int32))
