"""The replay entry point for callers that cannot allocate device memory.

`sr_replay_states_noalloc` takes no workspace: its scratch is a fixed array inside the library.
A caller that may not call cudaMalloc (or a framework allocator) on its serving path -- an engine
with a frozen memory pool, a plugin, a step that is set up once and re-issued -- uses it in place of
`sr_replay_states`.  This test drives it through the C boundary twice in a row (the second call
finds the first call's leftovers in the shared scratch) and checks both results against the
ordinary entry point on the same inputs.  That is a comparison of the CUDA path with itself: the
entry is a wrapper, and the call it wraps is compared with the CPU oracle on these same workloads in
test_parity_gpu.py.  This file sorts last so that every other test has already run if it fails; it
must also pass alone in a fresh process."""

import ctypes as C

import pytest
import torch

from paper_2609_33477_b200 import binding as B
from paper_2609_33477_b200 import build as sr_build
from paper_2609_33477_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _reference(name):
    wl = synth.build_workload(name, device=DEV)
    rep = B.Replayer(wl)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    return wl, rep, rep.out_ssm.clone(), rep.out_conv.clone()


def _call_noalloc(rep):
    stream = torch.cuda.current_stream(rep.device).cuda_stream
    return B.sr_replay_states_noalloc(rep.ctx, rep.pool, rep.table, rep.wl.replay_lens.data_ptr(), rep.layer_mask,
                                      rep.weights, rep._out_ssm, rep._out_conv, stream)


def test_noalloc_entry_matches_the_workspace_entry_on_two_calls_in_a_row():
    sr_build.build()
    B.load()
    # two different batches back to back: the second one runs on whatever the first left in the scratch
    seen_first_call = False
    for name in ("ragged_small", "trunks_small", "ragged_small"):
        wl, rep, ref_ssm, ref_conv = _reference(name)
        for call in range(2):
            rep.out_ssm.fill_(-1.0)
            rep.out_conv.fill_(-1.0)
            torch.cuda.synchronize()
            before = torch.cuda.memory_allocated(DEV)
            free_before = torch.cuda.mem_get_info(DEV)[0]
            assert _call_noalloc(rep) == B.SR_OK
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated(DEV) == before          # nothing came from torch's allocator
            # ... and nothing from the driver either.  The very first call on a device may materialise the
            # library's scratch array (the module that holds it is loaded on first use); later calls must not
            # move the device's free memory at all.
            if seen_first_call:
                assert torch.cuda.mem_get_info(DEV)[0] == free_before
            seen_first_call = True
            active = [l for l, m in enumerate(wl.layer_mask) if m]
            # same kernels, same inputs, same order of operations: identical bits, so also within the 2e-3
            # relative Frobenius bound the oracle tests use for the state
            assert torch.equal(rep.out_ssm[:, active], ref_ssm[:, active])
            assert torch.equal(rep.out_conv[:, active], ref_conv[:, active])
            num = torch.linalg.matrix_norm((rep.out_ssm[:, active] - ref_ssm[:, active]).double())
            den = torch.linalg.matrix_norm(ref_ssm[:, active].double()).clamp_min(1e-30)
            assert float((num / den).max()) <= 2e-3
            masked = [l for l, m in enumerate(wl.layer_mask) if not m]
            if masked:
                assert torch.all(rep.out_ssm[:, masked] == -1.0)       # masked layers stay untouched
        rep.close()


def test_noalloc_entry_refuses_batches_beyond_its_fixed_scratch():
    sr_build.build()
    wl = synth.build_workload("ragged_small", device=DEV)
    rep = B.Replayer(wl)
    # bounds that would need more scratch than the library holds: refused on the host, nothing launched
    big = B.sr_page_table(rep.table.pages, None, rep.table.n_requests, rep.table.max_pages,
                          rep.table.max_replay_len, 1 << 20)
    big.max_pages = 1 << 16
    big.max_replay_len = 1 << 20
    need = B.sr_workspace_bytes(rep.ctx, big)
    assert need > B.SR_NOALLOC_SCRATCH_BYTES
    stream = torch.cuda.current_stream(rep.device).cuda_stream
    st = B.sr_replay_states_noalloc(rep.ctx, rep.pool, big, wl.replay_lens.data_ptr(), rep.layer_mask, rep.weights,
                                    rep._out_ssm, rep._out_conv, stream)
    assert st == B.SR_ERR_WORKSPACE
    assert B.sr_last_launch_count(rep.ctx) == 0
    rep.close()
