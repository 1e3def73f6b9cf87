"""Parity of the CUDA path with the CPU oracle, through the C boundary, on seeded inputs.

Floating point: per (request, layer, head) relative Frobenius error of the fp32 state <= 2e-3.
Integer / byte work (gather, page tables, packing, masks, sentinels): bit-exact."""

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


def _run(name, **kw):
    wl = synth.build_workload(name, device=DEV)
    rep = B.Replayer(wl, **kw)
    rep.replay_states()
    torch.cuda.synchronize()
    return wl, rep


def _active(wl):
    return [l for l, m in enumerate(wl.layer_mask) if m]


# ---------------------------------------------------------------------------------- parity

@pytest.mark.parametrize("name", ["cfg0", "ragged_d64", "ragged_small", "trunks_small", "fp8_small", "cfg1_narrow",
                                  "grouped_small", "decay_none", "decay_strong", "grouped3_small", "wide_v_small",
                                  "decay_only_small", "decay_only_d64", "geom_16_32", "geom_16_48", "geom_96_192",
                                  "w8a8_small", "w8a8_ragged"])
def test_small_workloads_match_oracle_everywhere(name):
    wl, rep = _run(name)
    assert rep.device_status() == 0
    worst = 0.0
    for i in range(wl.spec.n_requests):
        for l in _active(wl):
            worst = max(worst, U.check_request_layer(rep, wl, i, l))
    print(f"{name}: worst rel Frobenius error per head {worst:.3e}")
    assert rep.last_launch_count() > 0


def test_cfg1_full_size_sampled_requests():
    wl, rep = _run("cfg1")
    assert rep.device_status() == 0
    for i in (0, 5, 7):
        U.check_request_layer(rep, wl, i, 0)


def test_more_requests_than_packing_threads():
    wl, rep = _run("many_requests")
    assert rep.device_status() == 0
    lens = wl.replay_lens.cpu()
    picks = [0, 1023, 1024, 1499, int(torch.nonzero(lens == 0)[0]), int(torch.nonzero(lens == 128)[-1])]
    for i in picks:
        U.check_request_layer(rep, wl, i, 0)
    empty = torch.nonzero(lens == 0).flatten()[:50]
    assert not rep.out_ssm[empty.to(DEV)].any()                      # nothing replayed: zero state


def test_identity_activation_variant():
    wl, rep = _run("ragged_d64", conv_activation=B.SR_CONV_IDENTITY)
    for i in (2, 4):
        U.check_request_layer(rep, wl, i, 0, activation="identity")


# ------------------------------------------------------------------------- bit-exact parts

@pytest.mark.parametrize("name", ["ragged_small", "trunks_small", "cfg1_narrow"])
def test_gather_is_bit_exact(name):
    wl = synth.build_workload(name, device=DEV)
    rep = B.Replayer(wl)
    for l in _active(wl):
        got = rep.debug_gather(l)
        torch.cuda.synchronize()
        got = got.view(torch.int16).cpu().numpy().view(np.uint16)
        pool = synth.bits_u16(wl.anchor_pool)
        at = 0
        for i, R in enumerate(wl.replay_lens.cpu().tolist()):
            pages = wl.page_table[i].cpu().tolist()
            for t in range(R):
                want = pool[pages[t // 64], wl.layer_to_pool[l], t % 64]
                assert np.array_equal(got[at + t], want), (i, t)
            at += R
        assert not got[at:].any()            # nothing written past the packed rows


def test_activation_quantiser_is_bit_exact():
    """W8A8: the codes and scales the projection multiplies, against the oracle's quantiser on the same rows."""
    from oracle import gdn_replay_oracle as orc
    wl = synth.build_workload("w8a8_ragged", device=DEV)
    rep = B.Replayer(wl)
    for l in _active(wl):
        codes, scales = rep.debug_quantise(l)
        torch.cuda.synchronize()
        codes, scales = codes.cpu().numpy(), scales.cpu().numpy()
        at = 0
        for i, R in enumerate(wl.replay_lens.cpu().tolist()):
            if R == 0:
                continue
            pages = wl.page_table[i, : -(-R // 64)].cpu().tolist()
            pl = wl.layer_to_pool[l]
            X = orc.gather_anchor_rows(synth.fetch_pages(wl, pages, pl), pages, R, pl)
            want_codes, want_scales = orc.quantise_e4m3_1x128(X)
            assert np.array_equal(codes[at:at + R], want_codes), (l, i)
            assert np.array_equal(scales[at:at + R], want_scales), (l, i)
            at += R
        assert not codes[at:].any() and not scales[at:].any()


def test_masked_layers_and_other_slots_are_not_touched():
    wl = synth.build_workload("ragged_small", device=DEV)
    rep = B.Replayer(wl, n_slots=wl.spec.n_requests + 2)
    rep.out_ssm.fill_(7.25)
    rep.out_conv.fill_(-3.0)
    rep.replay_states()
    torch.cuda.synchronize()
    assert torch.all(rep.out_ssm[:, 1] == 7.25) and torch.all(rep.out_conv[:, 1] == -3.0)     # masked layer
    assert torch.all(rep.out_ssm[-2:] == 7.25) and torch.all(rep.out_conv[-2:] == -3.0)       # unused slots
    # request 0 replays nothing: zero state, zero conv state
    assert torch.all(rep.out_ssm[0, 0] == 0) and torch.all(rep.out_conv[0, 0] == 0)
    U.check_request_layer(rep, wl, 5, 2)


def test_state_slots_and_sentinel_segments():
    wl = synth.build_workload("ragged_d64", device=DEV)
    slots = torch.tensor([3, -1, 0, 4, -1], dtype=torch.int32, device=DEV)
    rep = B.Replayer(wl, state_slots=slots, n_slots=5)
    rep.out_ssm.fill_(1.5)
    rep.out_conv.fill_(2.0)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0                                   # a sentinel is not an error
    for s in (1, 2):                                                  # no request writes slots 1 and 2
        assert torch.all(rep.out_ssm[s] == 1.5) and torch.all(rep.out_conv[s] == 2.0)
    for req, s in ((0, 3), (2, 0), (3, 4)):
        for l in (0, 1):
            U.check_request_layer(rep, wl, req, l, slot=s)


def test_invalid_requests_are_skipped_and_flagged():
    wl = synth.build_workload("ragged_d64", device=DEV)
    wl.page_table[2, 1] = wl.n_phys_pages + 5         # request 2 (127 rows) uses a page outside the pool
    wl.replay_lens[3] = -4                            # request 3 has a negative length
    rep = B.Replayer(wl, max_total_rows=4 + 63 + 127 + 128 + 321, max_replay_len=321)
    rep.out_ssm.fill_(9.0)
    rep.out_conv.fill_(9.0)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == (B.SR_DEV_BAD_PAGE_ID | B.SR_DEV_BAD_REPLAY_LEN)
    for bad in (2, 3):
        assert torch.all(rep.out_ssm[bad] == 9.0) and torch.all(rep.out_conv[bad] == 9.0)
    for good in (0, 1, 4):
        U.check_request_layer(rep, wl, good, 1)


def test_destination_slot_beyond_the_output_arrays_is_a_miss():
    wl = synth.build_workload("ragged_d64", device=DEV)
    slots = torch.tensor([0, 1, 7, 3, 4], dtype=torch.int32, device=DEV)      # the arrays hold 5 slots: 7 is outside
    rep = B.Replayer(wl, state_slots=slots, n_slots=5)
    rep.out_ssm.fill_(9.0)
    rep.out_conv.fill_(9.0)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == B.SR_DEV_BAD_SLOT
    assert torch.all(rep.out_ssm[2] == 9.0) and torch.all(rep.out_conv[2] == 9.0)      # nobody wrote slot 2
    for req in (0, 1, 3, 4):
        U.check_request_layer(rep, wl, req, 0)


def test_rows_beyond_the_declared_bound_are_a_miss():
    wl = synth.build_workload("ragged_d64", device=DEV)
    rep = B.Replayer(wl, max_total_rows=4 + 63 + 127, max_replay_len=321)     # last two requests do not fit
    rep.out_ssm.fill_(9.0)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == B.SR_DEV_ROWS_OVERFLOW
    assert torch.all(rep.out_ssm[3:] == 9.0)
    U.check_request_layer(rep, wl, 2, 0)


def test_physical_page_placement_does_not_change_a_bit():
    wl, rep = _run("ragged_small")
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    perm = torch.randperm(wl.n_phys_pages, generator=torch.Generator().manual_seed(5)).to(DEV)
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(wl.n_phys_pages, device=DEV)
    wl2 = synth.build_workload("ragged_small", device=DEV)
    wl2.anchor_pool = wl.anchor_pool[perm].contiguous()            # page p now lives at inv[p]
    valid = wl2.page_table >= 0
    wl2.page_table[valid] = inv[wl2.page_table[valid].long()].to(torch.int32)
    rep2 = B.Replayer(wl2)
    rep2.replay_states()
    torch.cuda.synchronize()
    assert torch.equal(rep2.out_ssm, ref_ssm) and torch.equal(rep2.out_conv, ref_conv)


def test_strided_pool_layout_gives_the_same_bits():
    wl, rep = _run("trunks_small")
    ref = rep.out_ssm.clone()
    # same anchors stored layer-major with padded rows: [L_pool][n_phys][64][d + 64]
    n_phys, L_pool, P, d = wl.anchor_pool.shape
    padded = torch.zeros((L_pool, n_phys, P, d + 64), dtype=torch.bfloat16, device=DEV)
    padded[..., :d] = wl.anchor_pool.permute(1, 0, 2, 3)
    rep.set_pool(padded.permute(1, 0, 2, 3)[..., :d])
    rep.out_ssm.zero_()
    rep.replay_states()
    torch.cuda.synchronize()
    assert torch.equal(rep.out_ssm, ref)


def test_run_to_run_bit_reproducible():
    wl, rep = _run("cfg1_narrow")
    a, c = rep.out_ssm.clone(), rep.out_conv.clone()
    for _ in range(3):
        rep.out_ssm.zero_()
        rep.replay_states()
        torch.cuda.synchronize()
        assert torch.equal(rep.out_ssm, a) and torch.equal(rep.out_conv, c)


def test_replay_of_a_longer_window_converges_to_the_same_state():
    """Suffix replay forgets the distant past (Eq. 2): two windows ending at the same row give
    states whose difference is bounded by the decay accumulated over the shorter window."""
    spec = synth.SPECS["cfg1_narrow"]
    wl = synth.build_workload(spec, device=DEV)
    # request 1 replays only the last half of request 0's pages
    wl.page_table[1, :4] = wl.page_table[0, 4:8]
    wl.replay_lens[1] = 256
    rep = B.Replayer(wl, max_total_rows=4 * 512, max_replay_len=512)
    rep.replay_states()
    torch.cuda.synchronize()
    full, half = rep.out_ssm[0, 0].double(), rep.out_ssm[1, 0].double()
    rel = (torch.linalg.matrix_norm(full - half) / torch.linalg.matrix_norm(full)).max().item()
    assert rel < 1e-4          # exp(-0.1 * 0.8 * 256) is ~1e-9: the first half of the window is forgotten
    assert torch.equal(rep.out_conv[0, 0], rep.out_conv[1, 0])   # same last rows -> same conv state


def test_host_buffer_entry_matches_device_entry():
    wl, rep = _run("ragged_small")
    ref_ssm, ref_conv = rep.out_ssm.cpu(), rep.out_conv.cpu()
    host_pool = wl.anchor_pool.cpu().pin_memory()
    host_pages = wl.page_table.cpu().pin_memory()
    host_lens = wl.replay_lens.cpu().pin_memory()
    out_ssm = torch.full_like(ref_ssm, 7.0).pin_memory()
    out_conv = torch.full_like(ref_conv, 7.0).pin_memory()
    staging = torch.zeros_like(wl.anchor_pool)
    rep.set_pool(staging)
    wl.page_table.zero_()
    wl.replay_lens.zero_()
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    for _ in range(2):      # twice back to back: the second call's copies must wait for the first call's kernels
        rep.replay_states_host(host_pool, host_pages, host_lens, out_ssm, out_conv)
    torch.cuda.synchronize()
    for l in range(wl.spec.n_layers):
        if wl.layer_mask[l]:
            assert torch.equal(out_ssm[:, l], ref_ssm[:, l]) and torch.equal(out_conv[:, l], ref_conv[:, l])
        else:               # layers that are not rebuilt are not copied back
            assert bool((out_ssm[:, l] == 7.0).all()) and bool((out_conv[:, l] == 7.0).all())


def test_host_buffer_entry_with_a_layer_major_padded_pool():
    """Per-layer uploads of a pool stored [L_pool][n_phys][64][d + pad]: a pool layer is one contiguous run of
    page blocks whose rows carry padding; the host image has the same bytes."""
    wl, rep = _run("trunks_small")
    ref_ssm, ref_conv = rep.out_ssm.cpu(), rep.out_conv.cpu()
    n_phys, L_pool, P, d = wl.anchor_pool.shape
    host = torch.zeros((L_pool, n_phys, P, d + 64), dtype=torch.bfloat16).pin_memory()
    host[..., :d] = wl.anchor_pool.permute(1, 0, 2, 3).cpu()
    staging = torch.zeros((L_pool, n_phys, P, d + 64), dtype=torch.bfloat16, device=DEV)
    rep.set_pool(staging.permute(1, 0, 2, 3)[..., :d])
    host_pages, host_lens = wl.page_table.cpu().pin_memory(), wl.replay_lens.cpu().pin_memory()
    out_ssm, out_conv = torch.zeros_like(ref_ssm).pin_memory(), torch.zeros_like(ref_conv).pin_memory()
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    rep.replay_states_host(host, host_pages, host_lens, out_ssm, out_conv)
    torch.cuda.synchronize()
    for l in _active(wl):
        assert torch.equal(out_ssm[:, l], ref_ssm[:, l]) and torch.equal(out_conv[:, l], ref_conv[:, l])
    assert torch.equal(staging[..., :d].cpu(), host[..., :d])            # every pool layer in use went up


def test_host_buffer_entry_with_a_row_major_pool_goes_up_in_one_piece():
    """A pool stored [64 rows][n_phys][L_pool][d]: a page-layer block is not contiguous, so the host entry cannot
    slice it by layer and copies the whole image once; the strides are still what the kernels read through."""
    wl, rep = _run("ragged_small")
    ref_ssm, ref_conv = rep.out_ssm.cpu(), rep.out_conv.cpu()
    host = wl.anchor_pool.permute(2, 0, 1, 3).contiguous().cpu().pin_memory()         # [P][n_phys][L_pool][d]
    staging = torch.zeros(host.shape, dtype=torch.bfloat16, device=DEV)
    rep.set_pool(staging.permute(1, 2, 0, 3))
    host_pages, host_lens = wl.page_table.cpu().pin_memory(), wl.replay_lens.cpu().pin_memory()
    out_ssm, out_conv = torch.zeros_like(ref_ssm).pin_memory(), torch.zeros_like(ref_conv).pin_memory()
    rep.replay_states_host(host, host_pages, host_lens, out_ssm, out_conv)
    torch.cuda.synchronize()
    for l in _active(wl):
        assert torch.equal(out_ssm[:, l], ref_ssm[:, l]) and torch.equal(out_conv[:, l], ref_conv[:, l])


# ----------------------------------------------------- second forms of single steps (debug flags)

@pytest.mark.parametrize("flag,name", [
    (B.SR_DEBUG_FP8_EXACT, "fp8_small"),          # fp32 promotion of bare-code partial sums, no fp16 staging
    (B.SR_DEBUG_DOT_CONV_STATE, "ragged_small"),  # conv state by per-channel dot products
    (B.SR_DEBUG_DOT_CONV_STATE, "fp8_small"),
    (B.SR_DEBUG_SINGLE_CTA_MMA, "cfg1_narrow"),   # one-CTA form of the fused projection
    (B.SR_DEBUG_CHECK_BOUNDS, "ragged_small"),    # device-side range checks on: same results, no flag raised
    (B.SR_DEBUG_CHECK_BOUNDS, "trunks_small"),
    (B.SR_DEBUG_CHECK_BOUNDS, "geom_96_192"),
    (B.SR_DEBUG_CHECK_BOUNDS | B.SR_DEBUG_DOT_CONV_STATE, "fp8_small"),
])
def test_second_forms_match_oracle(flag, name):
    wl, rep = _run(name, debug_flags=flag)
    assert rep.device_status() == 0
    for i in range(wl.spec.n_requests):
        for l in _active(wl):
            U.check_request_layer(rep, wl, i, l)


# ----------------------------------------------------- layers of one call side by side

def test_layers_run_side_by_side_with_the_same_bits_as_one_after_the_other():
    """A small batch with nine rebuilt layers: with the recommended workspace the call spreads the layers over
    several streams of the context, with the minimum workspace it runs them in order.  Same bits either way, and
    both match the oracle."""
    wl = synth.build_workload("layers_small", device=DEV)
    wide = B.Replayer(wl)
    narrow = B.Replayer(wl, min_workspace=True)
    assert wide.workspace_bytes > narrow.workspace_bytes
    for rep in (wide, narrow):
        for _ in range(2):
            rep.out_ssm.fill_(float("nan"))
            rep.replay_states()
            torch.cuda.synchronize()
            assert rep.device_status() == 0
    assert torch.equal(wide.out_ssm, narrow.out_ssm) and torch.equal(wide.out_conv, narrow.out_conv)
    for l in (0, 4, 8):
        for i in range(wl.spec.n_requests):
            U.check_request_layer(wide, wl, i, l)
    # and inside a captured graph: the side streams fork from and join the capturing stream
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        wide.replay_states(torch.cuda.current_stream())
    wide.out_ssm.zero_()
    wide.out_conv.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(wide.out_ssm, narrow.out_ssm) and torch.equal(wide.out_conv, narrow.out_conv)


# ----------------------------------------------------- a bounded in-kernel wait that runs out

def test_an_expired_wait_raises_the_status_bit_and_leaves_the_device_usable():
    """Fault injection without a GPU fault: with SR_DEBUG_EXPIRE_WAIT the state chain never requests the first
    key tile and its waits give up after about a millisecond.  The kernel must then return normally: status bit
    set, state outputs untouched, tensor memory released -- shown by a following ordinary call on the same
    device giving the same bits as before."""
    wl, rep = _run("ragged_small")
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    wl2 = synth.build_workload("ragged_small", device=DEV)
    bad = B.Replayer(wl2, debug_flags=B.SR_DEBUG_EXPIRE_WAIT)
    bad.out_ssm.fill_(5.0)
    bad.replay_states()
    torch.cuda.synchronize()
    assert bad.device_status() & B.SR_DEV_WAIT_EXPIRED
    lens = wl2.replay_lens.cpu().tolist()
    for i, R in enumerate(lens):
        for l in _active(wl2):
            if R > 0:
                assert torch.all(bad.out_ssm[i, l] == 5.0)            # a chain that gave up writes nothing
            else:
                assert torch.all(bad.out_ssm[i, l] == 0.0)            # nothing to wait for: zero state as usual
    assert torch.equal(bad.out_conv, ref_conv)                        # the conv state does not pass through the chain
    bad.close()
    for _ in range(2):
        rep.out_ssm.zero_()
        rep.replay_states()
        torch.cuda.synchronize()
        assert rep.device_status() == 0
        assert torch.equal(rep.out_ssm, ref_ssm) and torch.equal(rep.out_conv, ref_conv)


# ----------------------------------------------------- windows that end inside a page

def test_rows_past_the_window_in_its_last_page_are_never_used():
    """A window may end anywhere inside its last page (R = 65 and 200 here).  The rows behind it on that page
    are not part of the replay -- in a live pool they are stale or not yet written -- so filling them with NaN,
    infinities and huge values must not change one bit of the result."""
    wl, rep = _run("ragged_small")
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    wl2 = synth.build_workload("ragged_small", device=DEV)
    junk = torch.tensor([float("nan"), float("inf"), -float("inf"), 3.0e38], dtype=torch.bfloat16, device=DEV)
    for i, R in enumerate(wl2.replay_lens.cpu().tolist()):
        if R % 64:
            page = int(wl2.page_table[i, R // 64])
            tail = wl2.anchor_pool[page, :, R % 64:, :]
            tail.copy_(junk[torch.arange(tail.numel(), device=DEV) % 4].view(tail.shape))
    rep2 = B.Replayer(wl2)
    rep2.replay_states()
    torch.cuda.synchronize()
    assert rep2.device_status() == 0
    assert torch.equal(rep2.out_ssm, ref_ssm) and torch.equal(rep2.out_conv, ref_conv)


def test_long_window_with_a_partial_last_chunk():
    """Many full chunks followed by a partial one at d_k = d_v = 128: R = 4096 + 17 rows in one request."""
    spec = synth.WorkloadSpec(name="long_ragged", n_layers=1, d_model=1024, n_k_heads=4, n_v_heads=4, d_k=128,
                              d_v=128, n_requests=2, replay=("list", (4096 + 17, 64 * 3 + 63)))
    wl = synth.build_workload(spec, device=DEV)
    rep = B.Replayer(wl)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    for i in range(2):
        U.check_request_layer(rep, wl, i, 0)


def test_guard_bands_around_outputs_and_workspace_stay_intact():
    """Outputs and workspace sit inside larger allocations whose margins are filled with a pattern: the call must
    not write one byte outside the extents the boundary states (a stand-in for a memory checker)."""
    wl = synth.build_workload("ragged_small", device=DEV)
    s = wl.spec
    band = 1 << 16
    L, B_ = s.n_layers, s.n_requests
    ssm_elems = B_ * L * s.n_v_heads * s.d_k * s.d_v
    conv_elems = B_ * L * s.conv_channels * (s.conv_width - 1)
    big_ssm = torch.full((ssm_elems + 2 * band,), 123.0, dtype=torch.float32, device=DEV)
    big_conv = torch.full((conv_elems + 2 * band,), 123.0, dtype=torch.bfloat16, device=DEV)
    out_ssm = big_ssm[band:band + ssm_elems].view(B_, L, s.n_v_heads, s.d_k, s.d_v)
    out_conv = big_conv[band:band + conv_elems].view(B_, L, s.conv_channels, s.conv_width - 1)
    rep = B.Replayer(wl, out_ssm=out_ssm, out_conv=out_conv)
    big_ws = torch.full((rep.workspace_bytes + 2 * band + 256,), 0x5A, dtype=torch.uint8, device=DEV)
    ws_ptr = (big_ws.data_ptr() + band + 255) // 256 * 256
    off = ws_ptr - big_ws.data_ptr()
    rep.workspace, rep._ws_ptr = big_ws, ws_ptr
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    assert bool((big_ssm[:band] == 123.0).all()) and bool((big_ssm[band + ssm_elems:] == 123.0).all())
    assert bool((big_conv[:band] == 123.0).all()) and bool((big_conv[band + conv_elems:] == 123.0).all())
    assert bool((big_ws[:off] == 0x5A).all()) and bool((big_ws[off + rep.workspace_bytes:] == 0x5A).all())
    U.check_request_layer(rep, wl, 5, 2)


# ----------------------------------------------------- graph capture (Section 6, "Replay graphs": static buffers)

def test_call_is_graph_capturable_with_device_side_boundaries():
    """The call allocates nothing, never synchronises and reads lengths, pages and slots on the device, so one
    captured graph serves batches of different lengths; padding requests carry the sentinel slot."""
    wl = synth.build_workload("ragged_small", device=DEV)
    rep = B.Replayer(wl)
    side = torch.cuda.Stream()
    lens_a = wl.replay_lens.clone()
    lens_b = torch.tensor([0, 0, 2, 33, 64, 129], dtype=torch.int32, device=DEV)   # within each request's pages
    with torch.cuda.stream(side):
        rep.replay_states(side)                     # warm-up outside the capture (one-time function attributes)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        rep.replay_states(torch.cuda.current_stream())
    for lens in (lens_b, lens_a):
        wl.replay_lens.copy_(lens)
        rep.out_ssm.fill_(float("nan"))
        rep.out_conv.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got_ssm, got_conv = rep.out_ssm.clone(), rep.out_conv.clone()
        assert rep.device_status() == 0
        rep.out_ssm.fill_(float("nan"))
        rep.out_conv.zero_()
        rep.replay_states()
        torch.cuda.synchronize()
        for l in range(wl.spec.n_layers):
            if wl.layer_mask[l]:
                assert torch.equal(got_ssm[:, l], rep.out_ssm[:, l]) and torch.equal(got_conv[:, l], rep.out_conv[:, l])
    U.check_request_layer(rep, wl, 5, 0)


@pytest.mark.parametrize("name", ["many_requests", "fp8_many"])
def test_a_request_gets_the_same_bits_alone_and_in_a_large_batch(name):
    """The conv-state kernel gives every quarter of the k range its own CTA on small batches and walks the quarters in
    one CTA on large ones; the sums are formed in the same order, so both states of a request are bit-identical
    whatever batch it arrives in (a comparison of the CUDA path with itself; both batch sizes are compared with the
    oracle elsewhere)."""
    import dataclasses
    if name == "fp8_many":
        spec = dataclasses.replace(synth.SPECS["many_requests"], name="fp8_many", n_requests=120, weight_format="e4m3_block128")
    else:
        spec = synth.SPECS[name]
    wl = synth.build_workload(spec, device="cuda")
    rep = B.Replayer(wl)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    lens = wl.replay_lens.cpu().tolist()
    picks = [i for i, r in enumerate(lens) if r > 0][:2] + [max(range(len(lens)), key=lambda i: lens[i])]
    for i in picks:
        n_pg = max(1, -(-lens[i] // 64))
        one = dataclasses.replace(wl, page_table=wl.page_table[i:i + 1, :n_pg].contiguous(), replay_lens=wl.replay_lens[i:i + 1].clone())
        rep1 = B.Replayer(one)
        rep1.replay_states()
        torch.cuda.synchronize()
        assert torch.equal(rep1.out_conv[0], rep.out_conv[i]) and torch.equal(rep1.out_ssm[0], rep.out_ssm[i])
        rep1.close()


def test_layers_projected_in_one_launch_match_layers_projected_alone():
    """A small batch with bf16 weights runs the projections of all its layers as one launch; a call that rebuilds a
    single layer runs that layer's own launch.  Tile for tile the arithmetic is the same, so both states of every
    layer are bit-identical (a comparison of the CUDA path with itself; `layers_small` is compared with the oracle
    in the named-workload test)."""
    import dataclasses
    wl = synth.build_workload("layers_small", device="cuda")
    rep = B.Replayer(wl)
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    n = len(wl.layer_mask)
    for l in (0, 4, n - 1):
        one = dataclasses.replace(wl, layer_mask=[1 if j == l else 0 for j in range(n)])
        rep1 = B.Replayer(one)
        rep1.replay_states()
        torch.cuda.synchronize()
        assert rep1.device_status() == 0
        assert torch.equal(rep1.out_ssm[:, l], rep.out_ssm[:, l]) and torch.equal(rep1.out_conv[:, l], rep.out_conv[:, l])
        assert rep1.last_launch_count() < rep.last_launch_count()
        rep1.close()
    rep.close()
