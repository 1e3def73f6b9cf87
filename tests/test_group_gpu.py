"""Group-propagated replay (Section 4.1) through the C boundary against the oracle's group_replay: the states and conv
states of every layer of a group rebuilt from the group-entry anchors alone, and the rows handed from layer to layer.

Tolerances.  Layer 0 of a group sees exactly the oracle's input, so its states obey the single-layer bounds.  The rows
it hands on are bf16(r + increment): the CUDA path forms the increment (y W_o^T, then the MLP's) from bf16 / fp16
operands with fp32 sums -- gate, gated output and hidden rows are stored in bf16, q, k, the chunk states and the
pseudo-values in fp16 -- so the increment carries a relative error of about 2^-8 of its RMS, the same size as half a
bf16 step of the row entry it is added to.  The rounded sum therefore lands on a neighbouring bf16 value for a large
part of the entries (about a third without an MLP, half with one; measured), and a second rounding after the MLP can
move it a step further.  Allowed per entry after hand-over j: one bf16 step of the entry plus 2^-5 (j + 1) of the
row's RMS; in aggregate the RMS difference must stay below 2^-7 (j + 1) of the row's RMS, and at least a quarter of the
entries must be bit-identical.  Layer l >= 1 then reads rows whose relative RMS perturbation is about 2^-8 per
hand-over; the state is linear in v, so that passes to the state undiminished (measured 4..6e-3 per hand-over):
tolerance = the single-layer bound + 1e-2 l.  Its conv state is the bf16 image of a projection of those rows and
gets the per-entry rule of the rows."""

import numpy as np
import pytest
import torch

import parity_util as U
from oracle import gdn_replay_oracle as orc
from paper_2609_33477_b200 import binding, synth
from paper_2609_33477_b200 import build as sr_build

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    sr_build.build()
    binding.load()


def _bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def _close_rows(got_bits, ref_bits, what, hops, aggregate=True):
    """Per-entry and aggregate closeness of bf16 rows `hops` hand-overs into a group; returns the identical fraction."""
    a, b = orc.bf16_bits_to_f64(got_bits), orc.bf16_bits_to_f64(ref_bits)
    if not b.size:
        return 1.0
    assert np.all(np.isfinite(a)), what
    rms = np.sqrt(np.mean(b * b, axis=-1, keepdims=True))
    step = np.where(b != 0, 2.0 ** (np.floor(np.log2(np.abs(np.where(b != 0, b, 1.0)))) - 7), 0.0)
    ok = np.abs(a - b) <= step + rms * 2.0 ** -5 * hops
    assert ok.all(), f"{what}: {np.count_nonzero(~ok)} entries off, worst {np.abs(a - b)[~ok].max():.3e}"
    if aggregate:
        rel = np.sqrt(np.mean((a - b) ** 2)) / np.sqrt(np.mean(b * b))
        assert rel <= 2.0 ** -7 * hops, f"{what}: relative RMS difference {rel:.3e}"
    return float((got_bits == ref_bits).mean())


def _strict_conv(tail_gpu, tail_ref):
    """The single-layer rule: one bf16 step at most (entries next to zero: 1e-5 absolute), nearly all identical."""
    dist = U.bf16_ulp_distance(tail_gpu, tail_ref)
    a, b = orc.bf16_bits_to_f64(tail_gpu), orc.bf16_bits_to_f64(tail_ref)
    assert ((dist <= 1) | (np.abs(a - b) <= 1e-5)).all() and (dist > 0).mean() <= 0.02


def _oracle_group(wl, i, first=0, n=None):
    s = wl.spec
    n = s.n_layers - first if n is None else n
    pl = wl.layer_to_pool[first]
    R = int(wl.replay_lens[i].item())
    pages = wl.page_table[i, : -(-R // 64)].cpu().tolist()
    got = synth.fetch_pages(wl, pages, pl)
    rows = np.concatenate([orc.bf16_bits_to_f64(got[(p, pl)]) for p in pages])[:R] if R else np.zeros((0, s.d_model))
    layers = [synth.block_arrays(wl.layers[l], wl.blocks[l]) for l in range(first, first + n)]
    return orc.group_replay(rows, layers, return_rows=True, n_k_heads=s.n_k_heads, n_v_heads=s.n_v_heads, d_k=s.d_k, d_v=s.d_v)


@pytest.mark.parametrize("name", ["group_small", "group_128", "group_wide"])
def test_group_states_and_handed_rows_match_the_oracle(name):
    wl = synth.build_workload(name, device="cuda")
    s = wl.spec
    rep = binding.Replayer(wl)
    st, rows = rep.replay_group_states(debug_rows=True)
    torch.cuda.synchronize()
    assert st == 0 and rep.group_device_status() == 0
    lens = wl.replay_lens.cpu().tolist()
    slot0 = 0
    same = []
    for i, R in enumerate(lens):
        res, handed = _oracle_group(wl, i)
        for l, (S_ref, tail_ref) in enumerate(res):
            S_gpu = rep.out_ssm[i, l].cpu().numpy()
            assert np.all(np.isfinite(S_gpu))
            err = U.rel_frob_per_head(S_gpu, S_ref)
            tol = U.REL_FROB_TOL + 1e-2 * l
            assert err <= tol, f"{name} request {i} layer {l}: rel Frobenius {err:.3e} > {tol}"
            tail_gpu = _bits(rep.out_conv[i, l])
            if l == 0:
                _strict_conv(tail_gpu, tail_ref)
            else:
                _close_rows(tail_gpu.T, tail_ref.T, f"{name} request {i} layer {l} conv state", hops=l, aggregate=False)
        for j, ref_bits in enumerate(handed):
            got = _bits(rows[j, slot0 * 64: slot0 * 64 + R])
            same.append(_close_rows(got, ref_bits, f"{name} request {i} rows after layer {j}", hops=j + 1))
        slot0 += -(-R // 64)
    assert np.min(same) > 0.25          # a good part of the handed entries is bit-identical


def test_a_group_of_one_layer_and_the_prefix_of_a_longer_group_agree():
    """Layer j's states do not depend on how many layers follow it in the group (same kernels, same order)."""
    wl = synth.build_workload("group_small", device="cuda")
    rep = binding.Replayer(wl)
    rep.replay_group_states()
    torch.cuda.synchronize()
    full_ssm, full_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    rep.replay_group_states(first_layer=0, n_group_layers=2)
    torch.cuda.synchronize()
    assert torch.equal(rep.out_ssm[:, :2], full_ssm[:, :2]) and torch.equal(rep.out_conv[:, :2], full_conv[:, :2])
    assert not rep.out_ssm[:, 2].any()                      # the third layer was not touched
    assert rep.last_launch_count() > 0
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    rep.replay_group_states(first_layer=0, n_group_layers=1)    # a group of one: no block kernels at all
    torch.cuda.synchronize()
    assert rep.last_launch_count() == 6                     # packing + row norm, projection, conv state, chunk-local, chain
    assert torch.equal(rep.out_ssm[:, 0], full_ssm[:, 0]) and torch.equal(rep.out_conv[:, 0], full_conv[:, 0])
    assert not rep.out_ssm[:, 1:].any()
    # a group must start at a layer that has anchors: layer 1 of this workload has none
    assert rep.replay_group_states(first_layer=1, n_group_layers=2, check=False) == binding.SR_ERR_INVALID_ARG
    assert rep.replay_group_states(first_layer=0, n_group_layers=4, check=False) == binding.SR_ERR_INVALID_ARG


def test_group_at_the_benchmarked_size_matches_the_oracle_on_sampled_requests():
    """`group3_4b` as `bench.py --config group3_4b` runs it (three layers of the 4B geometry with MLPs, eight 512-row
    requests, 4096 packed rows): two requests are replayed by the oracle and every layer of the group is compared."""
    wl = synth.build_workload("group3_4b", device="cuda")
    rep = binding.Replayer(wl)
    st, rows = rep.replay_group_states(debug_rows=True)
    torch.cuda.synchronize()
    assert st == 0 and rep.group_device_status() == 0
    lens = wl.replay_lens.cpu().tolist()
    for i in (0, 5):
        res, handed = _oracle_group(wl, i)
        slot0 = sum(-(-r // 64) for r in lens[:i])
        for l, (S_ref, tail_ref) in enumerate(res):
            err = U.rel_frob_per_head(rep.out_ssm[i, l].cpu().numpy(), S_ref)
            assert err <= U.REL_FROB_TOL + 1e-2 * l, f"request {i} layer {l}: rel Frobenius {err:.3e}"
            tail_gpu = _bits(rep.out_conv[i, l])
            if l == 0:
                _strict_conv(tail_gpu, tail_ref)
            else:
                _close_rows(tail_gpu.T, tail_ref.T, f"request {i} layer {l} conv state", hops=l, aggregate=False)
        for j, ref_bits in enumerate(handed):
            _close_rows(_bits(rows[j, slot0 * 64: slot0 * 64 + lens[i]]), ref_bits, f"request {i} rows after layer {j}", hops=j + 1)


def _draw_group(seed):
    r = np.random.RandomState(2000 + seed)
    d_k = d_v = int(r.choice([64, 128]))
    h_k = int(r.randint(1, 4))
    h_v = h_k * int(r.randint(1, 4))
    n_layers = int(r.randint(2, 4))
    n_req = int(r.randint(1, 5))
    lens = tuple(int(x) for x in r.choice([0, 1, 3, 63, 64, 65, 129, 200, 257], size=n_req))
    d_ff = tuple(int(64 * r.randint(0, 9)) for _ in range(n_layers))
    return synth.WorkloadSpec(name=f"random_group_{seed}", n_layers=n_layers, d_model=int(64 * r.randint(2, 11)), n_k_heads=h_k,
                              n_v_heads=h_v, d_k=d_k, d_v=d_v, n_requests=n_req, replay=("list", lens), group=True, d_ff=d_ff,
                              paging=["shuffled", "identity"][r.randint(2)])


@pytest.mark.parametrize("seed", range(8))
def test_random_groups_match_the_oracle(seed):
    """Seeded random widths, head counts, group sizes, MLP widths and ragged batches, same comparison as above."""
    spec = _draw_group(seed)
    wl = synth.build_workload(spec, device="cuda", seed=seed)
    rep = binding.Replayer(wl)
    st, rows = rep.replay_group_states(debug_rows=True)
    torch.cuda.synchronize()
    assert st == 0 and rep.group_device_status() == 0
    slot0 = 0
    for i, R in enumerate(wl.replay_lens.cpu().tolist()):
        res, handed = _oracle_group(wl, i)
        for l, (S_ref, tail_ref) in enumerate(res):
            S_gpu = rep.out_ssm[i, l].cpu().numpy()
            assert np.all(np.isfinite(S_gpu))
            err = U.rel_frob_per_head(S_gpu, S_ref)
            assert err <= U.REL_FROB_TOL + 1e-2 * l, f"{spec} request {i} layer {l}: rel Frobenius {err:.3e}"
            tail_gpu = _bits(rep.out_conv[i, l])
            if l == 0:
                _strict_conv(tail_gpu, tail_ref)
            else:
                _close_rows(tail_gpu.T, tail_ref.T, f"request {i} layer {l} conv state", hops=l, aggregate=False)
        for j, ref_bits in enumerate(handed):
            _close_rows(_bits(rows[j, slot0 * 64: slot0 * 64 + R]), ref_bits, f"request {i} rows after layer {j}", hops=j + 1)
        slot0 += -(-R // 64)


def test_the_group_call_can_be_captured_in_a_cuda_graph():
    """No host synchronisation, no allocation: one captured graph replays the whole group call bit for bit."""
    wl = synth.build_workload("group_small", device="cuda")
    rep = binding.Replayer(wl)
    rep.replay_group_states()                        # one-time kernel attributes and the workspace, outside the capture
    torch.cuda.synchronize()
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        rep.replay_group_states(stream=torch.cuda.current_stream())
    graph.replay()
    torch.cuda.synchronize()
    assert rep.group_device_status() == 0
    assert torch.equal(rep.out_ssm, ref_ssm) and torch.equal(rep.out_conv, ref_conv)


def test_sentinel_requests_of_a_group_call_are_skipped_and_leave_the_others_unchanged():
    """Destination slot -1 (Section 5.2, padded batches): nothing is written for that request, and the other requests
    get the same bits as without it (rows of different requests never mix)."""
    wl = synth.build_workload("group_small", device="cuda")
    rep = binding.Replayer(wl)
    rep.replay_group_states()
    torch.cuda.synchronize()
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    slots = torch.tensor([0, 1, -1, 3], dtype=torch.int32, device="cuda")
    rep2 = binding.Replayer(wl, state_slots=slots, n_slots=4)
    rep2.out_ssm.fill_(7.0)
    rep2.out_conv.fill_(7.0)
    rep2.replay_group_states()
    torch.cuda.synchronize()
    assert rep2.group_device_status() == 0
    for i in (0, 1, 3):
        assert torch.equal(rep2.out_ssm[i], ref_ssm[i]) and torch.equal(rep2.out_conv[i], ref_conv[i])
    assert (rep2.out_ssm[2] == 7.0).all() and (rep2.out_conv[2] == 7.0).all()


def test_group_call_under_device_side_bounds_checks_raises_no_alarm():
    """SR_DEBUG_CHECK_BOUNDS: every table-driven index is tested before the access; a healthy call sets no bit and
    gives the same bits as without the checks."""
    wl = synth.build_workload("group_small", device="cuda")
    rep = binding.Replayer(wl)
    rep.replay_group_states()
    torch.cuda.synchronize()
    chk = binding.Replayer(wl, debug_flags=binding.SR_DEBUG_CHECK_BOUNDS)
    chk.replay_group_states()
    torch.cuda.synchronize()
    assert chk.group_device_status() == 0
    assert torch.equal(chk.out_ssm, rep.out_ssm) and torch.equal(chk.out_conv, rep.out_conv)



def test_several_groups_in_one_call_match_the_oracle_and_the_single_group_calls():
    """sr_replay_groups_states: the groups of a hybrid model side by side, each from its own anchors (Section 4.1)."""
    wl = synth.build_workload("groups_small", device="cuda")
    s = wl.spec
    assert wl.groups == [(0, 3), (3, 3), (6, 1)] and wl.anchor_pool.shape[1] == 3
    rep = binding.Replayer(wl)
    rep.replay_groups_states()
    torch.cuda.synchronize()
    assert rep.group_device_status() == 0
    all_ssm, all_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    for i in range(s.n_requests):
        for first, n in wl.groups:
            res, _ = _oracle_group(wl, i, first, n)
            for j, (S_ref, tail_ref) in enumerate(res):
                err = U.rel_frob_per_head(all_ssm[i, first + j].cpu().numpy(), S_ref)
                assert err <= U.REL_FROB_TOL + 1e-2 * j, f"request {i} group at {first} layer {j}: {err:.3e}"
                if j == 0:
                    _strict_conv(_bits(all_conv[i, first]), tail_ref)
    # the same bits one group at a time, and with the least workspace (groups one after the other)
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    for first, n in wl.groups:
        rep.replay_group_states(first_layer=first, n_group_layers=n)
    torch.cuda.synchronize()
    assert torch.equal(rep.out_ssm, all_ssm) and torch.equal(rep.out_conv, all_conv)
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    rep.replay_groups_states(min_workspace=True)
    torch.cuda.synchronize()
    assert torch.equal(rep.out_ssm, all_ssm) and torch.equal(rep.out_conv, all_conv)
    # overlapping groups are refused on the host
    assert rep.replay_groups_states(groups=[(0, 3), (2, 2)], check=False) == binding.SR_ERR_INVALID_ARG


def test_the_multi_group_call_can_be_captured_in_a_cuda_graph():
    """The side streams fork from and join the capturing stream, so the whole call becomes one graph."""
    wl = synth.build_workload("groups_small", device="cuda")
    rep = binding.Replayer(wl)
    rep.replay_groups_states()                       # creates the side streams and the workspace, outside the capture
    torch.cuda.synchronize()
    ref_ssm, ref_conv = rep.out_ssm.clone(), rep.out_conv.clone()
    rep.out_ssm.zero_()
    rep.out_conv.zero_()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        rep.replay_groups_states(stream=torch.cuda.current_stream())
    graph.replay()
    torch.cuda.synchronize()
    assert rep.group_device_status() == 0
    assert torch.equal(rep.out_ssm, ref_ssm) and torch.equal(rep.out_conv, ref_conv)
