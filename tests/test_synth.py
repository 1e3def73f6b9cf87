"""The seeded input generators: determinism, shapes and page-table structure."""

import numpy as np
import torch

from paper_2609_33477_b200 import synth


def test_same_seed_same_bytes_and_other_seed_differs():
    a = synth.build_workload("ragged_small", seed=0)
    b = synth.build_workload("ragged_small", seed=0)
    c = synth.build_workload("ragged_small", seed=1)
    assert torch.equal(a.anchor_pool.view(torch.int16), b.anchor_pool.view(torch.int16))
    assert torch.equal(a.page_table, b.page_table)
    assert torch.equal(a.layers[0].w_qkv.view(torch.int16), b.layers[0].w_qkv.view(torch.int16))
    assert not torch.equal(a.anchor_pool.view(torch.int16), c.anchor_pool.view(torch.int16))


def test_shapes_masks_and_pool_layers():
    wl = synth.build_workload("ragged_small")
    s = wl.spec
    assert wl.layer_mask == [1, 0, 1] and wl.layer_to_pool == [0, -1, 1]
    assert wl.layers[1] is None
    assert wl.anchor_pool.shape[1:] == (2, synth.PAGE_ROWS, s.d_model)
    assert wl.layers[0].w_qkv.shape == (s.conv_channels, s.d_model)
    assert wl.layers[0].w_ab.shape == (2 * s.n_v_heads, s.d_model)
    assert wl.layers[0].conv_w.shape == (s.conv_channels, 4)
    assert wl.replay_lens.tolist() == [0, 1, 3, 64, 65, 200]
    assert wl.total_rows == 333 and wl.layer_tokens == 666


def test_shuffled_tables_are_a_partition_of_the_pool():
    wl = synth.build_workload("ragged_d64")
    used = []
    for i, R in enumerate(wl.replay_lens.tolist()):
        n = -(-R // synth.PAGE_ROWS)
        row = wl.page_table[i].tolist()
        assert all(p >= 0 for p in row[:n]) and all(p == -1 for p in row[n:])
        used += row[:n]
    assert sorted(used) == list(range(wl.n_phys_pages))


def test_trunk_tables_share_pages_and_cover_the_pool_exactly():
    wl = synth.build_workload("trunks_small")
    used = []
    for i, R in enumerate(wl.replay_lens.tolist()):
        assert R % synth.PAGE_ROWS == 0 and R > 0
        used += wl.page_table[i, : R // synth.PAGE_ROWS].tolist()
    assert set(used) == set(range(wl.n_phys_pages))
    assert len(used) > len(set(used))          # some windows overlap on their trunk


def test_fp8_weights_are_codes_with_block_scales():
    wl = synth.build_workload("fp8_small")
    p = wl.layers[0]
    assert p.w_qkv.dtype == torch.uint8 and p.w_qkv_scale.dtype == torch.float32
    assert p.w_qkv_scale.shape == ((wl.spec.conv_channels + 127) // 128, wl.spec.d_model // 128)
    assert int(((p.w_qkv & 0x7F) == 0x7F).sum()) == 0      # no NaN codes
    arr = synth.layer_arrays(p)
    assert arr["w_qkv_codes"].dtype == np.uint8 and "w_qkv_bits" not in arr


def test_benchmark_specs_match_their_stated_shapes():
    s = synth.SPECS
    assert (s["cfg0"].d_model, s["cfg0"].n_v_heads, s["cfg0"].d_k, s["cfg0"].replay) == (256, 2, 64, ("fixed", 256))
    assert (s["cfg1"].d_model, s["cfg1"].n_requests, s["cfg1"].replay) == (2560, 8, ("fixed", 2048))
    assert (s["cfg2"].n_layers, s["cfg2"].d_model, s["cfg2"].conv_channels) == (48, 5120, 12288)
    assert s["cfg3"].layer_mask == "even" and s["cfg3"].n_requests == 64
    assert s["cfg4"].weight_format == "e4m3_block128" and abs(s["cfg4"].decay_scale - 0.03) < 1e-12


def test_group_workloads_carry_block_weights_and_feed_the_oracle():
    """Group workloads (Section 4.1): one pool layer holding the group-entry rows, every layer with mixer and block
    weights; the fp64 images handed to the oracle are exact and the oracle runs on them."""
    import numpy as np
    from oracle import gdn_replay_oracle as orc
    wl = synth.build_workload("group_small", device="cpu")
    s = wl.spec
    assert wl.anchor_pool.shape[1] == 1 and wl.layer_to_pool == [0, -1, -1] and wl.layer_mask == [1, 1, 1]
    assert len(wl.blocks) == s.n_layers and all(p is not None for p in wl.layers)
    assert [b.w_gate is not None for b in wl.blocks] == [False, True, False]          # d_ff = (0, 192, 0)
    assert wl.blocks[1].w_gate.shape == (192, s.d_model) and wl.blocks[1].w_down.shape == (s.d_model, 192)
    layers = [synth.block_arrays(wl.layers[l], wl.blocks[l]) for l in range(s.n_layers)]
    assert np.array_equal(layers[0]["w_z"].astype(np.float32), wl.blocks[0].w_z.float().numpy())   # bf16 -> fp64 is exact
    assert "w_gate" in layers[1] and "w_gate" not in layers[0]
    i = 1
    R = int(wl.replay_lens[i])
    pages = wl.page_table[i, : -(-R // 64)].tolist()
    got = synth.fetch_pages(wl, pages, 0)
    rows = np.concatenate([orc.bf16_bits_to_f64(got[(p, 0)]) for p in pages])[:R]
    res, handed = orc.group_replay(rows, layers, return_rows=True, n_k_heads=s.n_k_heads, n_v_heads=s.n_v_heads, d_k=s.d_k, d_v=s.d_v)
    assert len(res) == 3 and len(handed) == 2 and handed[0].shape == (R, s.d_model)
    assert all(np.all(np.isfinite(S)) and S.shape == (s.n_v_heads, s.d_k, s.d_v) for S, _ in res)
    # same seed, same bytes
    wl2 = synth.build_workload("group_small", device="cpu")
    assert all(torch.equal(a.w_o, b.w_o) and torch.equal(a.norm_w, b.norm_w) for a, b in zip(wl.blocks, wl2.blocks))
