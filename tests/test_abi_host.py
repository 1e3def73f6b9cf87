"""Host side of the C boundary: the library loads, exports every declared symbol, checks its
arguments before launching anything, and reports the state sizes the paper prints.
No compute call is made here (no GPU needed)."""

import ctypes as C
import os
import re

import pytest

from paper_2609_33477_b200 import binding as B
from paper_2609_33477_b200 import build as sr_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    sr_build.build()
    return B.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sr_replay.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sr_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert "sr_replay_states" in names and "sr_create" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names
    assert b"sm_100a" in lib.sr_version()


def _desc(**kw):
    d = dict(n_layers=2, d_model=512, n_k_heads=4, n_v_heads=4, d_k=128, d_v=128, conv_width=4, page_rows=64,
             weight_format=B.SR_W_BF16, conv_activation=B.SR_CONV_SILU, l2_eps=1e-6)
    d.update(kw)
    return B.sr_model_desc(**d)


def test_state_sizes_reproduce_appendix_a(lib):
    rows = [ln.split() for ln in open(os.path.join(ROOT, "tests", "golden", "appendix_a_state_sizes.txt"))
            if ln.strip() and not ln.startswith("#")]
    for name, L, d, Hk, Hv, dk, dv, Cc, B_rec, B_conv, _ in rows:
        ctx = B.sr_create(_desc(n_layers=int(L), d_model=int(d), n_k_heads=int(Hk), n_v_heads=int(Hv),
                                d_k=int(dk), d_v=int(dv)))
        assert B.sr_ssm_bytes_per_layer(ctx) == int(B_rec), name
        assert B.sr_conv_bytes_per_layer(ctx) == int(B_conv), name
        B.sr_destroy(ctx)


def test_create_rejects_inconsistent_geometry(lib):
    for bad in (dict(n_layers=0), dict(d_model=-1), dict(n_v_heads=6), dict(weight_format=7),
                dict(conv_activation=3), dict(l2_eps=-1.0), dict(conv_width=1)):
        ctx = C.c_void_p()
        assert lib.sr_create(C.byref(_desc(**bad)), C.byref(ctx)) == B.SR_ERR_INVALID_ARG, bad
        assert not ctx.value
    assert lib.sr_create(None, C.byref(C.c_void_p())) == B.SR_ERR_INVALID_ARG
    lib.sr_destroy(None)


def test_geometry_without_a_kernel_is_refused_not_emulated(lib):
    ctx = B.sr_create(_desc(d_k=80, d_v=160))          # sizes can be asked, replay cannot
    table = B.sr_page_table(None, None, 1, 1, 64, 64)
    n = C.c_size_t()
    assert lib.sr_workspace_bytes(ctx, C.byref(table), C.byref(n)) == B.SR_ERR_UNSUPPORTED_SHAPE
    B.sr_destroy(ctx)


def test_workspace_query_and_argument_checks_happen_before_any_launch(lib):
    ctx = B.sr_create(_desc())
    table = B.sr_page_table(None, None, 3, 4, 256, 600)
    ws = B.sr_workspace_bytes(ctx, table)
    # at least the projection's hand-over to the scan: (600/64 + 3 -> 12 slots) * 64 rows * (512 + 512) fp16 values
    assert ws >= 12 * 64 * 1024 * 2 and ws % 256 == 0
    bigger = B.sr_page_table(None, None, 3, 4, 256, 768)
    assert B.sr_workspace_bytes(ctx, bigger) >= ws
    bad = B.sr_page_table(None, None, 3, 4, 257, 600)        # max_replay_len beyond the table's pages
    n = C.c_size_t()
    assert lib.sr_workspace_bytes(ctx, C.byref(bad), C.byref(n)) == B.SR_ERR_INVALID_ARG
    neg = B.sr_page_table(None, None, -1, 4, 256, 600)
    assert lib.sr_workspace_bytes(ctx, C.byref(neg), C.byref(n)) == B.SR_ERR_INVALID_ARG

    # null pointers are caught on the host: nothing is launched, so this is safe without a GPU
    pool = B.sr_anchor_pool()
    out = B.sr_out()
    weights = (B.sr_layer_weights * 2)()
    mask = (C.c_uint8 * 2)(1, 1)
    st = lib.sr_replay_states(ctx, C.byref(pool), C.byref(table), None, mask, weights, C.byref(out), C.byref(out),
                              None, 0, None)
    assert st == B.SR_ERR_INVALID_ARG
    st = lib.sr_debug_gather(ctx, C.byref(pool), C.byref(table), None, 0, None, 0, None, 0, None)
    assert st == B.SR_ERR_INVALID_ARG
    assert lib.sr_device_status(ctx, None, None, None) == B.SR_ERR_INVALID_ARG
    assert B.sr_last_launch_count(ctx) == 0
    # a null context is an invalid argument for every entry, also where states to continue from are given
    st = lib.sr_replay_states_from(None, C.byref(pool), C.byref(table), None, mask, weights, C.byref(out), C.byref(out),
                                   C.byref(out), C.byref(out), None, 0, None)
    assert st == B.SR_ERR_INVALID_ARG
    st = lib.sr_replay_states(None, C.byref(pool), C.byref(table), None, mask, weights, C.byref(out), C.byref(out),
                              None, 0, None)
    assert st == B.SR_ERR_INVALID_ARG
    B.sr_destroy(ctx)


def test_more_requests_than_grid_rows_are_refused(lib):
    ctx = B.sr_create(_desc())
    n = C.c_size_t()
    assert lib.sr_workspace_bytes(ctx, C.byref(B.sr_page_table(None, None, 65535, 0, 0, 0)), C.byref(n)) == B.SR_OK
    assert lib.sr_workspace_bytes(ctx, C.byref(B.sr_page_table(None, None, 65536, 0, 0, 0)), C.byref(n)) == \
        B.SR_ERR_UNSUPPORTED_SHAPE
    B.sr_destroy(ctx)


def test_batches_beyond_the_slot_limit_are_refused(lib):
    ctx = B.sr_create(_desc())
    n = C.c_size_t()
    ok = B.sr_page_table(None, None, 100, 700, 700 * 64, 65000 * 64)
    big = B.sr_page_table(None, None, 100, 700, 700 * 64, 65536 * 64)
    assert lib.sr_workspace_bytes(ctx, C.byref(ok), C.byref(n)) == B.SR_OK
    assert lib.sr_workspace_bytes(ctx, C.byref(big), C.byref(n)) == B.SR_ERR_UNSUPPORTED_SHAPE
    B.sr_destroy(ctx)


def test_status_strings(lib):
    assert lib.sr_status_string(0) == b"SR_OK"
    assert lib.sr_status_string(B.SR_ERR_WORKSPACE) == b"SR_ERR_WORKSPACE"
    assert lib.sr_status_string(99) == b"SR_ERR_UNKNOWN"


def test_group_replay_checks_its_arguments_on_the_host(lib):
    """Section 4.1 entry: geometry, weight format, group range and null pointers are refused before any launch."""
    n = C.c_size_t()
    table = B.sr_page_table(None, None, 3, 4, 256, 600)
    ctx = B.sr_create(_desc())
    assert lib.sr_group_workspace_bytes(None, C.byref(table), 0, C.byref(n)) == B.SR_ERR_INVALID_ARG
    assert lib.sr_group_workspace_bytes(ctx, C.byref(table), -64, C.byref(n)) == B.SR_ERR_INVALID_ARG
    plain = B.sr_group_workspace_bytes(ctx, table, 0)
    wide = B.sr_group_workspace_bytes(ctx, table, 1024)
    assert wide - plain >= 12 * 64 * 1024 * 2 and plain > B.sr_workspace_bytes_min(ctx, table)   # the MLP's hidden rows
    pool, out = B.sr_anchor_pool(), B.sr_out()
    weights, blocks = (B.sr_layer_weights * 2)(), (B.sr_block_weights * 2)()
    args = (C.byref(pool), C.byref(table), None)
    tail = (weights, blocks, C.c_float(1e-6), C.byref(out), C.byref(out), None, None, 0, None)
    assert lib.sr_replay_group_states(ctx, *args, 0, 2, *tail) == B.SR_ERR_INVALID_ARG      # null pointers
    assert lib.sr_replay_group_states(None, *args, 0, 2, *tail) == B.SR_ERR_INVALID_ARG
    B.sr_destroy(ctx)
    fp8 = B.sr_create(_desc(weight_format=B.SR_W_E4M3_BLOCK128))       # block-scaled weights: single-layer replay only
    assert lib.sr_group_workspace_bytes(fp8, C.byref(table), 0, C.byref(n)) == B.SR_ERR_UNSUPPORTED_SHAPE
    B.sr_destroy(fp8)
    odd = B.sr_create(_desc(d_k=96, d_v=192, n_k_heads=2, n_v_heads=2))   # replayable, but no per-token output kernel
    assert lib.sr_workspace_bytes(odd, C.byref(table), C.byref(n)) == B.SR_OK
    assert lib.sr_group_workspace_bytes(odd, C.byref(table), 0, C.byref(n)) == B.SR_ERR_UNSUPPORTED_SHAPE
    B.sr_destroy(odd)


def test_recommended_workspace_holds_a_block_per_layer_in_flight(lib):
    """sr_workspace_bytes = the tables + N blocks of per-layer hand-over buffers, N the largest of 32, 24, 16, 8, 4, 2, 1
    that the model has layers for and that stays within 1 GiB; sr_workspace_bytes_min = the tables + one block."""
    table = B.sr_page_table(None, None, 1, 8, 512, 512)            # one hit of 512 anchors
    sizes = {}
    for n_layers in (1, 2, 3, 8, 23, 24, 31, 32, 48):
        ctx = B.sr_create(_desc(n_layers=n_layers))
        one, rec = B.sr_workspace_bytes_min(ctx, table), B.sr_workspace_bytes(ctx, table)
        sizes[n_layers] = (one, rec)
        B.sr_destroy(ctx)
    one = sizes[1][0]
    assert sizes[1][1] == one
    block = sizes[2][1] - one                                      # two blocks - one block
    assert block > 0 and all(s[0] == one for s in sizes.values())
    expect = {1: 1, 2: 2, 3: 2, 8: 8, 23: 16, 24: 24, 31: 24, 32: 32, 48: 32}
    for n_layers, blocks in expect.items():
        assert sizes[n_layers][1] == one + (blocks - 1) * block, n_layers
    # a batch whose blocks would pass 1 GiB together gets fewer of them
    big = B.sr_page_table(None, None, 64, 128, 8192, 64 * 8192)
    ctx = B.sr_create(_desc(n_layers=32, d_model=5120, n_k_heads=16, n_v_heads=32))
    one_big, rec_big = B.sr_workspace_bytes_min(ctx, big), B.sr_workspace_bytes(ctx, big)
    assert rec_big == one_big and one_big > (1 << 30)
    B.sr_destroy(ctx)
