"""Seeded random geometries, widths, batch shapes and weight formats through the C boundary against the oracle: every
(request, rebuilt layer) of every drawn workload, the same comparison as the named parity cases (state within 2e-3
relative Frobenius error per head, conv state within one bf16 step and nearly all identical)."""

import numpy as np
import pytest
import torch

import parity_util as U
from paper_2609_33477_b200 import binding, synth
from paper_2609_33477_b200 import build as sr_build

pytestmark = pytest.mark.gpu

GEOMETRIES = [(64, 64), (128, 128), (96, 192), (64, 128), (128, 64), (96, 96), (128, 256)]   # (d_k, d_v)


@pytest.fixture(scope="module", autouse=True)
def _built():
    sr_build.build()
    binding.load()


def _draw(seed):
    r = np.random.RandomState(1000 + seed)
    d_k, d_v = GEOMETRIES[r.randint(len(GEOMETRIES))]
    h_k = int(r.randint(1, 4))
    h_v = h_k * int(r.randint(1, 4))
    fmt = ["bf16", "bf16", "e4m3_block128", "w8a8"][r.randint(4)]
    if fmt == "bf16":
        d = int(64 * r.randint(2, 11))                    # 128 .. 640, any multiple of 64
    else:
        d = int(128 * r.randint(1, 6))                    # block-scaled weights: multiples of 128
        # the block-scaled kernels want whole 128-channel tiles of k | v
        while (h_k * d_k) % 128 or (h_k * d_k + h_v * d_v) % 128:
            h_k += 1
            h_v = h_k * max(1, h_v // max(1, h_k - 1))
    n_req = int(r.randint(1, 6))
    lens = tuple(int(x) for x in r.choice([0, 1, 2, 3, 5, 63, 64, 65, 127, 129, 200, 257, 321], size=n_req))
    n_layers = int(r.randint(1, 4))
    return synth.WorkloadSpec(
        name=f"random_{seed}", n_layers=n_layers, d_model=d, n_k_heads=h_k, n_v_heads=h_v, d_k=d_k, d_v=d_v,
        n_requests=n_req, replay=("list", lens), paging=["shuffled", "identity"][r.randint(2)],
        layer_mask=["all", "even"][r.randint(2)], weight_format="bf16" if fmt == "bf16" else "e4m3_block128",
        act_quant="e4m3_1x128" if fmt == "w8a8" else "none", decay_scale=float(r.choice([0.03, 0.1, 0.5])))


@pytest.mark.parametrize("seed", range(16))
def test_random_workload_matches_the_oracle(seed):
    spec = _draw(seed)
    wl = synth.build_workload(spec, device="cuda", seed=seed)
    try:
        rep = binding.Replayer(wl)
    except binding.SrError as e:                           # a geometry no kernel serves is refused, never emulated
        assert e.status == binding.SR_ERR_UNSUPPORTED_SHAPE
        pytest.skip(f"{spec}: refused as unsupported")
    rep.replay_states()
    torch.cuda.synchronize()
    assert rep.device_status() == 0
    for i in range(spec.n_requests):
        for l, m in enumerate(wl.layer_mask):
            if m:
                U.check_request_layer(rep, wl, i, l)
    rep.close()
