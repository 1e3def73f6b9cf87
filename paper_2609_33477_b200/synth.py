"""Seeded synthetic replay workloads (inputs only -- none of the method's arithmetic).

Every tensor the replay path reads is produced here from a seed: the paged bf16
anchor sidecar, the per-request page tables and replay lengths, the layer mask and
the per-layer projection / conv / gate parameters.  The same objects feed the CUDA
path (through ``binding``) and, read back as raw bytes, the CPU oracle's tests, so
both sides always see identical inputs.  Random numbers come from ``torch``'s seeded
generators and rounding to the storage types (bf16, e4m3) is done by ``torch``'s own
casts; nothing here projects, convolves, normalises or scans.

The five named workloads ``cfg0`` .. ``cfg4`` follow the benchmark configurations of
this build; they stand in for the hidden states and serving traces the paper
measures on (Section 7.1), which need trained models and are not reproduced.
Anchors are iid N(0,1) rounded to bf16, projection weights iid N(0, 1/d_model)
(variance), conv taps iid N(0, 1/w).  With that scaling the gate pre-activations are
close to N(0,1), so the decay ``exp(-c * softplus(a))`` and write strength
``sigmoid(b)`` produced by the projection have the distribution the configurations
name (``c`` = ``decay_scale``).
"""

from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

PAGE_ROWS = 64  # rows of one anchor page = tokens of one KV page (Section 5.1)


@dataclasses.dataclass(frozen=True)
class WorkloadSpec:
    name: str
    n_layers: int
    d_model: int
    n_k_heads: int
    n_v_heads: int
    d_k: int
    d_v: int
    n_requests: int
    # ("fixed", R) | ("pages_uniform", lo_pages, hi_pages) | ("list", (R0, R1, ...))
    replay: Tuple
    paging: str = "shuffled"          # "identity" | "shuffled" | "trunks"
    layer_mask: str = "all"           # "all" | "even"
    weight_format: str = "bf16"       # "bf16" | "e4m3_block128"
    act_quant: str = "none"           # "none" | "e4m3_1x128" (W8A8: anchors quantised on the fly; e4m3 weights only)
    decay_scale: float = 0.1
    conv_width: int = 4
    recurrence: str = "gated_delta"   # "gated_delta" | "decay_only" (the two families of Section 2.1)
    n_trunks: int = 16                # "trunks" paging only
    trunk_pages: int = 256            # "trunks" paging only
    requests_per_trunk: int = 4       # "trunks" paging only
    # group-propagated replay (Section 4.1): all n_layers form ONE group of consecutive linear-attention layers whose
    # only anchors are the rows entering layer 0; every layer gets block weights, and an MLP d_ff[l] wide (0: none)
    group: bool = False
    d_ff: Tuple = ()
    group_size: int = 0               # layers per group (0: all n_layers are one group); anchors enter each group's first layer

    @property
    def conv_channels(self) -> int:
        return 2 * self.n_k_heads * self.d_k + self.n_v_heads * self.d_v


def _spec(name, L, d, H, dh, B, replay, **kw) -> WorkloadSpec:
    return WorkloadSpec(name=name, n_layers=L, d_model=d, n_k_heads=H, n_v_heads=H,
                        d_k=dh, d_v=dh, n_requests=B, replay=replay, **kw)


SPECS = {
    # The five benchmark configurations.
    "cfg0": _spec("cfg0", 1, 256, 2, 64, 1, ("fixed", 256), paging="identity"),
    "cfg1": _spec("cfg1", 1, 2560, 16, 128, 8, ("fixed", 2048)),
    "cfg2": _spec("cfg2", 48, 5120, 32, 128, 16, ("fixed", 4096)),
    "cfg3": _spec("cfg3", 24, 5120, 32, 128, 64, ("pages_uniform", 8, 128),
                  paging="trunks", layer_mask="even"),
    "cfg4": _spec("cfg4", 24, 5120, 32, 128, 32, ("fixed", 8192),
                  weight_format="e4m3_block128", decay_scale=0.03),
    # Reduced cases for parity tests: same structure, sizes a CPU finishes in seconds.
    "ragged_small": _spec("ragged_small", 3, 512, 4, 128, 6,
                          ("list", (0, 1, 3, 64, 65, 200)), layer_mask="even"),
    "ragged_d64": _spec("ragged_d64", 2, 256, 2, 64, 5, ("list", (4, 63, 127, 128, 321))),
    "trunks_small": _spec("trunks_small", 4, 512, 4, 128, 8, ("pages_uniform", 1, 6),
                          paging="trunks", layer_mask="even", n_trunks=2, trunk_pages=8),
    "fp8_small": _spec("fp8_small", 2, 512, 4, 128, 3, ("list", (130, 64, 257)),
                       weight_format="e4m3_block128", decay_scale=0.03),
    "cfg1_narrow": _spec("cfg1_narrow", 1, 1024, 4, 128, 4, ("fixed", 512)),
    # grouped value heads (H_v = 2 H_k, as in the paper's 4B-class model): value head h reads key head h // 2
    "grouped_small": WorkloadSpec(name="grouped_small", n_layers=2, d_model=512, n_k_heads=2, n_v_heads=4,
                                  d_k=128, d_v=128, n_requests=4, replay=("list", (130, 64, 257, 5))),
    # the other geometries of the paper's models (Appendix A): three value heads per key head; d_k = 96, d_v = 192
    "grouped3_small": WorkloadSpec(name="grouped3_small", n_layers=1, d_model=512, n_k_heads=2, n_v_heads=6,
                                   d_k=128, d_v=128, n_requests=3, replay=("list", (130, 64, 200))),
    "wide_v_small": WorkloadSpec(name="wide_v_small", n_layers=2, d_model=256, n_k_heads=2, n_v_heads=2,
                                 d_k=96, d_v=192, n_requests=4, replay=("list", (70, 0, 129, 5)), layer_mask="even"),
    # head geometry of the paper's three models (Appendix A table: 16/32 heads of 128; 16/48 heads of 128; 16/16
    # heads of 96/192), few layers, narrow d_model: parity cases
    "geom_16_32": WorkloadSpec(name="geom_16_32", n_layers=1, d_model=256, n_k_heads=16, n_v_heads=32, d_k=128, d_v=128,
                               n_requests=2, replay=("list", (130, 64))),
    "geom_16_48": WorkloadSpec(name="geom_16_48", n_layers=1, d_model=256, n_k_heads=16, n_v_heads=48, d_k=128, d_v=128,
                               n_requests=2, replay=("list", (70, 129))),
    "geom_96_192": WorkloadSpec(name="geom_96_192", n_layers=1, d_model=256, n_k_heads=3, n_v_heads=3, d_k=96, d_v=192,
                                n_requests=3, replay=("list", (200, 64, 321))),
    # many layers, a small batch: the layers of one call run side by side
    "layers_small": _spec("layers_small", 9, 512, 4, 128, 3, ("list", (130, 64, 257)), layer_mask="all"),
    # the per-head-decay family (no erase)
    "decay_only_small": _spec("decay_only_small", 2, 512, 4, 128, 4, ("list", (130, 64, 257, 5)), recurrence="decay_only"),
    "decay_only_d64": _spec("decay_only_d64", 1, 256, 2, 64, 3, ("list", (70, 128, 3)), recurrence="decay_only"),
    # more requests than the packing kernel has threads, many of them empty
    "many_requests": _spec("many_requests", 1, 512, 4, 128, 1500, ("pages_uniform", 0, 2)),
    # the ends of the decay range: alpha = 1 exactly (a pure delta rule), and alpha ~ 1e-3 per token (exp(g_i - g_j)
    # underflows inside a chunk)
    "decay_none": _spec("decay_none", 1, 512, 4, 128, 3, ("list", (130, 64, 300)), decay_scale=0.0),
    "decay_strong": _spec("decay_strong", 1, 512, 4, 128, 3, ("list", (130, 64, 300)), decay_scale=8.0),
    # One rebuilt layer and 8 requests of cfg3: the same kernels, tile shapes and per-unit traffic as
    # cfg3 in about 2 GB, small enough for a multi-pass profiler capture.
    "cfg3_slice": _spec("cfg3_slice", 2, 5120, 32, 128, 8, ("pages_uniform", 8, 128),
                        paging="trunks", layer_mask="even", n_trunks=2, trunk_pages=256),
    "cfg4_slice": _spec("cfg4_slice", 1, 5120, 32, 128, 4, ("fixed", 8192),
                        weight_format="e4m3_block128", decay_scale=0.03),
}
# The head geometry of the paper's three models (Appendix A table) at their own d_model, two layers, 8 requests of
# 2048 rows: bench lines for the widths the five configurations do not cover.
SPECS["model_4b"] = WorkloadSpec(name="model_4b", n_layers=2, d_model=2560, n_k_heads=16, n_v_heads=32, d_k=128,
                                 d_v=128, n_requests=8, replay=("fixed", 2048))
SPECS["model_27b"] = WorkloadSpec(name="model_27b", n_layers=2, d_model=5120, n_k_heads=16, n_v_heads=48, d_k=128,
                                  d_v=128, n_requests=8, replay=("fixed", 2048))
SPECS["model_7b_96_192"] = WorkloadSpec(name="model_7b_96_192", n_layers=2, d_model=3840, n_k_heads=30, n_v_heads=30,
                                        d_k=96, d_v=192, n_requests=8, replay=("fixed", 2048))
# The paper's own operating point (Section 6: at most 512 anchors per hit on the 4B model, 4096 packed anchors per
# batch): one hit, and eight simultaneous hits, all 24 linear layers of the 4B geometry.
SPECS["hit_512"] = WorkloadSpec(name="hit_512", n_layers=24, d_model=2560, n_k_heads=16, n_v_heads=32, d_k=128,
                                d_v=128, n_requests=1, replay=("fixed", 512))
SPECS["hits8_512"] = WorkloadSpec(name="hits8_512", n_layers=24, d_model=2560, n_k_heads=16, n_v_heads=32, d_k=128,
                                  d_v=128, n_requests=8, replay=("fixed", 512))
# W8A8: the block-scaled configuration with on-the-fly e4m3 activations, and reduced cases of it
SPECS["cfg4_w8a8"] = dataclasses.replace(SPECS["cfg4"], name="cfg4_w8a8", act_quant="e4m3_1x128")
SPECS["cfg4_w8a8_slice"] = dataclasses.replace(SPECS["cfg4_slice"], name="cfg4_w8a8_slice", act_quant="e4m3_1x128")
SPECS["w8a8_small"] = dataclasses.replace(SPECS["fp8_small"], name="w8a8_small", act_quant="e4m3_1x128")
SPECS["w8a8_ragged"] = _spec("w8a8_ragged", 2, 1024, 4, 128, 5, ("list", (0, 3, 65, 200, 700)), weight_format="e4m3_block128",
                             act_quant="e4m3_1x128", layer_mask="even")
# Group-propagated replay: small cases per supported geometry (ragged lengths, an empty request, MLP on some layers)
# and the 4B geometry with three linear-attention layers per group (the 3 : 1 hybrid pattern), eight 512-row hits.
SPECS["group_small"] = WorkloadSpec(name="group_small", n_layers=3, d_model=256, n_k_heads=2, n_v_heads=4, d_k=64, d_v=64,
                                    n_requests=4, replay=("list", (0, 70, 200, 130)), group=True, d_ff=(0, 192, 0))
SPECS["group_128"] = WorkloadSpec(name="group_128", n_layers=2, d_model=512, n_k_heads=2, n_v_heads=4, d_k=128, d_v=128,
                                  n_requests=2, replay=("list", (300, 64)), group=True, d_ff=(512, 0))
SPECS["group_wide"] = WorkloadSpec(name="group_wide", n_layers=2, d_model=640, n_k_heads=1, n_v_heads=3, d_k=128, d_v=128,
                                   n_requests=3, replay=("list", (129, 1, 257)), group=True, d_ff=(448, 0))
# a cache hit on a hybrid model: all its linear-attention groups at once (Section 4.1; the 3 : 1 pattern gives groups of
# three) -- 24 layers of the 4B geometry in eight groups, MLPs behind every layer, one 512-anchor hit / eight of them
SPECS["groups8_hit_512"] = WorkloadSpec(name="groups8_hit_512", n_layers=24, d_model=2560, n_k_heads=16, n_v_heads=32, d_k=128,
                                        d_v=128, n_requests=1, replay=("fixed", 512), group=True, group_size=3,
                                        d_ff=(10240,) * 24)
SPECS["groups8_hits8_512"] = dataclasses.replace(SPECS["groups8_hit_512"], name="groups8_hits8_512", n_requests=8)
SPECS["groups_small"] = WorkloadSpec(name="groups_small", n_layers=7, d_model=256, n_k_heads=2, n_v_heads=4, d_k=64, d_v=64,
                                     n_requests=3, replay=("list", (70, 0, 200)), group=True, group_size=3,
                                     d_ff=(0, 192, 0, 128, 0, 0, 64))
SPECS["group3_4b"] = WorkloadSpec(name="group3_4b", n_layers=3, d_model=2560, n_k_heads=16, n_v_heads=32, d_k=128, d_v=128,
                                  n_requests=8, replay=("fixed", 512), group=True, d_ff=(10240, 10240, 10240))
for _r in (1024, 2048, 4096):
    SPECS[f"cfg4_R{_r}"] = dataclasses.replace(SPECS["cfg4"], name=f"cfg4_R{_r}", replay=("fixed", _r))


@dataclasses.dataclass
class LayerParams:
    """Parameters of one linear-attention layer's in-projection, conv and gates."""
    w_qkv: torch.Tensor                 # [C, d] bf16, or uint8 e4m3 codes; rows q | k | v, head-major
    w_qkv_scale: Optional[torch.Tensor]  # [ceil(C/128), d/128] fp32 block scales (e4m3 only)
    w_ab: torch.Tensor                  # [2*H_v, d] bf16: decay rows a_0.., then write-strength rows b_0..
    conv_w: torch.Tensor                # [C, w] bf16; tap w-1 multiplies the current row
    decay_scale: torch.Tensor           # [H_v] fp32  (c_h)
    dt_bias: torch.Tensor               # [H_v] fp32  (delta_h)


@dataclasses.dataclass
class BlockParams:
    """The rest of one block of a group (Section 4.1): norms, output gate and projection, optional MLP.  All bf16."""
    norm_w: torch.Tensor                # [d]
    w_z: torch.Tensor                   # [H_v d_v, d]
    o_norm_w: torch.Tensor              # [d_v]
    w_o: torch.Tensor                   # [d, H_v d_v]
    mlp_norm_w: Optional[torch.Tensor] = None   # [d]
    w_gate: Optional[torch.Tensor] = None       # [f, d]
    w_up: Optional[torch.Tensor] = None         # [f, d]
    w_down: Optional[torch.Tensor] = None       # [d, f]


@dataclasses.dataclass
class Workload:
    spec: WorkloadSpec
    anchor_pool: torch.Tensor           # [n_phys, L_pool, PAGE_ROWS, d] bf16
    layer_to_pool: List[int]            # per model layer: pool layer index or -1
    layer_mask: List[int]               # per model layer: 1 = rebuild this layer's state
    page_table: torch.Tensor            # [B, max_pages] int32, oldest page first, -1 padding
    replay_lens: torch.Tensor           # [B] int32, rows to replay per request
    layers: List[Optional[LayerParams]]  # None for masked-out layers
    blocks: Optional[List[BlockParams]] = None   # group workloads only

    @property
    def groups(self) -> List[Tuple[int, int]]:
        """(first layer, layers) of every group of a group workload."""
        gs = self.spec.group_size or self.spec.n_layers
        return [(f, min(gs, self.spec.n_layers - f)) for f in range(0, self.spec.n_layers, gs)]

    @property
    def n_phys_pages(self) -> int:
        return int(self.anchor_pool.shape[0])

    @property
    def total_rows(self) -> int:
        return int(self.replay_lens.sum().item())

    @property
    def n_active_layers(self) -> int:
        return int(sum(self.layer_mask))

    @property
    def layer_tokens(self) -> int:
        """Replayed tokens summed over the layers that are rebuilt."""
        return self.total_rows * self.n_active_layers


def _generator(device, seed: int, tensor_id: int, layer: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1_000_003 + tensor_id * 10_007 + layer) & 0x7FFFFFFFFFFFFFFF)
    return g


def _normal(shape: Sequence[int], std: float, gen: torch.Generator, device, dtype,
            chunk: int = 1 << 27) -> torch.Tensor:
    """iid N(0, std^2) drawn in fp32 and cast once to ``dtype``, in bounded chunks."""
    out = torch.empty(tuple(shape), dtype=dtype, device=device)
    flat = out.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        x = torch.randn(e - s, generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            x.mul_(std)
        flat[s:e] = x.to(dtype)
    return out


def _replay_pages(spec: WorkloadSpec, rng: np.random.RandomState) -> Tuple[np.ndarray, np.ndarray]:
    kind = spec.replay[0]
    B = spec.n_requests
    if kind == "fixed":
        lens = np.full(B, int(spec.replay[1]), dtype=np.int64)
    elif kind == "pages_uniform":
        lo, hi = int(spec.replay[1]), int(spec.replay[2])
        lens = rng.randint(lo, hi + 1, size=B).astype(np.int64) * PAGE_ROWS
    elif kind == "list":
        lens = np.asarray(spec.replay[1], dtype=np.int64)
        assert lens.shape[0] == B
    else:
        raise ValueError(kind)
    pages = (lens + PAGE_ROWS - 1) // PAGE_ROWS
    return lens, pages


def _page_tables(spec: WorkloadSpec, seed: int) -> Tuple[np.ndarray, np.ndarray, int]:
    """Returns (page_table [B, max_pages] int32 with -1 padding, replay_lens [B], n_phys)."""
    rng = np.random.RandomState((seed * 7919 + 17) & 0x7FFFFFFF)
    lens, n_pages = _replay_pages(spec, rng)
    B = spec.n_requests
    max_pages = max(1, int(n_pages.max()))
    table = np.full((B, max_pages), -1, dtype=np.int32)
    if spec.paging in ("identity", "shuffled"):
        n_phys = max(1, int(n_pages.sum()))
        ids = np.arange(n_phys, dtype=np.int32)
        if spec.paging == "shuffled":
            rng.shuffle(ids)
        at = 0
        for i in range(B):
            table[i, : n_pages[i]] = ids[at: at + n_pages[i]]
            at += int(n_pages[i])
    elif spec.paging == "trunks":
        # Requests branch from shared prefixes ("trunks").  Request i sits on trunk
        # i // requests_per_trunk; its cached boundary is a page index on that trunk and
        # its replay window is the n_i logical pages before the boundary.  Only logical
        # pages covered by some window get a physical page (anchors are kept only for the
        # rows that some boundary replays); overlapping windows share physical pages.
        trunk_of = [min(i // spec.requests_per_trunk, spec.n_trunks - 1) for i in range(B)]
        first = np.zeros(B, dtype=np.int64)
        for i in range(B):
            n_i = int(n_pages[i])
            assert n_i <= spec.trunk_pages
            boundary = int(rng.randint(max(n_i, 1), spec.trunk_pages + 1))
            first[i] = boundary - n_i
        covered = sorted({(trunk_of[i], int(first[i]) + p) for i in range(B) for p in range(int(n_pages[i]))})
        n_phys = max(1, len(covered))
        perm = np.arange(n_phys, dtype=np.int32)
        rng.shuffle(perm)
        phys = {key: int(perm[j]) for j, key in enumerate(covered)}
        for i in range(B):
            for p in range(int(n_pages[i])):
                table[i, p] = phys[(trunk_of[i], int(first[i]) + p)]
    else:
        raise ValueError(spec.paging)
    return table, lens.astype(np.int32), n_phys


def build_workload(spec_or_name, device="cpu", seed: int = 0,
                   pool_on_device: bool = True) -> Workload:
    """Generate every input of one replay call for ``spec`` on ``device``."""
    spec = SPECS[spec_or_name] if isinstance(spec_or_name, str) else spec_or_name
    device = torch.device(device)
    d, C, Hv, w = spec.d_model, spec.conv_channels, spec.n_v_heads, spec.conv_width

    if spec.layer_mask == "all":
        mask = [1] * spec.n_layers
    elif spec.layer_mask == "even":
        mask = [1 if l % 2 == 0 else 0 for l in range(spec.n_layers)]
    else:
        raise ValueError(spec.layer_mask)
    layer_to_pool, n_pool = [], 0
    for l in range(spec.n_layers):
        if spec.group:                 # one anchor per group: the rows entering its first layer
            gs = spec.group_size or spec.n_layers
            if l % gs == 0:
                layer_to_pool.append(n_pool)
                n_pool += 1
            else:
                layer_to_pool.append(-1)
        elif mask[l]:
            layer_to_pool.append(n_pool)
            n_pool += 1
        else:
            layer_to_pool.append(-1)

    table, lens, n_phys = _page_tables(spec, seed)
    pool_device = device if pool_on_device else torch.device("cpu")
    pool = _normal((n_phys, n_pool, PAGE_ROWS, d), 1.0, _generator(pool_device, seed, 1),
                   pool_device, torch.bfloat16)

    layers: List[Optional[LayerParams]] = []
    for l in range(spec.n_layers):
        if not mask[l]:
            layers.append(None)
            continue
        if spec.weight_format == "bf16":
            w_qkv = _normal((C, d), d ** -0.5, _generator(device, seed, 2, l), device, torch.bfloat16)
            scale = None
        elif spec.weight_format == "e4m3_block128":
            # codes = e4m3(64 * xi), block scales lognormal (sigma 0.5) with E[scale^2]
            # chosen so that code * scale keeps variance 1/d.
            codes = _normal((C, d), 64.0, _generator(device, seed, 2, l), device, torch.float32)
            w_qkv = codes.to(torch.float8_e4m3fn).view(torch.uint8)
            del codes
            z = _normal(((C + 127) // 128, (d + 127) // 128), 1.0, _generator(device, seed, 3, l),
                        device, torch.float32)
            scale = (torch.exp(0.5 * z - 0.25) / (64.0 * math.sqrt(d))).to(torch.float32).contiguous()
        else:
            raise ValueError(spec.weight_format)
        w_ab = _normal((2 * Hv, d), d ** -0.5, _generator(device, seed, 4, l), device, torch.bfloat16)
        conv_w = _normal((C, w), w ** -0.5, _generator(device, seed, 5, l), device, torch.bfloat16)
        layers.append(LayerParams(
            w_qkv=w_qkv, w_qkv_scale=scale, w_ab=w_ab, conv_w=conv_w,
            decay_scale=torch.full((Hv,), spec.decay_scale, dtype=torch.float32, device=device),
            dt_bias=torch.zeros((Hv,), dtype=torch.float32, device=device)))

    blocks = None
    if spec.group:
        hv = Hv * spec.d_v
        blocks = []

        def uniform(n, tid, l):        # norm weights around 1
            g = _generator(device, seed, tid, l)
            return (0.5 + torch.rand(n, generator=g, device=device, dtype=torch.float32)).to(torch.bfloat16)

        for l in range(spec.n_layers):
            b = BlockParams(norm_w=uniform(d, 6, l),
                            w_z=_normal((hv, d), d ** -0.5, _generator(device, seed, 7, l), device, torch.bfloat16),
                            o_norm_w=uniform(spec.d_v, 8, l),
                            w_o=_normal((d, hv), hv ** -0.5, _generator(device, seed, 9, l), device, torch.bfloat16))
            f = spec.d_ff[l] if l < len(spec.d_ff) else 0
            if f:
                b.mlp_norm_w = uniform(d, 10, l)
                b.w_gate = _normal((f, d), d ** -0.5, _generator(device, seed, 11, l), device, torch.bfloat16)
                b.w_up = _normal((f, d), d ** -0.5, _generator(device, seed, 12, l), device, torch.bfloat16)
                b.w_down = _normal((d, f), f ** -0.5, _generator(device, seed, 13, l), device, torch.bfloat16)
            blocks.append(b)

    return Workload(spec=spec, anchor_pool=pool, layer_to_pool=layer_to_pool, layer_mask=mask,
                    page_table=torch.from_numpy(table).to(device),
                    replay_lens=torch.from_numpy(lens).to(device), layers=layers, blocks=blocks)


# ---- raw-byte views for the CPU side -------------------------------------------------

def bits_u16(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 array of the same shape holding the raw bits."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def layer_arrays(p: LayerParams) -> dict:
    """One layer's parameters as plain numpy arrays of raw storage values."""
    out = {
        "w_ab_bits": bits_u16(p.w_ab),
        "conv_w_bits": bits_u16(p.conv_w),
        "decay_scale": p.decay_scale.detach().cpu().numpy().astype(np.float32),
        "dt_bias": p.dt_bias.detach().cpu().numpy().astype(np.float32),
    }
    if p.w_qkv.dtype == torch.bfloat16:
        out["w_qkv_bits"] = bits_u16(p.w_qkv)
    else:
        out["w_qkv_codes"] = p.w_qkv.detach().cpu().numpy().astype(np.uint8)
        out["w_qkv_scale"] = p.w_qkv_scale.detach().cpu().numpy().astype(np.float32)
    return out


def block_arrays(p: LayerParams, b: BlockParams) -> dict:
    """One group layer's parameters as fp64 arrays of the stored values (exact: bf16 -> fp64 loses nothing)."""
    f64 = lambda t: t.detach().to(torch.float64).cpu().numpy()
    out = dict(norm_w=f64(b.norm_w), w_qkv=f64(p.w_qkv), w_ab=f64(p.w_ab), conv_w=f64(p.conv_w),
               decay_scale=f64(p.decay_scale), dt_bias=f64(p.dt_bias), w_z=f64(b.w_z), o_norm_w=f64(b.o_norm_w), w_o=f64(b.w_o))
    if b.mlp_norm_w is not None:
        out.update(mlp_norm_w=f64(b.mlp_norm_w), w_gate=f64(b.w_gate), w_up=f64(b.w_up), w_down=f64(b.w_down))
    return out


def fetch_pages(wl: Workload, page_ids: Sequence[int], pool_layer: int) -> dict:
    """Copy whole pool pages back to the host by physical id: returns
    ``{(page_id, pool_layer): uint16 [PAGE_ROWS, d]}``.  Data movement only -- which page
    a request row lives on is for the consumer to work out from the page table.  Lets a
    CPU check read the few pages it needs out of a pool too large to copy back."""
    out = {}
    for pid in sorted({int(x) for x in page_ids}):
        if 0 <= pid < wl.n_phys_pages:
            out[(pid, pool_layer)] = bits_u16(wl.anchor_pool[pid, pool_layer])
    return out
