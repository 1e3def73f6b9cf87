"""ctypes binding of the C boundary (``include/sr_replay.h``): same names, argument
marshalling only.  Every step of the replay path runs in the CUDA kernels behind the
boundary; there is no CPU path, and loading fails loudly if the library is missing.

Two layers:
  * the raw entry points ``sr_create`` ... ``sr_device_status`` taking ctypes structs;
  * ``Replayer``: packs torch tensors (device memory, streams) into those structs.
"""

from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsr_replay.so")

SR_OK, SR_ERR_INVALID_ARG, SR_ERR_UNSUPPORTED_SHAPE, SR_ERR_WORKSPACE, SR_ERR_CUDA = 0, 1, 2, 3, 4
SR_DEV_BAD_REPLAY_LEN, SR_DEV_BAD_PAGE_ID, SR_DEV_BAD_SLOT, SR_DEV_ROWS_OVERFLOW, SR_DEV_WAIT_EXPIRED = 1, 2, 4, 8, 16
SR_W_BF16, SR_W_E4M3_BLOCK128 = 0, 1
SR_CONV_SILU, SR_CONV_IDENTITY = 0, 1
SR_REC_GATED_DELTA, SR_REC_DECAY_ONLY = 0, 1
SR_AQ_NONE, SR_AQ_E4M3_1X128 = 0, 1
SR_DEV_BOUNDS_CHECK = 32
SR_DEBUG_DOT_CONV_STATE, SR_DEBUG_SINGLE_CTA_MMA, SR_DEBUG_FP8_EXACT, SR_DEBUG_CHECK_BOUNDS, SR_DEBUG_EXPIRE_WAIT = 1, 2, 4, 8, 16

EXPORTS = (
    "sr_version", "sr_status_string", "sr_create", "sr_destroy", "sr_ssm_bytes_per_layer",
    "sr_conv_bytes_per_layer", "sr_workspace_bytes", "sr_replay_states", "sr_replay_states_host",
    "sr_debug_gather", "sr_device_status", "sr_last_launch_count", "sr_profile_enable", "sr_profile_read",
    "sr_replay_states_noalloc", "sr_replay_states_from", "sr_anchor_write", "sr_workspace_bytes_min",
    "sr_debug_quantise", "sr_group_workspace_bytes", "sr_replay_group_states", "sr_groups_workspace_bytes",
    "sr_replay_groups_states",
)
SR_NOALLOC_SCRATCH_BYTES = 128 * 1024 * 1024
SR_KERNEL_SCHEDULE, SR_KERNEL_PROJECTION, SR_KERNEL_CONV_TAIL, SR_KERNEL_SCAN = 0, 1, 2, 3
KERNEL_KINDS = {"schedule": 0, "projection": 1, "conv_tail": 2, "scan": 3, "weight_decode": 4, "chunk_local": 5, "anchor_stage": 6,
                "group_block": 7}


class sr_model_desc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_k_heads", C.c_int32),
                ("n_v_heads", C.c_int32), ("d_k", C.c_int32), ("d_v", C.c_int32),
                ("conv_width", C.c_int32), ("page_rows", C.c_int32), ("weight_format", C.c_int32),
                ("conv_activation", C.c_int32), ("l2_eps", C.c_float), ("recurrence", C.c_int32),
                ("debug_flags", C.c_uint32), ("act_quant", C.c_int32)]


class sr_layer_weights(C.Structure):
    _fields_ = [("w_qkv", C.c_void_p), ("w_qkv_scale", C.c_void_p), ("w_ab", C.c_void_p),
                ("conv_w", C.c_void_p), ("decay_scale", C.c_void_p), ("dt_bias", C.c_void_p)]


class sr_anchor_pool(C.Structure):
    _fields_ = [("base", C.c_void_p), ("page_stride_bytes", C.c_int64), ("layer_stride_bytes", C.c_int64),
                ("row_stride_bytes", C.c_int64), ("n_phys_pages", C.c_int32), ("n_pool_layers", C.c_int32),
                ("layer_to_pool", C.POINTER(C.c_int32))]


class sr_page_table(C.Structure):
    _fields_ = [("pages", C.c_void_p), ("state_slots", C.c_void_p), ("n_requests", C.c_int32),
                ("max_pages", C.c_int32), ("max_replay_len", C.c_int32), ("max_total_rows", C.c_int64),
                ("n_state_slots", C.c_int32)]


class sr_block_weights(C.Structure):
    _fields_ = [("norm_w", C.c_void_p), ("w_z", C.c_void_p), ("o_norm_w", C.c_void_p), ("w_o", C.c_void_p),
                ("mlp_norm_w", C.c_void_p), ("w_gate", C.c_void_p), ("w_up", C.c_void_p), ("w_down", C.c_void_p),
                ("d_ff", C.c_int32)]


class sr_out(C.Structure):
    _fields_ = [("base", C.c_void_p), ("slot_stride_bytes", C.c_int64), ("layer_stride_bytes", C.c_int64)]


_lib = None


def load() -> C.CDLL:
    """Load the CUDA library (built in-tree by ``paper_2609_33477_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    path = os.environ.get("SR_REPLAY_LIB", LIB_PATH)      # e.g. an instrumented build of the same sources
    if not os.path.exists(path):
        raise RuntimeError(
            f"{path} is missing: build it with `python -m paper_2609_33477_b200.build`. "
            "There is no CPU fallback for the replay path.")
    lib = C.CDLL(path)
    lib.sr_version.restype = C.c_char_p
    lib.sr_status_string.restype = C.c_char_p
    lib.sr_status_string.argtypes = [C.c_int]
    lib.sr_create.argtypes = [C.POINTER(sr_model_desc), C.POINTER(C.c_void_p)]
    lib.sr_destroy.argtypes = [C.c_void_p]
    lib.sr_destroy.restype = None
    lib.sr_ssm_bytes_per_layer.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
    lib.sr_conv_bytes_per_layer.argtypes = [C.c_void_p, C.POINTER(C.c_size_t)]
    lib.sr_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(sr_page_table), C.POINTER(C.c_size_t)]
    lib.sr_workspace_bytes_min.argtypes = [C.c_void_p, C.POINTER(sr_page_table), C.POINTER(C.c_size_t)]
    lib.sr_replay_states.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_void_p,
        C.POINTER(sr_layer_weights), C.POINTER(sr_out), C.POINTER(sr_out), C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_replay_states_from.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_void_p,
        C.POINTER(sr_layer_weights), C.POINTER(sr_out), C.POINTER(sr_out), C.POINTER(sr_out), C.POINTER(sr_out),
        C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_replay_states_noalloc.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_void_p,
        C.POINTER(sr_layer_weights), C.POINTER(sr_out), C.POINTER(sr_out), C.c_void_p]
    lib.sr_replay_states_host.argtypes = [
        C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
        C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.POINTER(sr_layer_weights),
        C.POINTER(sr_out), C.c_size_t, C.c_void_p, C.POINTER(sr_out), C.c_size_t, C.c_void_p,
        C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_anchor_write.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(C.c_int32), C.c_int32, C.c_void_p, C.c_int64, C.c_int64,
        C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
    lib.sr_debug_gather.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_int32, C.c_void_p,
        C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_debug_quantise.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
        C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_group_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(sr_page_table), C.c_int32, C.POINTER(C.c_size_t)]
    lib.sr_replay_group_states.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_int32, C.c_int32,
        C.POINTER(sr_layer_weights), C.POINTER(sr_block_weights), C.c_float, C.POINTER(sr_out), C.POINTER(sr_out),
        C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_groups_workspace_bytes.argtypes = [C.c_void_p, C.POINTER(sr_page_table), C.c_int32, C.c_int32, C.POINTER(C.c_size_t)]
    lib.sr_replay_groups_states.argtypes = [
        C.c_void_p, C.POINTER(sr_anchor_pool), C.POINTER(sr_page_table), C.c_void_p, C.c_int32, C.POINTER(C.c_int32),
        C.POINTER(C.c_int32), C.POINTER(sr_layer_weights), C.POINTER(sr_block_weights), C.c_float, C.POINTER(sr_out),
        C.POINTER(sr_out), C.c_void_p, C.c_size_t, C.c_void_p]
    lib.sr_device_status.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_uint32)]
    lib.sr_last_launch_count.argtypes = [C.c_void_p, C.POINTER(C.c_int64)]
    lib.sr_profile_enable.argtypes = [C.c_void_p, C.c_int]
    lib.sr_profile_read.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
    for name in EXPORTS:
        if name not in ("sr_version", "sr_status_string", "sr_destroy"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


class SrError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {load().sr_status_string(status).decode()}")


def _check(status: int, where: str) -> None:
    if status != SR_OK:
        raise SrError(status, where)


# ---- raw entry points, same names as the header -------------------------------------

def sr_version() -> str:
    return load().sr_version().decode()


def sr_create(desc: sr_model_desc) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(load().sr_create(C.byref(desc), C.byref(ctx)), "sr_create")
    return ctx


def sr_destroy(ctx) -> None:
    load().sr_destroy(ctx)


def sr_ssm_bytes_per_layer(ctx) -> int:
    n = C.c_size_t()
    _check(load().sr_ssm_bytes_per_layer(ctx, C.byref(n)), "sr_ssm_bytes_per_layer")
    return n.value


def sr_conv_bytes_per_layer(ctx) -> int:
    n = C.c_size_t()
    _check(load().sr_conv_bytes_per_layer(ctx, C.byref(n)), "sr_conv_bytes_per_layer")
    return n.value


def sr_workspace_bytes(ctx, table: sr_page_table) -> int:
    n = C.c_size_t()
    _check(load().sr_workspace_bytes(ctx, C.byref(table), C.byref(n)), "sr_workspace_bytes")
    return n.value


def sr_workspace_bytes_min(ctx, table: sr_page_table) -> int:
    n = C.c_size_t()
    _check(load().sr_workspace_bytes_min(ctx, C.byref(table), C.byref(n)), "sr_workspace_bytes_min")
    return n.value


def sr_group_workspace_bytes(ctx, table: sr_page_table, max_d_ff: int) -> int:
    out = C.c_size_t()
    _check(load().sr_group_workspace_bytes(ctx, C.byref(table), int(max_d_ff), C.byref(out)), "sr_group_workspace_bytes")
    return int(out.value)


def sr_groups_workspace_bytes(ctx, table: sr_page_table, max_d_ff: int, n_groups: int) -> int:
    out = C.c_size_t()
    _check(load().sr_groups_workspace_bytes(ctx, C.byref(table), int(max_d_ff), int(n_groups), C.byref(out)),
           "sr_groups_workspace_bytes")
    return int(out.value)


def sr_replay_groups_states(ctx, pool, table, replay_lens_ptr, first_layers: Sequence[int], group_sizes: Sequence[int], weights,
                            blocks, norm_eps, out_ssm, out_conv, workspace_ptr, workspace_bytes, stream_ptr) -> int:
    n = len(first_layers)
    return load().sr_replay_groups_states(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, n, (C.c_int32 * n)(*first_layers),
                                          (C.c_int32 * n)(*group_sizes), weights, blocks, float(norm_eps), C.byref(out_ssm),
                                          C.byref(out_conv), workspace_ptr, workspace_bytes, stream_ptr)


def sr_replay_group_states(ctx, pool, table, replay_lens_ptr, first_layer, n_group_layers, weights, blocks, norm_eps,
                           out_ssm, out_conv, debug_rows_ptr, workspace_ptr, workspace_bytes, stream_ptr) -> int:
    return load().sr_replay_group_states(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, int(first_layer),
                                         int(n_group_layers), weights, blocks, float(norm_eps), C.byref(out_ssm),
                                         C.byref(out_conv), debug_rows_ptr, workspace_ptr, workspace_bytes, stream_ptr)


def sr_replay_states(ctx, pool, table, replay_lens_ptr, layer_mask, weights, out_ssm, out_conv,
                     workspace_ptr, workspace_bytes, stream_ptr) -> int:
    return load().sr_replay_states(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, layer_mask, weights,
                                   C.byref(out_ssm), C.byref(out_conv), workspace_ptr, workspace_bytes, stream_ptr)


def sr_replay_states_from(ctx, pool, table, replay_lens_ptr, layer_mask, weights, in_ssm, in_conv, out_ssm, out_conv,
                          workspace_ptr, workspace_bytes, stream_ptr) -> int:
    """Replay that continues the states in ``in_ssm`` / ``in_conv`` (``None`` = zero) instead of starting from zero."""
    return load().sr_replay_states_from(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, layer_mask, weights,
                                        C.byref(in_ssm) if in_ssm is not None else None,
                                        C.byref(in_conv) if in_conv is not None else None,
                                        C.byref(out_ssm), C.byref(out_conv), workspace_ptr, workspace_bytes, stream_ptr)


def sr_replay_states_noalloc(ctx, pool, table, replay_lens_ptr, layer_mask, weights, out_ssm, out_conv,
                             stream_ptr) -> int:
    """The replay call for callers that cannot allocate device memory: no workspace argument, the
    scratch is a fixed SR_NOALLOC_SCRATCH_BYTES array inside the library (see the header)."""
    return load().sr_replay_states_noalloc(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, layer_mask,
                                           weights, C.byref(out_ssm), C.byref(out_conv), stream_ptr)


def sr_anchor_write(ctx, pool, pool_layers: Sequence[int], hidden_ptr, hidden_layer_stride, hidden_row_stride,
                    dest_page_ptr, dest_row_ptr, n_tokens, status_ptr, stream_ptr) -> int:
    """Indexed stores of a step's sampled hidden states into the anchor pool (``sr_anchor_write``)."""
    arr = (C.c_int32 * len(pool_layers))(*pool_layers)
    return load().sr_anchor_write(ctx, C.byref(pool), arr, len(pool_layers), hidden_ptr, hidden_layer_stride,
                                  hidden_row_stride, dest_page_ptr, dest_row_ptr, n_tokens, status_ptr, stream_ptr)


def sr_debug_gather(ctx, pool, table, replay_lens_ptr, layer, out_rows_ptr, capacity_rows,
                    workspace_ptr, workspace_bytes, stream_ptr) -> int:
    return load().sr_debug_gather(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, layer, out_rows_ptr,
                                  capacity_rows, workspace_ptr, workspace_bytes, stream_ptr)


def sr_debug_quantise(ctx, pool, table, replay_lens_ptr, layer, out_codes_ptr, out_scales_ptr, capacity_rows,
                      workspace_ptr, workspace_bytes, stream_ptr) -> int:
    return load().sr_debug_quantise(ctx, C.byref(pool), C.byref(table), replay_lens_ptr, layer, out_codes_ptr,
                                    out_scales_ptr, capacity_rows, workspace_ptr, workspace_bytes, stream_ptr)


def sr_device_status(ctx, workspace_ptr, stream_ptr) -> int:
    v = C.c_uint32()
    _check(load().sr_device_status(ctx, workspace_ptr, stream_ptr, C.byref(v)), "sr_device_status")
    return v.value


def sr_last_launch_count(ctx) -> int:
    v = C.c_int64()
    _check(load().sr_last_launch_count(ctx, C.byref(v)), "sr_last_launch_count")
    return v.value


def sr_profile_enable(ctx, enable: bool) -> None:
    _check(load().sr_profile_enable(ctx, 1 if enable else 0), "sr_profile_enable")


def sr_profile_read(ctx, kind: int):
    ms, n = C.c_float(), C.c_int64()
    _check(load().sr_profile_read(ctx, kind, C.byref(ms), C.byref(n)), "sr_profile_read")
    return ms.value, n.value


# ---- marshalling of torch tensors ---------------------------------------------------

def model_desc(spec, conv_activation: int = SR_CONV_SILU, l2_eps: float = 1e-6, debug_flags: int = 0) -> sr_model_desc:
    fmt = SR_W_E4M3_BLOCK128 if spec.weight_format == "e4m3_block128" else SR_W_BF16
    return sr_model_desc(spec.n_layers, spec.d_model, spec.n_k_heads, spec.n_v_heads, spec.d_k, spec.d_v,
                         spec.conv_width, 64, fmt, conv_activation, l2_eps,
                         SR_REC_DECAY_ONLY if getattr(spec, "recurrence", "gated_delta") == "decay_only" else SR_REC_GATED_DELTA,
                         debug_flags, SR_AQ_E4M3_1X128 if getattr(spec, "act_quant", "none") == "e4m3_1x128" else SR_AQ_NONE)


class Replayer:
    """Holds a context plus the ctypes images of one workload's device buffers.

    ``workload`` is a ``synth.Workload`` whose tensors live on a CUDA device (only the
    anchor pool may be given separately, e.g. a staging buffer).  Nothing is computed
    here: the methods fill structs with ``data_ptr()`` values and call the C boundary.
    """

    def __init__(self, workload, conv_activation: int = SR_CONV_SILU, l2_eps: float = 1e-6,
                 state_slots: Optional[torch.Tensor] = None, n_slots: Optional[int] = None,
                 max_total_rows: Optional[int] = None, max_replay_len: Optional[int] = None,
                 out_ssm: Optional[torch.Tensor] = None, out_conv: Optional[torch.Tensor] = None,
                 debug_flags: int = 0, min_workspace: bool = False):
        self.wl = workload
        spec = workload.spec
        self.spec = spec
        self.desc = model_desc(spec, conv_activation, l2_eps, debug_flags)
        self.ctx = sr_create(self.desc)
        dev = workload.page_table.device
        if dev.type != "cuda":
            raise RuntimeError("the replay path runs on a CUDA device only (no CPU fallback)")
        self.device = dev
        L = spec.n_layers
        self._l2p = (C.c_int32 * L)(*workload.layer_to_pool)
        self.layer_mask = (C.c_uint8 * L)(*workload.layer_mask)
        self.weights = (sr_layer_weights * L)()
        for l, p in enumerate(workload.layers):
            if p is None:
                continue
            self.weights[l] = sr_layer_weights(
                p.w_qkv.data_ptr(), p.w_qkv_scale.data_ptr() if p.w_qkv_scale is not None else None,
                p.w_ab.data_ptr(), p.conv_w.data_ptr(), p.decay_scale.data_ptr(), p.dt_bias.data_ptr())
        self.set_pool(workload.anchor_pool)
        B, max_pages = workload.page_table.shape
        self.state_slots = state_slots
        lens_host = workload.replay_lens.cpu()
        if max_total_rows is None:
            max_total_rows = int(lens_host.clamp(min=0).sum().item())
        if max_replay_len is None:
            max_replay_len = min(int(max_pages) * 64, max(0, int(lens_host.max().item()) if B else 0))
        self.table = sr_page_table(
            workload.page_table.data_ptr(), state_slots.data_ptr() if state_slots is not None else None,
            B, max_pages, max_replay_len, max_total_rows, int(n_slots) if n_slots is not None else B)
        self.n_slots = int(n_slots) if n_slots is not None else B
        self.ssm_layer_bytes = sr_ssm_bytes_per_layer(self.ctx)
        self.conv_layer_bytes = sr_conv_bytes_per_layer(self.ctx)
        C_ch = spec.conv_channels
        ssm_shape = (self.n_slots, L, spec.n_v_heads, spec.d_k, spec.d_v)
        conv_shape = (self.n_slots, L, C_ch, spec.conv_width - 1)
        if out_ssm is not None:      # state-slot arrays owned by the caller (shared between several Replayers)
            assert tuple(out_ssm.shape) == ssm_shape and out_ssm.dtype == torch.float32 and out_ssm.is_contiguous()
        if out_conv is not None:
            assert tuple(out_conv.shape) == conv_shape and out_conv.dtype == torch.bfloat16 and out_conv.is_contiguous()
        self.out_ssm = out_ssm if out_ssm is not None else torch.zeros(ssm_shape, dtype=torch.float32, device=dev)
        self.out_conv = out_conv if out_conv is not None else torch.zeros(conv_shape, dtype=torch.bfloat16, device=dev)
        self._out_ssm = sr_out(self.out_ssm.data_ptr(), L * self.ssm_layer_bytes, self.ssm_layer_bytes)
        self._out_conv = sr_out(self.out_conv.data_ptr(), L * self.conv_layer_bytes, self.conv_layer_bytes)
        # min_workspace: the least scratch the call accepts (layers one after the other) instead of the recommended size
        self.workspace_bytes = (sr_workspace_bytes_min if min_workspace else sr_workspace_bytes)(self.ctx, self.table)
        self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=dev)
        self._ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256

    def set_pool(self, pool: torch.Tensor) -> None:
        """Point the call at an anchor pool tensor [n_phys, L_pool, 64, d] (bf16, device)."""
        assert pool.dtype == torch.bfloat16 and pool.dim() == 4 and pool.stride(3) == 1
        self.pool_tensor = pool
        self.pool = sr_anchor_pool(pool.data_ptr(), pool.stride(0) * 2, pool.stride(1) * 2, pool.stride(2) * 2,
                                   pool.shape[0], pool.shape[1], self._l2p)

    def close(self) -> None:
        if self.ctx is not None:
            sr_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _stream_ptr(self, stream) -> int:
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        return s.cuda_stream

    def replay_states(self, stream=None, check: bool = True) -> int:
        """One ``sr_replay_states`` call on the workload's buffers (asynchronous)."""
        st = sr_replay_states(self.ctx, self.pool, self.table, self.wl.replay_lens.data_ptr(), self.layer_mask,
                              self.weights, self._out_ssm, self._out_conv, self._ws_ptr, self.workspace_bytes,
                              self._stream_ptr(stream))
        if check:
            _check(st, "sr_replay_states")
        return st

    def replay_group_states(self, first_layer: int = 0, n_group_layers: Optional[int] = None, norm_eps: float = 1e-6,
                            debug_rows: bool = False, stream=None, check: bool = True):
        """One ``sr_replay_group_states`` call: the workload's layers first_layer .. as one group, fed by the anchors of
        the first (Section 4.1).  With ``debug_rows`` also returns the rows handed from layer to layer, bf16
        [n_group_layers - 1, max_slots * 64, d] in packed page-slot order."""
        wl, spec = self.wl, self.spec
        if wl.blocks is None:
            raise ValueError("not a group workload")
        g = spec.n_layers - first_layer if n_group_layers is None else int(n_group_layers)
        self._group_setup()
        rows = None
        if debug_rows and g > 1:
            B = self.table.n_requests
            max_slots = (min(self.table.max_total_rows // 64 + B, B * self.table.max_pages) + 3) // 4 * 4
            rows = torch.zeros((g - 1, max(max_slots, 4) * 64, spec.d_model), dtype=torch.bfloat16, device=self.device)
        st = sr_replay_group_states(self.ctx, self.pool, self.table, wl.replay_lens.data_ptr(), first_layer, g, self.weights,
                                    self._blocks, norm_eps, self._out_ssm, self._out_conv,
                                    rows.data_ptr() if rows is not None else None, self._group_ws_ptr, self._group_ws_bytes,
                                    self._stream_ptr(stream))
        if check:
            _check(st, "sr_replay_group_states")
        return (st, rows) if debug_rows else st

    def _group_setup(self, n_groups: int = 1) -> None:
        """Block-weight structs and a workspace with room for ``n_groups`` groups side by side (made once, grown on demand)."""
        wl, spec = self.wl, self.spec
        if not hasattr(self, "_blocks"):
            self._blocks = (sr_block_weights * spec.n_layers)()
            ptr = lambda t: t.data_ptr() if t is not None else None
            for l, b in enumerate(wl.blocks):
                self._blocks[l] = sr_block_weights(ptr(b.norm_w), ptr(b.w_z), ptr(b.o_norm_w), ptr(b.w_o), ptr(b.mlp_norm_w),
                                                   ptr(b.w_gate), ptr(b.w_up), ptr(b.w_down),
                                                   int(b.w_gate.shape[0]) if b.w_gate is not None else 0)
            self._max_ff = max([int(b.w_gate.shape[0]) for b in wl.blocks if b.w_gate is not None] + [0])
            self._group_ws_bytes = 0
        need = sr_groups_workspace_bytes(self.ctx, self.table, self._max_ff, n_groups)
        if need > self._group_ws_bytes:
            self._group_ws_bytes = need
            self._group_ws = torch.empty(need + 256, dtype=torch.uint8, device=self.device)
            self._group_ws_ptr = (self._group_ws.data_ptr() + 255) // 256 * 256

    def replay_groups_states(self, groups: Optional[Sequence] = None, norm_eps: float = 1e-6, stream=None, check: bool = True,
                             min_workspace: bool = False) -> int:
        """One ``sr_replay_groups_states`` call: ``groups`` = [(first_layer, n_layers), ...] (default: the workload's own
        groups), replayed side by side where the workspace has room (``min_workspace``: one group's worth only)."""
        wl = self.wl
        if wl.blocks is None:
            raise ValueError("not a group workload")
        groups = list(wl.groups) if groups is None else list(groups)
        self._group_setup(1 if min_workspace else len(groups))
        ws_bytes = sr_group_workspace_bytes(self.ctx, self.table, self._max_ff) if min_workspace else self._group_ws_bytes
        st = sr_replay_groups_states(self.ctx, self.pool, self.table, wl.replay_lens.data_ptr(), [g[0] for g in groups],
                                     [g[1] for g in groups], self.weights, self._blocks, norm_eps, self._out_ssm, self._out_conv,
                                     self._group_ws_ptr, ws_bytes, self._stream_ptr(stream))
        if check:
            _check(st, "sr_replay_groups_states")
        return st

    def group_device_status(self, stream=None) -> int:
        return sr_device_status(self.ctx, self._group_ws_ptr, self._stream_ptr(stream))

    def replay_states_from(self, in_ssm: Optional[torch.Tensor], in_conv: Optional[torch.Tensor], stream=None,
                           check: bool = True) -> int:
        """``sr_replay_states_from``: continue the given states (tensors shaped like ``out_ssm`` / ``out_conv``;
        ``None`` = zero; may be the output tensors themselves)."""
        L = self.spec.n_layers
        a = None if in_ssm is None else sr_out(in_ssm.data_ptr(), L * self.ssm_layer_bytes, self.ssm_layer_bytes)
        b = None if in_conv is None else sr_out(in_conv.data_ptr(), L * self.conv_layer_bytes, self.conv_layer_bytes)
        st = sr_replay_states_from(self.ctx, self.pool, self.table, self.wl.replay_lens.data_ptr(), self.layer_mask,
                                   self.weights, a, b, self._out_ssm, self._out_conv, self._ws_ptr,
                                   self.workspace_bytes, self._stream_ptr(stream))
        if check:
            _check(st, "sr_replay_states_from")
        return st

    def replay_states_host(self, host_pool: torch.Tensor, host_pages: torch.Tensor, host_lens: torch.Tensor,
                           host_out_ssm: torch.Tensor, host_out_conv: torch.Tensor, stream=None) -> None:
        """``sr_replay_states_host``: host anchors/tables in, host states out, copies included."""
        st = load().sr_replay_states_host(
            self.ctx, host_pool.data_ptr(), host_pool.numel() * host_pool.element_size(), host_pages.data_ptr(),
            None, host_lens.data_ptr(), self.wl.replay_lens.data_ptr(), C.byref(self.pool), C.byref(self.table),
            self.layer_mask, self.weights, C.byref(self._out_ssm), self.out_ssm.numel() * 4, host_out_ssm.data_ptr(),
            C.byref(self._out_conv), self.out_conv.numel() * 2, host_out_conv.data_ptr(), self._ws_ptr,
            self.workspace_bytes, self._stream_ptr(stream))
        _check(st, "sr_replay_states_host")

    def debug_gather(self, layer: int, stream=None) -> torch.Tensor:
        rows = max(1, int(self.table.max_total_rows))
        out = torch.zeros((rows, self.spec.d_model), dtype=torch.bfloat16, device=self.device)
        st = sr_debug_gather(self.ctx, self.pool, self.table, self.wl.replay_lens.data_ptr(), layer, out.data_ptr(),
                             rows, self._ws_ptr, self.workspace_bytes, self._stream_ptr(stream))
        _check(st, "sr_debug_gather")
        return out

    def debug_quantise(self, layer: int, stream=None):
        """W8A8 contexts: the activation codes [rows, d] (uint8) and scales [rows, d / 128] (fp32) of one layer."""
        rows = max(1, int(self.table.max_total_rows))
        codes = torch.zeros((rows, self.spec.d_model), dtype=torch.uint8, device=self.device)
        scales = torch.zeros((rows, self.spec.d_model // 128), dtype=torch.float32, device=self.device)
        st = sr_debug_quantise(self.ctx, self.pool, self.table, self.wl.replay_lens.data_ptr(), layer, codes.data_ptr(),
                               scales.data_ptr(), rows, self._ws_ptr, self.workspace_bytes, self._stream_ptr(stream))
        _check(st, "sr_debug_quantise")
        return codes, scales

    def device_status(self, stream=None) -> int:
        return sr_device_status(self.ctx, self._ws_ptr, self._stream_ptr(stream))

    def last_launch_count(self) -> int:
        return sr_last_launch_count(self.ctx)
