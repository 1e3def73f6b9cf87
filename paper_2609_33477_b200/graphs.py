"""Replay graphs with static buffers (Section 5.2, "Batched replay"; Section 6, "Replay graphs").

The replay call reads lengths, page tables and destination slots on the device and allocates nothing, so one
captured CUDA graph serves every batch that fits the bounds it was captured with.  Grids and scratch are sized by
those bounds, so a few graphs are kept, one per bucket of (requests, total packed rows); a batch is copied into
the static buffers, padded with sentinel segments (slot -1: nothing is read or written for them), and the
smallest bucket that holds it is replayed.  Host logic only: every step of the path runs in the captured kernels.
"""

from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence, Tuple

import torch

from . import binding


class BucketedGraphReplayer:
    """``buckets``: (max_requests, max_total_rows) pairs.  ``workload`` supplies the model, the weights, the anchor
    pool and the widest page table; states go to ``n_slots`` state slots shared by all buckets."""

    def __init__(self, workload, buckets: Sequence[Tuple[int, int]], n_slots: int, max_replay_len: Optional[int] = None):
        dev = workload.page_table.device
        spec = workload.spec
        self.device = dev
        self.max_pages = int(workload.page_table.shape[1])
        self.buckets: List[Tuple[int, int]] = sorted((int(b), int(r)) for b, r in buckets)
        b_max = max(b for b, _ in self.buckets)
        max_replay_len = self.max_pages * 64 if max_replay_len is None else int(max_replay_len)
        # static inputs, shared by every bucket (a bucket reads its first max_requests entries)
        self.pages = torch.zeros((b_max, self.max_pages), dtype=torch.int32, device=dev)
        self.lens = torch.zeros((b_max,), dtype=torch.int32, device=dev)
        self.slots = torch.full((b_max,), -1, dtype=torch.int32, device=dev)
        L = spec.n_layers
        self.out_ssm = torch.zeros((n_slots, L, spec.n_v_heads, spec.d_k, spec.d_v), dtype=torch.float32, device=dev)
        self.out_conv = torch.zeros((n_slots, L, spec.conv_channels, spec.conv_width - 1), dtype=torch.bfloat16, device=dev)
        self._stream = torch.cuda.Stream(dev)
        self._reps: List[binding.Replayer] = []
        self._graphs: List[torch.cuda.CUDAGraph] = []
        for b, rows in self.buckets:
            view = dataclasses.replace(workload, page_table=self.pages[:b], replay_lens=self.lens[:b])
            rep = binding.Replayer(view, state_slots=self.slots[:b], n_slots=n_slots, max_total_rows=rows,
                                   max_replay_len=min(max_replay_len, rows), out_ssm=self.out_ssm, out_conv=self.out_conv)
            with torch.cuda.stream(self._stream):
                rep.replay_states(self._stream)              # one-time function attributes, outside the capture
            self._stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=self._stream):
                rep.replay_states(torch.cuda.current_stream(dev))
            self._reps.append(rep)
            self._graphs.append(graph)

    def pick(self, n_requests: int, total_rows: int) -> int:
        """Index of the smallest bucket that holds the batch; ValueError if none does."""
        for i, (b, rows) in enumerate(self.buckets):
            if n_requests <= b and total_rows <= rows:
                return i
        raise ValueError(f"no bucket holds {n_requests} requests / {total_rows} rows")

    def replay(self, pages: torch.Tensor, lens: torch.Tensor, slots: torch.Tensor) -> int:
        """Rebuilds the states of one batch: ``pages`` [n, <= max_pages] int32 and ``slots`` [n] int32 (host or
        device tensors), ``lens`` [n] int32 on the HOST -- the bucket is chosen from the lengths the scheduler
        already holds, so nothing here waits for the device (the hit path adds no host synchronisation,
        Section 5.2).  Returns the bucket used.  Asynchronous on the current stream."""
        if lens.device.type != "cpu":
            raise ValueError("replay lengths must be a host tensor: the bucket is picked on the host, without a device sync")
        n = int(lens.shape[0])
        i = self.pick(n, int(lens.clamp(min=0).sum()))
        b = self.buckets[i][0]
        self.slots[:b].fill_(-1)                              # padding segments: sentinel
        self.lens[:b].zero_()
        self.pages[:n, :pages.shape[1]].copy_(pages, non_blocking=True)
        self.lens[:n].copy_(lens, non_blocking=True)
        self.slots[:n].copy_(slots, non_blocking=True)
        self._graphs[i].replay()
        return i

    def device_status(self, bucket: int) -> int:
        return self._reps[bucket].device_status()
