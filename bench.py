#!/usr/bin/env python
"""Benchmark of the suffix-replay hot path: replayed tokens/s across linear layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg3] [--impl ours|reference]

One step = one pass of the whole hot path (schedule, anchor gather + in-projection, conv state,
conv/SiLU/norm/gates + gated-delta state scan for every rebuilt layer) over one synthetic batch.
Prints ONE JSON line.  `value` counts layer-tokens (replayed rows x rebuilt layers) per second
with inputs resident in HBM; `e2e` is the same metric through the host-buffer entry point
(anchors and tables copied host->device and both states device->host inside the timed region).
With N > 1 every rank replays its own copy of the batch (requests, layers and heads are independent
units: no collective on the data path), so the scaling is weak.  Started under torchrun the ranks come
from the environment; started plainly with --gpus N the script launches its N ranks itself.
"""

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "replayed tokens/s across linear layers"
UNIT = "layer-tokens/s"
DEFAULT_CONFIG = "cfg3"

# Where the DRAM traffic of the dominant kernel comes from: the committed summary of an ncu capture of that
# kernel -- at full size where the two DRAM counters fit one ncu pass (cfg3), else on a slice of the workload (same
# kernel, tile shapes and per-row traffic, small enough to capture).
# Each summary carries one line `traffic_per_launch: read_bytes=... write_bytes=... rows=...`; the figure
# reported here is that capture scaled by rows (an upper bound: the weight part of the reads does not grow).
NCU_TRAFFIC_SUMMARY = {
    "cfg3_slice": "sr_proj_fused2_kernel_cfg3_slice.md", "cfg4_slice": "sr_proj_fused2_kernel_fp8_cfg4_slice.md",
}
NCU_TRAFFIC_SUMMARY.update({c: "dram_traffic_full_size.md" for c in
                            ("cfg0", "cfg1", "cfg2", "cfg3", "cfg4", "cfg4_w8a8", "hit_512", "hits8_512")})


def ncu_traffic(config, rows):
    """(bytes per launch, source) from the committed ncu summary for `config`, scaled to `rows`; (None, None) if
    no capture of that kernel shape exists."""
    import re
    name = NCU_TRAFFIC_SUMMARY.get(config)
    if name is None:
        return None, None
    path = os.path.join(ROOT, "profiles", name)
    try:
        text = open(path).read()
    except OSError:
        return None, None
    pat = r"\s*read_bytes=([0-9.eE+]+)\s+write_bytes=([0-9.eE+]+)\s+rows=(\d+)"
    m = re.search("traffic_per_launch_" + config + ":" + pat, text) or re.search("traffic_per_launch:" + pat, text)
    if not m:
        return None, None
    cap_rows = int(m.group(3))
    total = float(m.group(1)) + float(m.group(2))
    if cap_rows == rows:
        return total, f"profiles/{name} (captured at this size, {rows} rows)"
    return total * rows / cap_rows, f"profiles/{name} ({cap_rows} rows captured, scaled by rows to {rows})"


def measure_fp8_peak(dev):
    """Dense e4m3 GEMM throughput of this GPU through the library (TFLOP/s), the yardstick for the W8A8 projection:
    MEASURED_PEAKS.json holds no 8-bit figure.  Returns None where the library call is unavailable."""
    import torch
    try:
        n = 8192
        a = torch.randn(n, n, device=dev).to(torch.float8_e4m3fn)
        b = torch.randn(n, n, device=dev).to(torch.float8_e4m3fn).t()          # column-major second operand
        one = torch.ones((), device=dev, dtype=torch.float32)
        for _ in range(3):
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(10):
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        e1.record()
        torch.cuda.synchronize(dev)
        return 10 * 2.0 * n ** 3 / (e0.elapsed_time(e1) * 1e-3) / 1e12
    except Exception:
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.05)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def _oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_one(wl, req, layer, rows):
    """Times the CPU oracle, as it stands, on the first `rows` rows of one (request, layer)."""
    import numpy as np
    from oracle import gdn_replay_oracle as orc
    from paper_2609_33477_b200 import synth
    s = wl.spec
    pages = wl.page_table[req, : -(-rows // 64)].cpu().tolist()
    pl = wl.layer_to_pool[layer]
    pool = synth.fetch_pages(wl, pages, pl)
    arrays = synth.layer_arrays(wl.layers[layer])
    t0 = time.perf_counter()
    S, _ = orc.replay_request_layer(pool, pages, rows, pl, arrays, n_k_heads=s.n_k_heads, n_v_heads=s.n_v_heads,
                                    d_k=s.d_k, d_v=s.d_v, erase=s.recurrence != "decay_only",
                                    act_quant=getattr(s, "act_quant", "none"))
    dt = time.perf_counter() - t0
    assert np.all(np.isfinite(S))
    return dt


ORACLE_JOB_ROWS = 4096


def oracle_job(wl, reps=1):
    """The fixed job the CPU oracle is timed on, the same for every caller: the first min(R, 4096) rows of the
    longest request, first rebuilt layer, all heads.  Returns (seconds, layer_tokens, description, threads)."""
    s = wl.spec
    lens = wl.replay_lens.cpu().tolist()
    layer = next(l for l, m in enumerate(wl.layer_mask) if m)
    if not lens or max(lens) <= 0:
        return 1e-9, 0, f"{s.name}: empty batch", _oracle_threads()
    req = max(range(len(lens)), key=lambda i: (lens[i], -i))
    rows = int(min(lens[req], ORACLE_JOB_ROWS))
    total_t = sum(oracle_one(wl, req, layer, rows) for _ in range(reps))
    desc = (f"{s.name}: request {req} (the longest, {lens[req]} rows), its first {rows} rows, layer {layer}, all "
            f"{s.n_v_heads} heads, {reps}x (of {len(lens) * wl.n_active_layers} request-layers in a step)")
    return total_t, rows * reps, desc, _oracle_threads()


def max_over_ranks(value, device):
    """A per-rank time -> the slowest rank's time, on every rank (no-op without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(layer_tokens_per_rank, steps, total_ms, world):
    """Whole-job layer-tokens/s: every rank replays its own batch, the slowest rank's clock counts."""
    return world * layer_tokens_per_rank * steps / (total_ms * 1e-3)


def shard_units(units, rank, world):
    """Independent units (requests, layers, heads) dealt round-robin to ranks: no exchange is needed."""
    return list(units[rank::world])


def launch_ranks(n, argv):
    """Re-runs this script as `n` ranks on this node (one per GPU) under torch.distributed.run; returns its exit code."""
    import socket
    import subprocess
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_dry(args, rank, world):
    """The multi-rank plumbing without the kernels: rendezvous, barrier, max over ranks, one line from rank 0."""
    import torch
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group(args.backend)
        dist.barrier()
    dev = torch.device("cpu")
    total_ms = max_over_ranks(args.steps * (10.0 + rank), dev)          # the slowest rank's clock counts
    value = aggregate_throughput(1000, args.steps, total_ms, world)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
                          "scaling": "weak", "dry": True, "data": "none",
                          "config": {"workload": args.config, "note": "dry run: no kernel was launched"}}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_reference(args, rank):
    """--impl reference: the CPU oracle timed on the host cores, same metric and config."""
    if rank != 0:
        return
    import torch
    from paper_2609_33477_b200 import synth
    # input generation only: the large pools are drawn on the GPU when there is one (seconds instead
    # of minutes); the oracle then reads the pages it samples back to the host and runs on the host cores
    gen_device = "cuda:0" if torch.cuda.is_available() else "cpu"
    wl = synth.build_workload(args.config, device=gen_device)
    for _ in range(args.warmup):
        oracle_job(wl)
    total_t, total_lt, desc, threads = 0.0, 0, "", 1
    for _ in range(args.steps):
        dt, lt, desc, threads = oracle_job(wl)
        total_t += dt
        total_lt += lt
    value = total_lt / total_t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.config, "note": "CPU oracle, one fixed bounded job per step (see cpu_baseline.sample)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_group(args, wl, dev, rank, world, warmup):
    """A group workload (Section 4.1: one anchor per group of linear-attention layers): times sr_replay_group_states.
    A side workload, not the headline configuration: no host-buffer arm and no oracle arm."""
    import torch
    from paper_2609_33477_b200 import binding
    spec = wl.spec
    rep = binding.Replayer(wl)
    stream = torch.cuda.current_stream(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    groups = wl.groups
    if len(groups) > 1:          # all the model's groups in one call, side by side
        call = lambda: rep.replay_groups_states(stream=stream)
    else:
        call = lambda: rep.replay_group_states(stream=stream)
    for _ in range(warmup):
        call()
    torch.cuda.synchronize(dev)
    assert rep.group_device_status() == 0
    launches = rep.last_launch_count()
    sampler = ClockSampler(int(os.environ.get("LOCAL_RANK", "0")))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    sampler.start()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)
        e0.record(stream)
        call()
        e1.record(stream)
        torch.cuda.synchronize(dev)
        times.append(e0.elapsed_time(e1))
    clocks = sampler.stop()
    in_turn_ms = None
    if len(groups) > 1:          # the same groups one after the other (the least workspace)
        seq = []
        for i in range(min(args.steps, 5)):
            flush.fill_(i & 0xFF)
            e0.record(stream)
            rep.replay_groups_states(stream=stream, min_workspace=True)
            e1.record(stream)
            torch.cuda.synchronize(dev)
            seq.append(e0.elapsed_time(e1))
        in_turn_ms = sorted(seq)[len(seq) // 2]
    total_ms = max_over_ranks(sum(times), dev)
    ms = total_ms / args.steps
    binding.sr_profile_enable(rep.ctx, True)
    call()
    torch.cuda.synchronize(dev)
    kernel_ms = {}
    for k, kind in binding.KERNEL_KINDS.items():
        t, n = binding.sr_profile_read(rep.ctx, kind)
        kernel_ms[k] = {"ms": t, "launches": n} if n else None
    binding.sr_profile_enable(rep.ctx, False)
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # the oracle on the host cores: the whole group for the first request (a fixed, bounded job)
        import numpy as np
        from oracle import gdn_replay_oracle as orc
        from paper_2609_33477_b200 import synth
        R0 = int(wl.replay_lens[0].item())
        pages = wl.page_table[0, : -(-R0 // 64)].cpu().tolist()
        got = synth.fetch_pages(wl, pages, 0)
        rows0 = np.concatenate([orc.bf16_bits_to_f64(got[(p, 0)]) for p in pages])[:R0]
        layers = [synth.block_arrays(wl.layers[l], wl.blocks[l]) for l in range(spec.n_layers)]
        t0 = time.perf_counter()
        orc.group_replay(rows0, layers, n_k_heads=spec.n_k_heads, n_v_heads=spec.n_v_heads, d_k=spec.d_k, d_v=spec.d_v)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": R0 * spec.n_layers / dt, "unit": UNIT, "cores": _oracle_threads(), "kind": "oracle",
                        "sample": f"{spec.name}: request 0 ({R0} rows), all {spec.n_layers} layers of the group, once",
                        "seconds": dt}
    hv = spec.n_v_heads * spec.d_v
    L = spec.n_layers
    proj = L * 2.0 * spec.d_model * (spec.conv_channels + 2 * spec.n_v_heads)
    block = 0.0                  # every layer but the last of each group runs its block
    for first, n in groups:
        block += (n - 1) * 4.0 * spec.d_model * hv + sum(6.0 * spec.d_model * f for f in spec.d_ff[first:first + n - 1])
    rows = wl.total_rows
    peaks = measured_peaks()
    gb = kernel_ms.get("group_block")
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": world * rows * L / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": spec.name, "group_layers": L, "groups": len(groups), "groups_in_turn_ms": in_turn_ms,
                       "d_model": spec.d_model, "heads": spec.n_v_heads,
                       "d_head": spec.d_k, "d_ff": list(spec.d_ff), "requests": spec.n_requests, "replayed_rows": rows,
                       "l2": "256 MB flush buffer written between timed steps"},
            "clocks": clocks, "e2e": None, "gpu_launches": launches * args.steps,
            "roofline": {"kernel": "all dense products of the group (projections, output gate, output projection, MLP) over "
                                   "the call time", "bound": "tensor", "achieved": (proj + block) * rows / (ms * 1e-3) / 1e12,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": (proj + block) * rows / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                         "peak_source": f"{peaks['source']} bf16 burst", "traffic": None, "kernel_ms": kernel_ms,
                         "block_tflops": (block * rows / (gb["ms"] * 1e-3) / 1e12) if gb else None},
            "cpu_baseline": cpu_baseline}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default=DEFAULT_CONFIG)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"],
                    help="process-group backend for the timing barrier and the max over ranks")
    ap.add_argument("--dry", action="store_true",
                    help="launch and reduce only: every rank reports a made-up step time instead of running the "
                         "kernels (checks the N-rank plumbing on a box without GPUs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not started by a launcher: start one rank per GPU ourselves and let rank 0 print the line
        raise SystemExit(launch_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.dry:
        run_dry(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_33477_b200 import binding, synth
    from paper_2609_33477_b200 import build as sr_build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the replay path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group(args.backend, device_id=dev if args.backend == "nccl" else None)
    if rank == 0:
        sr_build.build()
    if world > 1:
        dist.barrier()
    binding.load()

    warmup = max(args.warmup, 3)
    wl = synth.build_workload(args.config, device=dev, seed=0)
    spec = wl.spec
    if spec.group:
        run_group(args, wl, dev, rank, world, warmup)
        return
    rep = binding.Replayer(wl)
    stream = torch.cuda.current_stream(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)     # > the 126 MB L2
    LT = wl.layer_tokens

    def step():
        rep.replay_states(stream)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize(dev)
    assert rep.device_status() == 0
    launches_per_step = rep.last_launch_count()

    # ---- timed region: K steps, CUDA events on the launching stream, L2 flushed between steps
    sampler = ClockSampler(local_rank)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(dev)
    sampler.start()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)
        starts[i].record(stream)
        step()
        ends[i].record(stream)
    torch.cuda.synchronize(dev)
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    times = sorted(s.elapsed_time(e) for s, e in zip(starts, ends))
    total_ms = sum(times)
    total_ms = max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    value = aggregate_throughput(LT, args.steps, total_ms, world)

    # ---- per-kernel device time (events inside the call).  Where the call keeps several layers in flight a kernel's
    # elapsed time includes what it shares its SMs with, so the per-kernel figures (and the roofline of the dominant
    # kernel, which must agree with a profiler's serialised launch list) are taken with the layers one after the
    # other -- the same kernels in the least workspace -- and the overlapped projection time is reported beside them.
    def profile(r, n_steps):
        binding.sr_profile_enable(r.ctx, True)
        acc = {k: [0.0, 0] for k in binding.KERNEL_KINDS}
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        whole = 0.0
        for i in range(n_steps):
            flush.fill_(i & 0xFF)
            t0.record(stream)
            r.replay_states(stream)
            t1.record(stream)
            torch.cuda.synchronize(dev)
            whole += t0.elapsed_time(t1)
            for k, kind in binding.KERNEL_KINDS.items():
                ms, n = binding.sr_profile_read(r.ctx, kind)
                acc[k][0] += ms
                acc[k][1] += n
        binding.sr_profile_enable(r.ctx, False)
        return acc, whole / n_steps

    prof_steps = min(args.steps, 5)
    overlap = None
    ws_min = binding.sr_workspace_bytes_min(rep.ctx, rep.table)
    if rep.workspace_bytes > ws_min:
        over, _ = profile(rep, min(prof_steps, 2))
        serial = binding.Replayer(wl, min_workspace=True, out_ssm=rep.out_ssm, out_conv=rep.out_conv)
        for _ in range(2):
            serial.replay_states(stream)
        torch.cuda.synchronize(dev)
        kern, serial_ms = profile(serial, prof_steps)
        serial.close()
        del serial
        overlap = {"workspace_bytes": rep.workspace_bytes, "workspace_bytes_min": ws_min,
                   "ms_per_step_layers_serialised": serial_ms,
                   "projection_ms_overlapped": over["projection"][0] / max(1, over["projection"][1]),
                   "note": "the timed steps keep several layers in flight; kernel_ms and the roofline below are of "
                           "the same kernels run one layer after the other"}
    else:
        kern, _ = profile(rep, prof_steps)
    kernel_ms = {k: (v[0] / v[1] if v[1] else None) for k, v in kern.items()}
    kernel_share = {k: v[0] / max(1e-9, sum(x[0] for x in kern.values())) for k, v in kern.items()}

    peaks = measured_peaks()
    w8a8 = getattr(spec, "act_quant", "none") == "e4m3_1x128"
    fp8_peak = measure_fp8_peak(dev) if w8a8 else None
    n_alg = spec.n_k_heads * spec.d_k + spec.n_v_heads * spec.d_v + 2 * spec.n_v_heads
    proj_flops_per_lt = 2.0 * spec.d_model * n_alg
    proj_ms = kernel_ms["projection"]
    long_step = ms_per_step > 50.0
    peak_tf = peaks["bf16_tflops_sustained"] if long_step else peaks["bf16_tflops"]
    peak_src = f"{peaks['source']} bf16 {'sustained' if long_step else 'burst'}"
    if fp8_peak:       # the 8-bit tensor path is held against an 8-bit library GEMM timed in this very run
        peak_tf, peak_src = fp8_peak, "torch._scaled_mm e4m3 x e4m3 -> bf16, 8192^3, timed in this run (burst)"
    achieved_tf = proj_flops_per_lt * wl.total_rows / (proj_ms * 1e-3) / 1e12 if proj_ms else None
    # the chunk scan (chunk-local + state chain): analytic FLOPs of the chunked form per token and head --
    # K K^T, the triangular solve, T [K | V], W S and K^T U at 64-row chunks -- over its two kernels' time
    Cn, dk, dv = 64, spec.d_k, spec.d_v
    scan_flops_per_lt = spec.n_v_heads * (2 * Cn * dk + Cn * Cn / 3 + 2 * Cn * (dk + dv) + 4 * dk * dv)
    scan_ms = (kernel_ms["scan"] or 0.0) + (kernel_ms["chunk_local"] or 0.0)
    scan_tf = scan_flops_per_lt * wl.total_rows / (scan_ms * 1e-3) / 1e12 if scan_ms else None
    path_tf = (proj_flops_per_lt + scan_flops_per_lt) * LT / (ms_per_step * 1e-3) / 1e12

    # the anchor gather on its own (it is otherwise fused into the projection's TMA loads): the debug entry
    # point copies every replayed row of one layer; bytes = rows * d * 2, read once and written once
    gather = None
    rows_cap = max(1, int(rep.table.max_total_rows))
    if rows_cap * spec.d_model * 2 <= (8 << 30):
        gl = next(l for l in range(spec.n_layers) if wl.layer_mask[l])
        gout = torch.empty((rows_cap, spec.d_model), dtype=torch.bfloat16, device=dev)

        def gather_once():
            st = binding.sr_debug_gather(rep.ctx, rep.pool, rep.table, wl.replay_lens.data_ptr(), gl, gout.data_ptr(),
                                         rows_cap, rep._ws_ptr, rep.workspace_bytes, rep._stream_ptr(stream))
            assert st == 0
        for _ in range(3):
            gather_once()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 5
        torch.cuda.synchronize(dev)
        g_ms = 0.0
        for i in range(reps):
            flush.fill_(i & 0xFF)
            g0.record(stream)
            gather_once()
            g1.record(stream)
            torch.cuda.synchronize(dev)
            g_ms += g0.elapsed_time(g1)
        g_bytes = 2.0 * wl.total_rows * spec.d_model * 2
        gbs = g_bytes / (g_ms / reps * 1e-3) / 1e9
        gather = {"kernel": "standalone gather (debug entry point: schedule + copy of one layer's rows)", "bound": "hbm",
                  "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                  "bytes": g_bytes, "ms": g_ms / reps}
        del gout

    # the sidecar's write side on its own: a step whose sampled tokens fill the first pages of the pool, all pool
    # layers at once; the hidden states are the pool's own rows, so the pool keeps its content
    anchor_write = None
    n_phys, l_pool = int(wl.anchor_pool.shape[0]), int(wl.anchor_pool.shape[1])
    w_pages = min(n_phys, 512)
    if w_pages >= 8:
        w_tokens = w_pages * 64
        hidden = wl.anchor_pool[:w_pages].permute(1, 0, 2, 3).reshape(l_pool, w_tokens, spec.d_model).contiguous()
        tok = torch.arange(w_tokens, device=dev, dtype=torch.int32)
        d_page, d_row = (tok // 64).contiguous(), (tok % 64).contiguous()

        def write_once():
            st = binding.sr_anchor_write(rep.ctx, rep.pool, list(range(l_pool)), hidden.data_ptr(), hidden.stride(0) * 2,
                                         hidden.stride(1) * 2, d_page.data_ptr(), d_row.data_ptr(), w_tokens, None,
                                         rep._stream_ptr(stream))
            assert st == 0
        for _ in range(3):
            write_once()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w_ms = 0.0
        for i in range(5):
            flush.fill_(i & 0xFF)
            w0.record(stream)
            write_once()
            w1.record(stream)
            torch.cuda.synchronize(dev)
            w_ms += w0.elapsed_time(w1)
        w_bytes = 2.0 * l_pool * w_tokens * spec.d_model * 2
        w_gbs = w_bytes / (w_ms / 5 * 1e-3) / 1e9
        anchor_write = {"kernel": "anchor write (indexed stores of a step's sampled hidden states, all pool layers)",
                        "bound": "hbm", "achieved": w_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": w_gbs / peaks["hbm_gbs"], "bytes": w_bytes, "ms": w_ms / 5, "tokens": w_tokens,
                        "layers": l_pool}
        del hidden

    # one boundary alone: the longest request of the batch as a batch of its own (its own bounds and workspace, as a
    # caller serving a single hit would set it up; the layers of such a small call run side by side)
    import dataclasses
    lens_host = wl.replay_lens.cpu()
    longest = int(torch.argmax(lens_host).item())
    single_rows = int(lens_host[longest].item())
    n_pg = max(1, -(-single_rows // 64))
    one = dataclasses.replace(wl, page_table=wl.page_table[longest:longest + 1, :n_pg].contiguous(),
                              replay_lens=wl.replay_lens[longest:longest + 1].clone())
    rep1 = binding.Replayer(one)
    for _ in range(3):
        rep1.replay_states(stream)
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    single = []
    for i in range(7):
        flush.fill_(i & 0xFF)
        s0.record(stream)
        rep1.replay_states(stream)
        s1.record(stream)
        torch.cuda.synchronize(dev)
        single.append(s0.elapsed_time(s1))
    assert rep1.device_status() == 0
    single_ms = sorted(single)[len(single) // 2]
    rep1.close()
    del rep1, one

    # short steps only: the same call captured once in a CUDA graph and replayed (Section 6, "Replay graphs")
    graph_ms = None
    if ms_per_step < 5.0:
        cap = torch.cuda.Stream(dev)
        with torch.cuda.stream(cap):
            rep.replay_states(cap)
        cap.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=cap):
            rep.replay_states(torch.cuda.current_stream(dev))
        for _ in range(3):
            g.replay()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gt = []
        for i in range(15):
            flush.fill_(i & 0xFF)
            q0.record()
            g.replay()
            q1.record()
            torch.cuda.synchronize(dev)
            gt.append(q0.elapsed_time(q1))
        graph_ms = sorted(gt)[len(gt) // 2]
        del g

    # group-propagated replay (Section 4.1) on its own workload: three linear-attention layers of the 4B geometry fed
    # by one group-entry anchor, eight 512-row hits; every layer's block (gate, outputs, output projection, MLP) runs
    group = None
    if rank == 0 and world == 1 and spec.weight_format == "bf16":
        gwl = synth.build_workload("group3_4b", device=dev, seed=0)
        grep_ = binding.Replayer(gwl)
        for _ in range(3):
            grep_.replay_group_states(stream=stream)
        torch.cuda.synchronize(dev)
        assert grep_.group_device_status() == 0
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gts = []
        for i in range(7):
            flush.fill_(i & 0xFF)
            g0.record(stream)
            grep_.replay_group_states(stream=stream)
            g1.record(stream)
            torch.cuda.synchronize(dev)
            gts.append(g0.elapsed_time(g1))
        g_ms = sorted(gts)[len(gts) // 2]
        gs = gwl.spec
        hv = gs.n_v_heads * gs.d_v
        g_flops = gwl.total_rows * (gs.n_layers * 2.0 * gs.d_model * (gs.conv_channels + 2 * gs.n_v_heads) +
                                    (gs.n_layers - 1) * 4.0 * gs.d_model * hv +
                                    sum(6.0 * gs.d_model * f for f in gs.d_ff[:gs.n_layers - 1]))
        group = {"workload": gs.name, "group_layers": gs.n_layers, "rows": gwl.total_rows, "ms": g_ms,
                 "layer_tokens_per_s": gwl.total_rows * gs.n_layers / (g_ms * 1e-3),
                 "dense_tflops": g_flops / (g_ms * 1e-3) / 1e12, "launches": grep_.last_launch_count(),
                 "note": "dense FLOPs of projections, gate, output projection and MLP over the call time"}
        grep_.close()
        del grep_, gwl

    traffic, traffic_source = ncu_traffic(args.config, wl.total_rows)
    roofline = {
        "kernel": "projection (anchor gather + in-projection), per layer launch",
        "bound": "tensor", "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s",
        "frac": achieved_tf / peak_tf if achieved_tf else None,
        "peak_source": peak_src,
        "flops_per_launch": proj_flops_per_lt * wl.total_rows,
        "traffic": traffic, "traffic_source": traffic_source,
        "kernel_ms": kernel_ms, "kernel_time_share": kernel_share, "overlap": overlap,
        "scan": {"kernels": "chunk-local + state chain, per layer", "achieved": scan_tf, "unit": "TFLOP/s",
                 "frac": scan_tf / peak_tf if scan_tf else None, "flops_per_layer_token": scan_flops_per_lt,
                 "ms": scan_ms, "note": "bound by the serial chain and short-CTA latency, not by the tensor pipe"},
        "path": {"what": "projection + scan FLOPs of the whole step over the step time", "achieved": path_tf,
                 "unit": "TFLOP/s", "frac_of_sustained": path_tf / peaks["bf16_tflops_sustained"],
                 "frac_of_burst": path_tf / peaks["bf16_tflops"]},
        "gather": gather,
        "anchor_write": anchor_write,
    }

    # ---- end to end: host buffers in, host states out, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        pool_bytes = wl.anchor_pool.numel() * 2
        host_pool = torch.empty(wl.anchor_pool.shape, dtype=torch.bfloat16, pin_memory=True)
        host_pool.copy_(wl.anchor_pool)
        host_pages = wl.page_table.cpu().pin_memory()
        host_lens = wl.replay_lens.cpu().pin_memory()
        host_ssm = torch.empty(rep.out_ssm.shape, dtype=torch.float32, pin_memory=True)
        host_conv = torch.empty(rep.out_conv.shape, dtype=torch.bfloat16, pin_memory=True)
        e2e_steps = max(1, min(args.steps, 5))
        for _ in range(2):
            rep.replay_states_host(host_pool, host_pages, host_lens, host_ssm, host_conv, stream)
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            rep.replay_states_host(host_pool, host_pages, host_lens, host_ssm, host_conv, stream)
            torch.cuda.synchronize(dev)        # the caller reads the states on the host
        e2e_s = time.perf_counter() - t0
        e2e_s = max_over_ranks(e2e_s, dev)
        # what the call copies: the pool layers the rebuilt layers read, the tables; the rebuilt layers' outputs
        active = [l for l in range(spec.n_layers) if wl.layer_mask[l]]
        used_pool_layers = len({wl.layer_to_pool[l] for l in active})
        n_phys, l_pool = wl.anchor_pool.shape[0], wl.anchor_pool.shape[1]
        h2d = pool_bytes // l_pool * used_pool_layers + host_pages.numel() * 4 + host_lens.numel() * 4
        d2h = (rep.out_ssm.numel() * 4 + rep.out_conv.numel() * 2) // spec.n_layers * len(active)
        e2e = {"value": world * LT * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": 1e3 * e2e_s / e2e_steps, "steps": e2e_steps}
        del host_pool

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        dt, lt, desc, threads = oracle_job(wl, reps=2)
        cpu_baseline = {"value": lt / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc,
                        "seconds": dt}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            # operand type of the tensor-core products: bf16, or fp16 for block-scaled weights (dequantised to fp16)
            "dtype": "e4m3" if w8a8 else ("f16" if spec.weight_format == "e4m3_block128" else "bf16"),
            "data": "synthetic",
            "config": {"workload": spec.name, "n_layers_rebuilt": wl.n_active_layers, "d_model": spec.d_model,
                       "heads": spec.n_v_heads, "d_head": spec.d_k, "requests": spec.n_requests,
                       "replayed_rows": wl.total_rows, "layer_tokens_per_step": LT,
                       "weights": spec.weight_format, "l2": "256 MB flush buffer written between timed steps",
                       "p50_rebuild_ms": times[len(times) // 2],
                       "p95_rebuild_ms": times[min(len(times) - 1, int(0.95 * len(times)))],
                       "single_boundary_ms": single_ms, "single_boundary_rows": single_rows,
                       "graph_replay_ms": graph_ms, "group_replay": group},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
