"""The N > 1 path of the benchmark on CPU: ranks replay independent replicas (no collective on the
data path); only the timing is reduced across ranks (max) and the throughput is the sum of what all
ranks processed.  Run as two gloo processes."""

import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, {root!r})
    import torch, torch.distributed as dist
    import bench
    dist.init_process_group("gloo", init_method="tcp://127.0.0.1:{port}", rank=int(sys.argv[1]), world_size=2)
    rank = dist.get_rank()
    # each rank "measures" a different time; the slowest rank defines the step
    total_ms = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
    value = bench.aggregate_throughput(layer_tokens_per_rank=1000, steps=4, total_ms=total_ms, world=2)
    shards = bench.shard_units(list(range(7)), rank, 2)
    out = dict(rank=rank, total_ms=total_ms, value=value, shards=shards)
    gathered = [None, None]
    dist.all_gather_object(gathered, out)
    if rank == 0:
        print(json.dumps(gathered))
    dist.destroy_process_group()
""")


def test_two_ranks_reduce_time_by_max_and_sum_throughput(tmp_path):
    import json
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, port=port))
    procs = [subprocess.Popen([sys.executable, str(script), str(r)], stdout=subprocess.PIPE, stderr=subprocess.PIPE,
                              text=True) for r in range(2)]
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    res = json.loads(outs[0][0].strip().splitlines()[-1])
    assert [r["total_ms"] for r in res] == [15.0, 15.0]                      # max over ranks, on every rank
    assert all(abs(r["value"] - 2 * 1000 * 4 / 15e-3) < 1e-6 for r in res)   # whole-job layer-tokens/s
    assert res[0]["shards"] == [0, 2, 4, 6] and res[1]["shards"] == [1, 3, 5]  # disjoint, covering


def test_bench_launches_its_own_ranks_when_not_under_a_launcher():
    """`python bench.py --gpus 2` outside torchrun starts two ranks itself; with --dry --backend gloo they only
    rendezvous, reduce a made-up time by max and print one line from rank 0 (no GPU needed)."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "4", "--dry",
                        "--backend", "gloo"], capture_output=True, text=True, timeout=300, env=env)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["dry"] is True
    assert abs(line["ms_per_step"] - 11.0) < 1e-9            # the slower rank (10 + 1 ms per step)
    assert abs(line["value"] - 2 * 1000 * 4 / (44.0 * 1e-3)) < 1e-6
