"""The multi-rank plumbing of bench.py on CPU (gloo, world size 2): the layer does not shard (replicas only), so
what more than one rank adds is the max-over-ranks timing, the aggregate throughput and the rule that only rank 0
reports.  No GPU is involved."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))     # rank 1 is the slow one
    out[rank] = (ms, bench.aggregate_tokens_per_s(256, world, ms))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_throughput_gloo_world2():
    world, port = 2, _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == 15.0 and res[1][0] == 15.0                # every rank sees the slowest rank's time
    assert abs(res[0][1] - 2 * 256 / 15e-3) < 1e-6                # both replicas' tokens over that time
    import bench
    assert bench.max_over_ranks(3.5, None, None) == 3.5           # single process: no collective


def test_reference_arm_prints_one_line_from_rank0_only_under_torchrun():
    port = _free_port()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
           "--warmup", "0", "--workload", "cfg1", "--reference-tokens", "64"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = lines[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
