"""The benchmark's multi-rank path on CPU: two gloo ranks, replicas only.  Each
rank reports its own device time; the job's time is the slowest rank's and the
work is the sum over ranks."""
import json
import os
import socket
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 20.0 - 3.0 * rank]          # rank 1 is slower on the first timing
    red = bench.reduce_max(mine, dist, "cpu")
    dist.barrier()
    if rank == 0:
        out.put(red)
    dist.destroy_process_group()


def test_two_rank_max_over_ranks_and_whole_job_value():
    ctx = mp.get_context("spawn")
    out = ctx.SimpleQueue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    red = out.get()
    assert red == [15.0, 20.0]
    one = bench.whole_job_tflops(1, 20, bench.attn_flops(bench.WL), 15.0)
    two = bench.whole_job_tflops(2, 20, bench.attn_flops(bench.WL), 15.0)
    assert abs(two - 2 * one) < 1e-9 and abs(one - 20 * 5.3831e11 / 15e-3 / 1e12) / one < 1e-3


def test_single_rank_reduce_is_identity():
    assert bench.reduce_max([1.5, 2.5], None) == [1.5, 2.5]


def test_gpus_flag_starts_the_ranks_itself():
    """`bench.py --gpus 2` without a launcher around it starts two ranks (here on CPU, gloo,
    with made-up device times) and prints one line for the whole job: the slowest rank's time,
    the work of both."""
    env = {k: v for k, v in os.environ.items()
           if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    root = os.path.dirname(os.path.abspath(bench.__file__))
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "5", "--dry-run"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["n_gpus"] == 2 and line["dry_run"] is True
    assert abs(line["ms_per_step"] - 11.0 / 5) < 1e-9                 # rank 1 reported 11 ms, rank 0 10 ms
    assert abs(line["value"] - bench.whole_job_tflops(2, 5, bench.attn_flops(bench.WL), 11.0)) < 1e-9
