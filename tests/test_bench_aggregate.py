"""The benchmark's multi-rank path on CPU: two gloo ranks, replicas only.  Each
rank reports its own device time; the job's time is the slowest rank's and the
work is the sum over ranks."""
import os
import socket

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
