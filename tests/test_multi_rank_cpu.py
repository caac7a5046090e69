"""The N > 1 path of bench.py on CPU: two gloo ranks.  Ranks compress independent prompts (no data-path
collective); the only exchange is the max-reduce of the step time, and the reported value is the
whole-job aggregate."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = bench.rank_workload("long_video_19k", rank, layers=2)
    ms = bench.max_over_ranks(10.0 * (rank + 1), world, "cpu")          # rank 1 is the slow one
    # every rank generates its own, different prompt from the shared recipe
    from paper_2502_17599_b200 import workloads as W
    q, _, _ = W.make_layer(wl.with_(spans=((0, 64, 0), (64, 128, 1)), frame_tokens=0, window=8), 0, "cpu")
    seeds = [None] * world
    dist.all_gather_object(seeds, (wl.seed, float(q.float().sum())))
    out.put((rank, ms, bench.whole_job_throughput(wl, world, ms), wl.n_layers, seeds))
    dist.destroy_process_group()


def test_two_ranks_shard_by_prompt_and_report_the_slowest_time():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, layers, seeds in results:
        assert ms == 20.0                                    # max over ranks, on every rank
        assert layers == 2
        assert value == world * 2 * 18944 / 20e-3            # aggregate over both ranks
        assert seeds[0][0] != seeds[1][0] and seeds[0][1] != seeds[1][1]   # different prompts
