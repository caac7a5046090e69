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


def _shard_rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import numpy as np
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import meda_oracle as O
    from paper_2502_17599_b200 import workloads as W
    from paper_2502_17599_b200.pipeline import exchange_entropies, owned_layers
    wl = W.small_variant("shard_by_layer", n_layers=5, seed=9)
    mod = wl.modality().numpy()
    mine = owned_layers(wl.n_layers, rank, world)
    # this rank's layers only; the others stay zero, as in the device buffer before the exchange
    ent = torch.zeros(wl.n_layers, dtype=torch.float32)
    for l in mine:
        q, k, _ = (t.to(torch.float64).numpy() for t in W.make_layer(wl, l, "cpu"))
        ent[l] = float(np.float32(O.cross_modal_entropy(q, k, mod)))
    exchange_entropies(ent)                                   # the pass's only collective (Eq. 7 couples the layers)
    budgets = O.allocate_budgets(ent.numpy().astype(np.float64), wl.global_budget, wl.n_tokens, wl.min_budget)
    out.put((rank, mine, ent.tolist(), budgets.tolist()))
    dist.destroy_process_group()


def test_two_ranks_shard_one_prompt_by_layer_and_agree_on_the_budgets():
    """One prompt, layers dealt round-robin to two gloo ranks: after the single exchange of the entropies both
    ranks hold the same vector, bit for bit, and so compute identical budgets, equal to a single process's."""
    import numpy as np
    sys.path.insert(0, ROOT)
    from oracle import meda_oracle as O
    from paper_2502_17599_b200 import workloads as W
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_shard_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, mine0, ent0, b0), (_, mine1, ent1, b1) = results
    wl = W.small_variant("shard_by_layer", n_layers=5, seed=9)
    assert sorted(mine0 + mine1) == list(range(wl.n_layers)) and not set(mine0) & set(mine1)
    assert ent0 == ent1 and b0 == b1
    mod = wl.modality().numpy()
    whole = []
    for l in range(wl.n_layers):
        q, k, _ = (t.to(torch.float64).numpy() for t in W.make_layer(wl, l, "cpu"))
        whole.append(float(np.float32(O.cross_modal_entropy(q, k, mod))))
    assert whole == ent0
    want = O.allocate_budgets(np.array(whole, dtype=np.float64), wl.global_budget, wl.n_tokens, wl.min_budget)
    assert want.tolist() == b0 and int(want[:, 0].sum()) == wl.global_budget
