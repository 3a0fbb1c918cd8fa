"""The N > 1 path of the benchmark on CPU: two gloo ranks own different layers (no data-path collective) and
the whole-job figures are MAX of time and SUM of work over ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ids = bench.layer_ids_for_rank(rank, 3)
    ms, fl = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100.0 * (rank + 1), world, "cpu")
    # every rank draws different inputs for "its" layers: check on a tiny layer shape
    from paper_2506_11104_b200 import synth
    w = synth.llama_layer(256, 128, 1, ids[0], "cpu")
    sig = float(w.Q.float().abs().sum())
    gathered = [None] * world
    dist.all_gather_object(gathered, (ids, ms, fl, sig))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharding_and_aggregation():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (ids0, ms0, fl0, sig0), (ids1, ms1, fl1, sig1) = res
    assert set(ids0).isdisjoint(ids1)
    assert ms0 == ms1 == 15.0            # max over ranks
    assert fl0 == fl1 == 300.0           # sum over ranks
    assert sig0 != sig1                  # different seeds -> different inputs per rank
