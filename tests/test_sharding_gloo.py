"""Multi-process host logic of the replica/sharded run (scenarios are independent, so ranks
share nothing but the final timing reduction): two gloo ranks on CPU generate their own
scenario ranges from the global scenario ids, schedule them, and the gathered result equals
the single-process result; the step time is the maximum over ranks."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, per_rank, out_dir):
    sys.path.insert(0, ROOT)
    import oracle
    from workloads import generate, make_workload
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = make_workload("cfg1", n_scenarios=per_rank * world)
    lo = rank * per_rank                                   # seed = base + global scenario id
    a = generate(w, lo, lo + per_rank)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    mine = torch.from_numpy(o["n_selected"].astype(np.int64))
    gathered = [torch.zeros_like(mine) for _ in range(world)]
    dist.all_gather(gathered, mine)
    t = torch.tensor([10.0 + rank], dtype=torch.float64)  # each rank's "step time"
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    if rank == 0:
        np.save(os.path.join(out_dir, "nsel.npy"), torch.cat(gathered).numpy())
        np.save(os.path.join(out_dir, "tmax.npy"), t.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_cover_the_scenarios_once(tmp_path, oracle):
    from workloads import generate, make_workload
    world, per_rank = 2, 3
    mp.spawn(_worker, args=(world, 29611, per_rank, str(tmp_path)), nprocs=world, join=True)
    w = make_workload("cfg1", n_scenarios=world * per_rank)
    whole = oracle.schedule_batch(w.pools, generate(w), depth=w.depth)
    assert np.array_equal(np.load(tmp_path / "nsel.npy"), whole["n_selected"])
    assert np.load(tmp_path / "tmax.npy")[0] == 11.0
