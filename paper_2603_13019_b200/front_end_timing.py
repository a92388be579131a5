"""Device times of the queue front ends on the large mixed configuration: the sort of every queue
(Section 4.2, other queue orders), the whole round on the sorted queue, and the pinning of trajectories
to CPU nodes (Section 5.2).

    python -m paper_2603_13019_b200.front_end_timing [--scenarios 16384] [--steps 20]

Prints one JSON line.  Needs a GPU; there is no CPU path."""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def _timed(fn, steps, torch):
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def main():
    import numpy as np
    import torch
    from paper_2603_13019_b200 import binding, build
    from workloads import POOL_CPU, POOL_GPU, Pool, add_trajectories, generate, make_workload

    ap = argparse.ArgumentParser()
    ap.add_argument("--scenarios", type=int, default=16384)
    ap.add_argument("--steps", type=int, default=20)
    args = ap.parse_args()
    build.build()
    w = make_workload("cfg4", n_scenarios=args.scenarios)
    S, N = w.n_scenarios, w.max_actions
    chunk = max(1, min(S, (64 << 20) // N))
    parts = [generate(w, c, min(S, c + chunk)) for c in range(0, S, chunk)]
    a = {k: (None if parts[0][k] is None else np.concatenate([p[k] for p in parts])) for k in parts[0]}
    dev = binding.to_device(a)
    rnd = binding.Round(S, N, w.pools, depth=w.depth)
    res = rnd.new_result()
    out = {"workload": "cfg4", "scenarios": S, "actions_per_scenario": N, "steps": args.steps}
    out["round_ms"] = _timed(lambda: rnd.schedule_batch(dev, 0, res), args.steps, torch)
    for policy, name in ((1, "shortest"), (3, "arrival")):
        out["sort_%s_ms" % name] = _timed(lambda: rnd.order_queue(dev, policy), args.steps, torch)
        out["ordered_round_%s_ms" % name] = _timed(lambda: rnd.schedule_batch_ordered(dev, policy, 0, res), args.steps, torch)
    rnd.destroy()
    # per-node CPU scheduling: the core pool of cfg4 as eight nodes of 1024 cores, the GPU pool beside them
    pools = tuple(Pool(POOL_CPU, 1024, 64) for _ in range(7)) + (Pool(POOL_GPU, 128, 8),)
    b = dict(a, pool=np.where(a["pool"] == 1, 7, 0).astype(np.uint8))
    b = add_trajectories(1, b, pools, max_traj=1024, mem_hi=16, pinned=0.5, mem_free_hi=20000)
    devb = binding.to_device(b)
    devb["traj_mem"] = devb["traj_mem"].view(torch.int32)
    state = (devb["traj_node"].clone(), devb["node_mem_free"].clone())
    rnd = binding.Round(S, N, pools, depth=w.depth)

    def pin():
        devb["traj_node"].copy_(state[0]); devb["node_mem_free"].copy_(state[1])
        return rnd.pin_trajectories(devb)

    def reset_only():
        devb["traj_node"].copy_(state[0]); devb["node_mem_free"].copy_(state[1])

    out["pin_ms"] = _timed(pin, args.steps, torch) - _timed(reset_only, args.steps, torch)
    out["pin_bytes_per_action"] = 1 + 4 + 4 + 4 + 1 + 1      # pool, trajectory, memory, mask, unit in; pool out
    out["pin_gbs"] = out["pin_bytes_per_action"] * S * N / (out["pin_ms"] * 1e-3) / 1e9
    rnd.destroy()
    print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
