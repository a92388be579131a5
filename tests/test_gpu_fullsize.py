"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: the whole
batch runs on the GPU, a sample of scenarios is recomputed by the oracle one by one, and
size-independent invariants are checked on everything."""
import numpy as np
import pytest

from workloads import POOL_GPU, generate, make_workload

pytestmark = pytest.mark.gpu

KEYS = ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us")


def _run_full(name):
    import torch
    from paper_2603_13019_b200 import binding
    w = make_workload(name)
    S, N = w.n_scenarios, w.max_actions
    chunk = max(1, (64 << 20) // N)
    parts = [generate(w, c, min(S, c + chunk)) for c in range(0, S, chunk)]
    a = {k: (None if parts[0][k] is None else np.concatenate([p[k] for p in parts], axis=1 if k.startswith("side_") else 0))
         for k in parts[0]}
    rnd = binding.Round(S, N, w.pools, depth=w.depth, cache_slots=int(w.params.get("cache_slots", 0)),
                        side_costs=int(w.params.get("side_costs", 0)))
    dev = binding.to_device(a)
    out = rnd.schedule_batch(dev)
    torch.cuda.synchronize()
    g = {k: v.cpu().numpy() for k, v in out.items()}
    if "cache_tag" in a:                                         # the cache state is updated in place
        g["cache_tag"] = dev["cache_tag"].cpu().numpy().view(np.uint32)
        g["cache_use"] = dev["cache_use"].cpu().numpy()
    rnd.destroy()
    return w, a, g


@pytest.mark.parametrize("name,n_sample", [("cfg4", 96), ("cfg1", 128), ("cfg3", 24), ("cfg4_vec", 64), ("cfg1_cache", 96)])
def test_full_size_sampled_scenarios_match_oracle(oracle, name, n_sample):
    w, a, g = _run_full(name)
    S = w.n_scenarios
    K = int(w.params.get("cache_slots", 0))
    assert np.all(g["status"] == 0)
    rng = np.random.default_rng(11)
    sample = np.unique(np.concatenate([[0, S - 1], rng.integers(0, S, n_sample)]))
    for sc in sample:
        o = oracle.schedule_batch(w.pools, a, depth=w.depth, lo=int(sc), hi=int(sc) + 1, cache_slots=K)
        for k in KEYS + (("cache_tag", "cache_use") if K else ()):
            assert np.array_equal(o[k][0], g[k][sc]), f"{name}: scenario {sc}: {k} differs"
    # invariants on every scenario: capacity per pool, totals, sentinels
    sel = g["alloc_units"] > 0
    assert np.array_equal(sel.sum(1), g["n_selected"])
    assert np.array_equal(np.where(sel, g["act_us"], 0).sum(1), g["total_act_us"])
    assert np.all(g["act_us"][~sel] == -1) and np.all(g["place_node"][~sel] == -1)
    for j, p in enumerate(w.pools):
        used = np.where(a["pool"] == j, g["alloc_units"], 0).sum(1)
        if "side_pool" in a:                                     # the further amounts of what was scheduled
            for e in range(a["side_pool"].shape[0]):
                used = used + np.where(sel & (a["side_pool"][e] == j), a["side_units"][e], 0).sum(1)
        busy = 0
        if p.type == POOL_GPU and a["gpu_busy"] is not None:
            busy = np.unpackbits(a["gpu_busy"], axis=1).sum(1)
        assert np.all(used + busy <= p.capacity)


def test_host_buffers_in_chunks_give_the_same_results():
    """A batch large enough to go through the host-buffer path in several chunks (copy-in,
    kernels and copy-out of successive chunks overlap) must equal the device-buffer run."""
    import torch
    from paper_2603_13019_b200 import binding
    w, a, g = _run_full("cfg1")                                  # 4096 x 1024: 176 MB of traffic, 2 chunks
    S, N = w.n_scenarios, w.max_actions
    rnd = binding.Round(S, N, w.pools, depth=w.depth, host_buffers=True)
    hin = binding.to_device(a, pin=True)
    for _ in range(2):                                           # twice: the staging area is reused
        out = rnd.schedule_batch(hin)
        torch.cuda.synchronize()
        for k in KEYS:
            assert np.array_equal(out[k].numpy(), g[k]), k
    rnd.destroy()
