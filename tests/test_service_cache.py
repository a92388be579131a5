"""Service cache of the GPU pools (Section 5.3, evict on execution): chunk preference, LRU entries,
restoration time.  The pins below are worked by hand from the rules; the GPU tests compare the CUDA
path with the oracle on random rounds and traces with a cache."""
import numpy as np
import pytest

from workloads import POOL_CPU, POOL_GPU, Pool, random_round

GANG = 0x80
NONE = 0xFFFF


def tag(service, size):
    """Instance tag as the interface defines it: (service * 8 + log2(chunk size)) + 1; 0 = empty."""
    return (service << 3 | int(np.log2(size))) + 1


def _arrays(rows, nodes, slots, cache=None, arrival=None):
    """rows: (unit, mask, s, p, service, restore) on a single GPU pool of `nodes` nodes of 8."""
    n = len(rows)
    a = dict(pool=np.zeros((1, n), np.uint8), unit=np.array([[r[0] for r in rows]], np.uint8),
             level_mask=np.array([[r[1] for r in rows]], np.uint32), s_us=np.array([[r[2] for r in rows]], np.int64),
             p_us=np.array([[r[3] for r in rows]], np.int64),
             arrival_us=None if arrival is None else np.array([arrival], np.int64),
             n_actions=np.array([n], np.int32), gpu_busy=np.zeros((1, nodes), np.uint8),
             service=np.array([[r[4] for r in rows]], np.uint16), restore_us=np.array([[r[5] for r in rows]], np.int64),
             cache_tag=np.zeros((1, nodes * 8 * slots), np.uint32), cache_use=np.zeros((1, nodes * 8 * slots), np.int64))
    for (node, gpu, slot), (tg, use) in (cache or {}).items():
        a["cache_tag"][0, (node * 8 + gpu) * slots + slot] = tg
        a["cache_use"][0, (node * 8 + gpu) * slots + slot] = use
    return a


def test_same_level_blocks_prefer_the_one_that_caches_the_instance(oracle):
    pools = [Pool(POOL_GPU, 16, 8)]
    row = [(2 | GANG, 1, 100, 0, 7, 5000)]                        # one chunk of 2 GPUs, service 7, runs 100 us
    # both nodes are free (one block of 8 each: the same level).  GPUs 0-1 of node 1 hold (7, 2):
    # the chunk that node 1's block would give, its low end, caches the instance -> node 1, no restoration
    a = _arrays(row, 2, 1, {(1, 0, 0): (tag(7, 2), 3), (1, 1, 0): (tag(7, 2), 3)})
    o = oracle.schedule_batch(pools, a, cache_slots=1, now_us=50)
    assert (o["place_node"][0, 0], o["place_off"][0, 0], o["act_us"][0, 0]) == (1, 0, 50 + 100)
    # cached on GPUs 2-3 of node 1 instead: the granted chunk would be GPUs 0-1, which do not hold it,
    # so nothing is preferred: node 0, and the instance is restored first (5000 us)
    a = _arrays(row, 2, 1, {(1, 2, 0): (tag(7, 2), 3), (1, 3, 0): (tag(7, 2), 3)})
    o = oracle.schedule_batch(pools, a, cache_slots=1, now_us=50)
    assert (o["place_node"][0, 0], o["place_off"][0, 0], o["act_us"][0, 0]) == (0, 0, 50 + 100 + 5000)
    assert o["cache_tag"][0, 0] == tag(7, 2) and o["cache_use"][0, 0] == 50      # now cached where it ran
    # another degree of parallelism of the same service is another instance: (7, 4) cached, (7, 2) asked
    a = _arrays(row, 2, 1, {(1, g, 0): (tag(7, 4), 3) for g in range(4)})
    o = oracle.schedule_batch(pools, a, cache_slots=1)
    assert (o["place_node"][0, 0], o["act_us"][0, 0]) == (0, 100 + 5000)
    # an action without a service never pays a restoration
    o = oracle.schedule_batch(pools, _arrays([(2 | GANG, 1, 100, 0, NONE, 5000)], 2, 1), cache_slots=1)
    assert (o["place_node"][0, 0], o["act_us"][0, 0]) == (0, 100)


def test_the_smallest_sufficient_level_comes_before_the_cache(oracle):
    # node 0 has one free block of 2 GPUs (2-3), node 1 is free and caches the instance on its low end:
    # the allocation takes the smallest sufficient chunk first (level 1 on node 0), the cache only
    # chooses among chunks of that level
    pools = [Pool(POOL_GPU, 16, 8)]
    a = _arrays([(2 | GANG, 1, 100, 0, 7, 5000)], 2, 1, {(1, 0, 0): (tag(7, 2), 3), (1, 1, 0): (tag(7, 2), 3)})
    a["gpu_busy"][0, 0] = 0xF3
    o = oracle.schedule_batch(pools, a, cache_slots=1)
    assert (o["place_node"][0, 0], o["place_off"][0, 0], o["act_us"][0, 0]) == (0, 2, 100 + 5000)


def test_least_recently_used_entry_is_replaced(oracle):
    pools = [Pool(POOL_GPU, 8, 8)]
    A, B, C = tag(1, 1), tag(2, 1), tag(3, 1)
    busy = 0xFE                                                    # only GPU 0 is free
    def run(rows, cache, now):
        a = _arrays(rows, 1, 2, cache)
        a["gpu_busy"][0, 0] = busy
        return oracle.schedule_batch(pools, a, cache_slots=2, now_us=now)
    # GPU 0 remembers A (used at 10) and B (used at 20); C arrives at 30: A, the older one, goes
    o = run([(1, 1, 7, 0, 3, 900)], {(0, 0, 0): (A, 10), (0, 0, 1): (B, 20)}, 30)
    assert o["act_us"][0, 0] == 30 + 7 + 900                      # waited 30 (arrival 0), restored, ran
    assert list(o["cache_tag"][0, :2]) == [C, B] and list(o["cache_use"][0, :2]) == [30, 20]
    # B is asked again at 40: a hit, no restoration, its use is refreshed
    o = run([(1, 1, 7, 0, 2, 900)], {(0, 0, 0): (A, 10), (0, 0, 1): (B, 20)}, 40)
    assert o["act_us"][0, 0] == 40 + 7
    assert list(o["cache_tag"][0, :2]) == [A, B] and list(o["cache_use"][0, :2]) == [10, 40]
    # an empty entry is filled before anything is evicted; equal uses: the lower entry goes
    o = run([(1, 1, 7, 0, 3, 900)], {(0, 0, 1): (B, 20)}, 30)
    assert list(o["cache_tag"][0, :2]) == [C, B]
    o = run([(1, 1, 7, 0, 3, 900)], {(0, 0, 0): (A, 20), (0, 0, 1): (B, 20)}, 30)
    assert list(o["cache_tag"][0, :2]) == [C, B]


def test_one_missed_replica_costs_one_restoration(oracle):
    # two replicas of one GPU each; GPU 0 caches the instance, GPU 1 does not: restored once
    pools = [Pool(POOL_GPU, 8, 8)]
    a = _arrays([(1, 0b10, 100, 0, 4, 700)], 1, 1, {(0, 0, 0): (tag(4, 1), 1)})
    a["gpu_busy"][0, 0] = 0xFC
    o = oracle.schedule_batch(pools, a, cache_slots=1)
    assert o["alloc_units"][0, 0] == 2 and o["act_us"][0, 0] == 100 + 700
    assert list(o["cache_tag"][0, :2]) == [tag(4, 1), tag(4, 1)]


def test_replay_keeps_the_instance_cached_after_the_action(oracle):
    # rounds every 1000 us, one node.  x asks for (5, 4) at t = 0: miss, runs 300 + 2000 on GPUs 0-3.
    # y, the same instance, arrives at 2500 and is scheduled at 3000: x is gone, GPUs 0-3 still hold the
    # instance (the block of 8 is free again and its low end caches it): hit, 300 us.
    # z asks for (6, 4) at 3000 too: it gets GPUs 4-7 (what is left), a miss.
    pools = [Pool(POOL_GPU, 8, 8)]
    rows = [(4 | GANG, 1, 300, 0, 5, 2000), (4 | GANG, 1, 300, 0, 5, 2000), (4 | GANG, 1, 300, 0, 6, 2000)]
    a = _arrays(rows, 1, 1, arrival=[0, 2500, 2600])
    o = oracle.replay_trace(pools, a, round_us=1000, max_rounds=20, cache_slots=1)
    assert list(o["act_us"][0]) == [2300, 500 + 300, 400 + 2300]
    assert list(o["place_off"][0]) == [0, 0, 4]
    assert list(o["cache_tag"][0, :8]) == [tag(5, 4)] * 4 + [tag(6, 4)] * 4
    assert list(o["cache_use"][0, :8]) == [3000] * 8
    assert o["rounds_used"][0] == 7                               # z finishes at 3000 + 2300 = 5300 -> round 6 is the last busy one


# ------------------------------------------------------------------ CUDA path against the oracle
def _with_services(seed, a, pools, slots, n_services=5):
    """Adds services, restoration times and a random cache state to a round's arrays (input generator only)."""
    rng = np.random.default_rng(seed)
    S, N = a["pool"].shape
    nodes = sum(p.capacity // p.group for p in pools if p.type == POOL_GPU)
    a = dict(a)
    a["service"] = np.where(rng.random((S, N)) < 0.85, rng.integers(0, n_services, (S, N)), NONE).astype(np.uint16)
    a["restore_us"] = rng.integers(0, 300_000, (S, N)).astype(np.int64)
    sv = rng.integers(0, n_services, (S, nodes * 8 * slots))
    sz = rng.integers(0, 4, (S, nodes * 8 * slots))
    a["cache_tag"] = np.where(rng.random((S, nodes * 8 * slots)) < 0.7, (sv << 3 | sz) + 1, 0).astype(np.uint32)
    a["cache_use"] = rng.integers(-50, 50, (S, nodes * 8 * slots)).astype(np.int64)
    return a


CACHE_KEYS = ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us",
              "cache_tag", "cache_use")


@pytest.mark.gpu
@pytest.mark.parametrize("seed,slots", [(0, 1), (1, 2), (2, 4), (3, 2)])
def test_rounds_with_a_service_cache_match_oracle(oracle, seed, slots):
    import torch
    from paper_2603_13019_b200 import binding
    pools = [(Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 32, 8)), (Pool(POOL_GPU, 64, 8),),
             (Pool(POOL_GPU, 16, 4), Pool(POOL_GPU, 24, 8)), (Pool(POOL_GPU, 8 * 70, 8),)][seed]
    w, a = random_round(9100 + seed, 48, [60, 90, 40, 700][seed], pools, busy_fraction=0.3, max_mult=4,
                        replicas=0.5, small_durations=0.3 if seed == 1 else 0.0)
    a = _with_services(seed, a, pools, slots)
    o = oracle.schedule_batch(pools, a, cache_slots=slots, now_us=100)
    S, N = a["pool"].shape
    rnd = binding.Round(S, N, pools, cache_slots=slots)
    dev = binding.to_device(a)
    out = rnd.schedule_batch(dev, now_us=100)
    torch.cuda.synchronize()
    g = {k: v.cpu().numpy() for k, v in out.items()}
    g["cache_tag"] = dev["cache_tag"].cpu().numpy().view(np.uint32)
    g["cache_use"] = dev["cache_use"].cpu().numpy()
    rnd.destroy()
    for k in CACHE_KEYS:
        assert np.array_equal(o[k], g[k]), k
    sel = o["alloc_units"] > 0
    assert sel.sum() > 50


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(3))
def test_traces_with_a_service_cache_match_oracle(oracle, seed):
    import torch
    from paper_2603_13019_b200 import binding
    pools = [(Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 32, 8)), (Pool(POOL_GPU, 40, 8),),
             (Pool(POOL_GPU, 16, 4), Pool(POOL_GPU, 32, 8))][seed]
    slots = [1, 2, 3][seed]
    w, a = random_round(9200 + seed, 12, 150, pools, max_mult=4, replicas=0.5, busy_fraction=0.0)
    rng = np.random.default_rng(seed)
    a["arrival_us"] = np.cumsum(rng.integers(0, 6000, a["pool"].shape), axis=1).astype(np.int64)
    a = _with_services(seed, a, pools, slots, n_services=3)
    o = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=6000, cache_slots=slots)
    rnd = binding.Round(12, 150, pools, round_us=10_000, max_rounds=6000, cache_slots=slots)
    dev = binding.to_device(a)
    out = rnd.replay_trace(dev)
    torch.cuda.synchronize()
    g = {k: v.cpu().numpy() for k, v in out.items()}
    g["cache_tag"] = dev["cache_tag"].cpu().numpy().view(np.uint32)
    g["cache_use"] = dev["cache_use"].cpu().numpy()
    rnd.destroy()
    for k in CACHE_KEYS + ("rounds_used", "occupancy"):
        assert np.array_equal(o[k], g[k]), k
    assert (o["alloc_units"] > 0).sum() > 800 and np.all(o["status"] == 0)


@pytest.mark.gpu
def test_cfg1_with_a_service_cache_matches_oracle(oracle):
    import torch
    from paper_2603_13019_b200 import binding
    from workloads import generate, make_workload
    w = make_workload("cfg1_cache", n_scenarios=96)
    a = generate(w)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth, cache_slots=2)
    rnd = binding.Round(96, w.max_actions, w.pools, depth=w.depth, cache_slots=2)
    dev = binding.to_device(a)
    out = rnd.schedule_batch(dev)
    torch.cuda.synchronize()
    g = {k: v.cpu().numpy() for k, v in out.items()}
    g["cache_tag"] = dev["cache_tag"].cpu().numpy().view(np.uint32)
    g["cache_use"] = dev["cache_use"].cpu().numpy()
    rnd.destroy()
    for k in CACHE_KEYS:
        assert np.array_equal(o[k], g[k]), k
