"""Parity of the device-resident trace replay with the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from workloads import POOL_API, POOL_CPU, POOL_GPU, Pool, generate, make_workload, random_round

pytestmark = pytest.mark.gpu

KEYS = ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us",
        "rounds_used", "occupancy")


def gpu_replay(pools, a, depth, round_us, max_rounds, host_buffers=False):
    import torch
    from paper_2603_13019_b200 import binding
    S, N = a["pool"].shape
    rnd = binding.Round(S, N, pools, depth=depth, round_us=round_us, max_rounds=max_rounds,
                        host_buffers=host_buffers)
    out = rnd.replay_trace(binding.to_device(a, pin=host_buffers))
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    rnd.destroy()
    return res


def assert_same(o, g):
    for k in KEYS:
        if not np.array_equal(o[k], g[k]):
            bad = np.argwhere(o[k] != g[k])
            first = tuple(bad[0])
            raise AssertionError(
                f"{k} differs at {first}: oracle {o[k][first]} cuda {g[k][first]} ({len(bad)} mismatches)")


def test_cfg2_shape_matches_oracle(oracle):
    w = make_workload("cfg2", n_scenarios=12, max_actions=900)
    a = generate(w)
    max_rounds = 3000
    o = oracle.replay_trace(w.pools, a, depth=w.depth, round_us=w.round_us, max_rounds=max_rounds)
    g = gpu_replay(w.pools, a, w.depth, w.round_us, max_rounds)
    assert_same(o, g)
    assert np.all(g["status"] == 0) and np.all(g["n_selected"] == 900)
    assert_same(o, gpu_replay(w.pools, a, w.depth, w.round_us, max_rounds, host_buffers=True))


POOLSETS = [
    (Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 16, 8), Pool(POOL_API, 5, 0, 200_000)),
    (Pool(POOL_GPU, 24, 8),),
    (Pool(POOL_CPU, 40, 8), Pool(POOL_GPU, 8, 4), Pool(POOL_API, 3, 0, 0)),
]


@pytest.mark.parametrize("seed", range(6))
def test_random_traces_match_oracle(oracle, seed):
    pools = POOLSETS[seed % len(POOLSETS)]
    N = 120
    w, a = random_round(700 + seed, 16, N, pools, small_durations=0.2, busy_fraction=0.25 if seed % 2 else 0.0,
                        max_mult=4)
    rng = np.random.default_rng(seed)
    # bursts: arrivals every ~2 ms on average while actions last up to 0.5 s
    a["arrival_us"] = np.cumsum(rng.integers(0, 4000, a["pool"].shape), axis=1).astype(np.int64)
    for depth, max_rounds in ((2, 4000), (1, 40)):
        o = oracle.replay_trace(pools, a, depth=depth, round_us=10_000, max_rounds=max_rounds)
        g = gpu_replay(pools, a, depth, 10_000, max_rounds)
        assert_same(o, g)
    assert o["n_selected"].sum() > 0


def test_replay_flags_bad_input(oracle):
    pools = (Pool(POOL_CPU, 8, 4),)
    w, a = random_round(5, 4, 10, pools, ragged=False)
    a["arrival_us"] = np.cumsum(np.full(a["pool"].shape, 1000), axis=1).astype(np.int64)
    a["arrival_us"][1, 3] = 0                       # not sorted
    a["level_mask"][2, 0] = 0                       # no usable level
    o = oracle.replay_trace(pools, a, depth=2, round_us=10_000, max_rounds=200)
    g = gpu_replay(pools, a, 2, 10_000, 200)
    assert_same(o, g)
    assert list(g["status"]) == [0, 2, 1, 0]


def test_cfg2_full_size_sampled_scenarios_match_oracle(oracle):
    # the whole 256 x 20000 trace on the GPU; eight scenarios recomputed by the oracle, everything compared
    w = make_workload("cfg2")
    a = generate(w)
    g = gpu_replay(w.pools, a, w.depth, w.round_us, w.max_rounds)
    assert np.all(g["status"] == 0) and np.all(g["n_selected"] == w.max_actions)
    rng = np.random.default_rng(3)
    for sc in np.unique(np.concatenate([[0, w.n_scenarios - 1], rng.integers(0, w.n_scenarios, 6)])):
        o = oracle.replay_trace(w.pools, a, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds,
                                lo=int(sc), hi=int(sc) + 1)
        for k in KEYS:
            assert np.array_equal(o[k][0], g[k][sc]), f"scenario {sc}: {k} differs"
    # conservation on every scenario: each action ran once, with a legal allocation
    assert np.all(g["alloc_units"] > 0) and np.all(g["act_us"] >= 0)
    assert np.array_equal(g["act_us"].sum(1), g["total_act_us"])


def test_long_running_sets_match_oracle(oracle):
    # a burst of long single-core actions on a pool of 600 cores: more than 448 actions run at once,
    # so the completion heap of the estimates outgrows the warp's shared-memory tree
    pools = (Pool(POOL_CPU, 600, 60),)
    S, N = 4, 1400
    rng = np.random.default_rng(17)
    elastic = rng.random((S, N)) < 0.3
    a = dict(pool=np.zeros((S, N), np.uint8), unit=np.ones((S, N), np.uint8),
             level_mask=np.where(elastic, 0xB, 1).astype(np.uint32),
             s_us=rng.integers(200_000, 900_000, (S, N)).astype(np.int64),
             p_us=np.where(elastic, rng.integers(0, 2_000_000, (S, N)), 0).astype(np.int64),
             arrival_us=np.cumsum(rng.integers(0, 600, (S, N)), axis=1).astype(np.int64),
             n_actions=np.full(S, N, np.int32), gpu_busy=None)
    o = oracle.replay_trace(pools, a, depth=2, round_us=10_000, max_rounds=600)
    g = gpu_replay(pools, a, 2, 10_000, 600)
    assert_same(o, g)
    assert o["occupancy"][:, :, 0].max() > 448 and np.all(o["n_selected"] == N)
