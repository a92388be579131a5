"""Parity of the CUDA path with the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest

from workloads import (POOL_API, POOL_CPU, POOL_GPU, Pool, contiguous_replica_round, generate, make_workload,
                       random_round)

pytestmark = pytest.mark.gpu

OUT_KEYS = ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us")


def gpu_round(pools, a, depth=2, now_us=0, host_buffers=False):
    import torch
    from paper_2603_13019_b200 import binding
    S, N = a["pool"].shape
    rnd = binding.Round(S, N, pools, depth=depth, host_buffers=host_buffers)
    t = binding.to_device(a, pin=host_buffers)
    out = rnd.schedule_batch(t, now_us=now_us)
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    rnd.destroy()
    return res


def assert_same(o, g):
    for k in OUT_KEYS:
        if not np.array_equal(o[k], g[k]):
            bad = np.argwhere(o[k] != g[k])
            first = tuple(bad[0])
            raise AssertionError(
                f"{k} differs at {first}: oracle {o[k][first]} cuda {g[k][first]} ({len(bad)} mismatches)")


@pytest.mark.parametrize("name,S", [("cfg0", 1), ("cfg1", 96), ("cfg3", 48), ("cfg4", 24)])
def test_named_configs_match_oracle(oracle, name, S):
    w = make_workload(name, n_scenarios=S)
    a = generate(w)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    g = gpu_round(w.pools, a, depth=w.depth)
    assert_same(o, g)
    assert np.all(g["status"] == 0)


POOLSETS = [
    (Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 16, 8), Pool(POOL_API, 5, 0, 1_000_000)),
    (Pool(POOL_GPU, 24, 8),),
    (Pool(POOL_CPU, 40, 8), Pool(POOL_GPU, 8, 4)),
    (Pool(POOL_CPU, 6, 2), Pool(POOL_API, 3, 0, 0)),
    (Pool(POOL_CPU, 320, 64), Pool(POOL_GPU, 64, 8), Pool(POOL_GPU, 6, 2), Pool(POOL_API, 40, 0, 1000)),
]


@pytest.mark.parametrize("seed", range(15))
def test_random_rounds_match_oracle(oracle, seed):
    pools = POOLSETS[seed % len(POOLSETS)]
    N = [40, 77, 300][seed % 3]
    w, a = random_round(500 + seed, 64, N, pools, small_durations=0.4 if seed % 2 else 0.0,
                        busy_fraction=0.3 if seed % 3 == 0 else 0.0, max_mult=[8, 4, 12][seed % 3])
    for depth, now in ((2, 12345), (1, 0), (3, 7)):
        o = oracle.schedule_batch(pools, a, depth=depth, now_us=now)
        g = gpu_round(pools, a, depth=depth, now_us=now)
        assert_same(o, g)


def test_ties_everywhere_match_oracle(oracle):
    # durations so small that many allocations tie on the duration sum
    pools = (Pool(POOL_CPU, 12, 4), Pool(POOL_GPU, 16, 8))
    w, a = random_round(901, 128, 24, pools, small_durations=1.0, busy_fraction=0.25, inelastic=0.1)
    o = oracle.schedule_batch(pools, a)
    g = gpu_round(pools, a)
    assert_same(o, g)


def test_edge_cases_match_oracle(oracle):
    pools = (Pool(POOL_CPU, 8, 4), Pool(POOL_GPU, 8, 8))
    w, a = random_round(77, 8, 16, pools)
    a["n_actions"][:] = [0, 1, 16, 16, 3, 16, 16, 2]
    a["level_mask"][3, 5] = 0                      # no usable level -> bad scenario
    a["pool"][5, 0] = 7                            # unknown pool -> bad scenario
    a["unit"][6, :] = 1                            # GPU actions become single-GPU replicas
    a["s_us"][2, :] = -5                           # clamped to 0
    a["p_us"][2, 0] = 1 << 50                      # clamped to 2^40
    o = oracle.schedule_batch(pools, a)
    g = gpu_round(pools, a)
    assert_same(o, g)
    assert list(g["status"][[3, 5]]) == [1, 1] and g["n_selected"][0] == 0


def test_arrivals_and_host_buffers_match_oracle(oracle):
    w = make_workload("cfg1", n_scenarios=16)
    a = generate(w)
    rng = np.random.default_rng(5)
    a["arrival_us"] = np.sort(rng.integers(0, 50_000, a["pool"].shape), axis=1).astype(np.int64)
    o = oracle.schedule_batch(w.pools, a, now_us=60_000)
    assert_same(o, gpu_round(w.pools, a, now_us=60_000))
    assert_same(o, gpu_round(w.pools, a, now_us=60_000, host_buffers=True))


def test_long_queue_spans_several_tiles(oracle):
    # 9000 actions per scenario: the prefix kernel walks three tiles with carried prefix sums
    pools = (Pool(POOL_CPU, 3008, 64), Pool(POOL_GPU, 512, 8), Pool(POOL_API, 2000, 0, 1_000_000))
    w, a = random_round(31, 6, 9000, pools, max_mult=4, ragged=False)
    a["n_actions"][:] = [9000, 8191, 4097, 4096, 100, 9000]
    o = oracle.schedule_batch(pools, a)
    g = gpu_round(pools, a)
    assert_same(o, g)
    assert o["n_selected"].max() > 300


@pytest.mark.parametrize("ties", [0.0, 0.6, 1.0])
def test_fragmented_gpu_pool_of_replica_requests_matches_oracle(oracle, ties):
    # replica requests only (no gang rows) on a fragmented pool: the per-size DPs merged through the
    # nested capacities; with tiny durations different splits tie and the general loop takes over
    pools = (Pool(POOL_GPU, 192, 8),)
    w, a = random_round(4242 + int(ties * 10), 48, 220, pools, replicas=1.0, busy_fraction=0.35,
                        small_durations=ties, inelastic=0.2, max_mult=4)
    for depth in (1, 2):
        o = oracle.schedule_batch(pools, a, depth=depth)
        g = gpu_round(pools, a, depth=depth)
        assert_same(o, g)
    assert o["n_selected"].max() > 20


def test_pools_beyond_the_thread_per_pool_placement_match_oracle(oracle):
    # 160 NUMA domains and 72 GPU nodes: these pools are placed by the warp-per-pool routines
    pools = (Pool(POOL_CPU, 160 * 4, 4), Pool(POOL_GPU, 72 * 8, 8), Pool(POOL_API, 50, 0, 1_000_000))
    w, a = random_round(77, 24, 700, pools, busy_fraction=0.2, max_mult=6, replicas=1.0)
    o = oracle.schedule_batch(pools, a)
    g = gpu_round(pools, a)
    assert_same(o, g)
    assert o["n_selected"].max() > 100


def test_invalid_record_far_behind_the_prefix_matches_oracle(oracle):
    # the record is found by the streaming kernel while the scenario's pools are being decided
    w = make_workload("cfg1", n_scenarios=12)
    a = generate(w)
    a["level_mask"][3, 900] = 0
    a["pool"][7, 1023] = 9
    a["unit"][9, 600] = 0
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    g = gpu_round(w.pools, a, depth=w.depth)
    assert_same(o, g)
    assert list(g["status"][[3, 7, 9]]) == [1, 1, 1] and g["n_selected"][3] == 0


def test_saturating_objectives_match_oracle(oracle):
    # queues of identical actions with s = p = 2^40: the completion times leave the 49 bits of the packed
    # simulation keys, and the sums of the longer queues pass 2^63 and are clamped
    pools = (Pool(POOL_CPU, 2, 2),)
    S, N = 6, 6000
    a = dict(pool=np.zeros((S, N), np.uint8), unit=np.ones((S, N), np.uint8),
             level_mask=np.full((S, N), 3, np.uint32), s_us=np.full((S, N), 1 << 40, np.int64),
             p_us=np.full((S, N), 1 << 40, np.int64), arrival_us=None,
             n_actions=np.array([3500, 6000, 40, 2900, 3000, 4096], np.int32), gpu_busy=None)
    a["s_us"][5, :] = 0                                # s < p / 2: the eviction pays while nothing saturates
    a["n_actions"][5] = 2
    for depth in (1, 2):
        o = oracle.schedule_batch(pools, a, depth=depth)
        g = gpu_round(pools, a, depth=depth)
        assert_same(o, g)
    assert list(o["alloc_units"][0][:2]) == [1, 1] and list(o["alloc_units"][5][:2]) == [2, 0]


@pytest.mark.parametrize("seed", range(6))
def test_unnarrowed_random_rounds_match_oracle(oracle, seed):
    # replica requests with up to 32 multiplicities, gang masks with unusable levels among usable ones,
    # elastic quota actions, a few invalid records
    pools = POOLSETS[seed % len(POOLSETS)]
    w, a = random_round(800 + seed, 96, [60, 150][seed % 2], pools, narrow=False, max_mult=[32, 12, 6][seed % 3],
                        small_durations=0.5 if seed % 2 else 0.0, busy_fraction=0.3 if seed % 3 == 0 else 0.0)
    for depth in (2, 1):
        o = oracle.schedule_batch(pools, a, depth=depth)
        g = gpu_round(pools, a, depth=depth)
        assert_same(o, g)
    assert (o["status"] == 0).sum() > 10


@pytest.mark.parametrize("seed,nodes", [(0, 32), (1, 40), (2, 64)])
def test_fragmented_pool_with_elastic_gang_requests_matches_oracle(oracle, seed, nodes):
    # gang requests (one chunk that grows with the level) couple the chunk sizes, so the per-size
    # decomposition does not apply; mixed with replica requests on a fragmented pool of many nodes
    pools = (Pool(POOL_GPU, 8 * nodes, 8),)
    w, a = random_round(6100 + seed, 10, 260, pools, replicas=0.5, busy_fraction=0.35, inelastic=0.2,
                        max_mult=8, small_durations=0.3 if seed == 1 else 0.0)
    o = oracle.schedule_batch(pools, a)
    g = gpu_round(pools, a)
    assert_same(o, g)
    assert np.all(g["status"] == 0) and o["n_selected"].max() > 30


@pytest.mark.parametrize("seed,nodes,N,max_mult,tiny", [(0, 128, 800, 8, 0.0), (1, 160, 1000, 12, 0.3),
                                                         (2, 64, 500, 16, 0.0), (3, 96, 600, 31, 0.7)])
def test_marginal_gain_classes_match_oracle(oracle, seed, nodes, N, max_mult, tiny):
    # hundreds of candidates with contiguous multiplicities on a fragmented pool: the chunk-size classes
    # are served from their sorted marginal gains (more than 512 steps in a class: sorted in global
    # memory); tiny durations break the monotony of some rows' gains, whose classes keep their DP
    w, a = contiguous_replica_round(7300 + seed, 5, N, nodes, max_mult, small_durations=tiny)
    for depth in (2, 1):
        o = oracle.schedule_batch(w.pools, a, depth=depth)
        g = gpu_round(w.pools, a, depth=depth)
        assert_same(o, g)
    assert np.all(g["status"] == 0) and o["n_selected"].max() > 80


@pytest.mark.parametrize("seed,nodes,N", [(0, 32, 24), (2, 64, 36), (3, 64, 48), (4, 128, 64)])
def test_gang_requests_with_a_large_feasible_box_match_oracle(oracle, seed, nodes, N):
    # short queues on a large fragmented pool: every action is a candidate, there is far more room than
    # the least levels need but not enough for everybody's best level, and gang requests couple the
    # chunk sizes: the dense table over the four chunk-count ranges has millions of cells, of which
    # the rows reach a few thousand (Algorithm 4 on the reachable states only)
    pools = (Pool(POOL_GPU, 8 * nodes, 8),)
    w, a = random_round(6200 + seed, 6, N, pools, replicas=0.5, busy_fraction=0.35, inelastic=0.1, max_mult=8,
                        ragged=False)
    o = oracle.schedule_batch(pools, a)
    g = gpu_round(pools, a)
    assert_same(o, g)
    assert np.all(g["status"] == 0) and o["n_selected"].min() >= N - 2


def _large_box_round(seed, S):
    pools = (Pool(POOL_GPU, 8 * 64, 8),)
    w, a = random_round(6200 + seed, S, 48, pools, replicas=0.5, busy_fraction=0.35, inelastic=0.1, max_mult=8,
                        ragged=False)
    return pools, a


def _gpu_round_ws(pools, a, **kw):
    import torch
    from paper_2603_13019_b200 import binding
    S, N = a["pool"].shape
    rnd = binding.Round(S, N, pools, **kw)
    out = rnd.schedule_batch(binding.to_device(a))
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    rnd.destroy()
    return res


def test_table_that_fits_no_slot_is_reported_per_scenario(oracle):
    # one MiB of scratch: the reachable-state tables of the large boxes do not fit a slot; those
    # scenarios get TANGRAM_STATUS_WORKSPACE, the call returns, the others are unaffected
    pools, a = _large_box_round(3, 6)
    o = oracle.schedule_batch(pools, a)
    g = _gpu_round_ws(pools, a, workspace_bytes=1 << 20)
    assert set(np.unique(g["status"])) <= {0, 4} and (g["status"] == 4).any()
    for sc in np.flatnonzero(g["status"] == 0):
        for k in OUT_KEYS:
            assert np.array_equal(o[k][sc], g[k][sc]), (sc, k)
    assert_same(o, _gpu_round_ws(pools, a))                      # the default scratch holds them all


def test_waiting_for_a_slot_ends(oracle):
    # four slots for 40 scenarios whose tables all need one: with a wait of one millisecond some warps
    # give up (status word, nothing else), with the default wait every warp gets its turn
    pools, a = _large_box_round(3, 40)
    o = oracle.schedule_batch(pools, a)
    short = _gpu_round_ws(pools, a, workspace_bytes=320 << 20, slot_wait_us=1000)
    assert set(np.unique(short["status"])) <= {0, 4}
    for sc in np.flatnonzero(short["status"] == 0):
        for k in OUT_KEYS:
            assert np.array_equal(o[k][sc], short[k][sc]), (sc, k)
    patient = _gpu_round_ws(pools, a, workspace_bytes=320 << 20, slot_wait_us=5_000_000)
    assert_same(o, patient)
