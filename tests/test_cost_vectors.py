"""Cost vectors (Section 4.1, vectorized resource cost): an action asks its key resource, which alone is
elastic, and fixed amounts of up to two further quota / concurrency pools (memory beside the cores, the
quotas of other sites).  The pins are worked by hand from the rules; the GPU tests compare the CUDA path
with the oracle on random rounds and traces."""
import numpy as np
import pytest

from workloads import POOL_API, POOL_CPU, POOL_GPU, Pool, add_side_costs, random_round

NONE = 0xFF


def _arrays(rows, arrival=None):
    """rows: (pool, unit, mask, s, p, [(side pool, amount), ...]); one scenario."""
    n = len(rows)
    a = dict(pool=np.array([[r[0] for r in rows]], np.uint8), unit=np.array([[r[1] for r in rows]], np.uint8),
             level_mask=np.array([[r[2] for r in rows]], np.uint32), s_us=np.array([[r[3] for r in rows]], np.int64),
             p_us=np.array([[r[4] for r in rows]], np.int64),
             arrival_us=None if arrival is None else np.array([arrival], np.int64),
             n_actions=np.array([n], np.int32), gpu_busy=None,
             side_pool=np.full((2, 1, n), NONE, np.uint8), side_units=np.zeros((2, 1, n), np.uint16))
    for i, r in enumerate(rows):
        for e, (k, c) in enumerate(r[5]):
            a["side_pool"][e, 0, i], a["side_units"][e, 0, i] = k, c
    return a


def test_a_further_amount_that_does_not_fit_ends_the_candidate_prefix(oracle):
    # 8 cores and 10 units of memory; every action takes one core for 100 us and 4 units of memory:
    # the third would bring the memory to 12, so the prefix ends there, and the action behind it
    # waits although it asks no memory and cores are free (first come first served)
    pools = [Pool(POOL_CPU, 8, 8), Pool(POOL_API, 10, 0, 0)]
    rows = [(0, 1, 1, 100, 0, [(1, 4)])] * 3 + [(0, 1, 1, 100, 0, [])]
    o = oracle.schedule_batch(pools, _arrays(rows))
    assert list(o["alloc_units"][0]) == [1, 1, 0, 0] and o["n_selected"][0] == 2 and o["status"][0] == 0
    # two entries of one action on the same pool add up: 3 + 4 = 7, then 7 more do not fit
    rows = [(0, 1, 1, 100, 0, [(1, 3), (1, 4)])] * 2
    assert list(oracle.schedule_batch(pools, _arrays(rows))["alloc_units"][0]) == [1, 0]
    # with 3 units each all four are candidates
    rows = [(0, 1, 1, 100, 0, [(1, 3)])] * 3 + [(0, 1, 1, 100, 0, [])]
    assert list(oracle.schedule_batch(pools, _arrays(rows))["alloc_units"][0]) == [1, 1, 1, 1]


def test_amounts_of_all_candidates_are_set_aside_before_the_key_actions_share_the_pool(oracle):
    # pool 0: 10 tokens (concurrency), pool 1: 8 cores.  x: key pool 0, 1/2/4/8 tokens, T(r) = 800 / r.
    # y: one core, and 5 tokens of pool 0 beside it.  y stands BEHIND x in the queue, yet its 5 tokens are set
    # aside first: x shares what is left, 5, and gets 4 tokens (200 us), not 8
    pools = [Pool(POOL_API, 10, 0, 0), Pool(POOL_CPU, 8, 8)]
    x = (0, 1, 0b10001011, 0, 800, [])
    o = oracle.schedule_batch(pools, _arrays([x, (1, 1, 1, 50, 0, [(0, 5)])]))
    assert list(o["alloc_units"][0]) == [4, 1] and list(o["act_us"][0]) == [200, 50]
    assert list(o["place_off"][0]) == [0, 0]
    # 2 tokens beside the core leave 8 for x
    o = oracle.schedule_batch(pools, _arrays([x, (1, 1, 1, 50, 0, [(0, 2)])]))
    assert list(o["alloc_units"][0]) == [8, 1] and o["act_us"][0, 0] == 100
    # 9 tokens leave one; 10 do not fit on top of x's least level: y is no candidate, x gets 8
    o = oracle.schedule_batch(pools, _arrays([x, (1, 1, 1, 50, 0, [(0, 9)])]))
    assert list(o["alloc_units"][0]) == [1, 1]
    o = oracle.schedule_batch(pools, _arrays([x, (1, 1, 1, 50, 0, [(0, 10)])]))
    assert list(o["alloc_units"][0]) == [8, 0]


def test_an_evicted_candidate_keeps_its_amounts_set_aside_but_consumes_nothing(oracle):
    # pool 0: 2 cores, pool 1: 10 tokens (concurrency).  a, b: 1 or 2 cores, T(r) = 1000 / r; b also asks
    # 5 tokens.  c: key pool 1, 1/2/4/8 tokens, T(r) = 800 / r.
    # Cores: both kept: 1000 + 1000 = 2000.  b evicted: a alone takes both cores (500); b then starts when a
    # ends, at 500, and at depth 2 its faster level counts: 500 + 500 = 1000; 500 + 1000 = 1500 < 2000: b goes.
    # Tokens: b's 5 stay set aside in this round, c gets 4 (200 us); after the round only c's 4 are in use.
    pools = [Pool(POOL_CPU, 2, 2), Pool(POOL_API, 10, 0, 0)]
    rows = [(0, 1, 0b11, 0, 1000, []), (0, 1, 0b11, 0, 1000, [(1, 5)]), (1, 1, 0b10001011, 0, 800, [])]
    o = oracle.schedule_batch(pools, _arrays(rows))
    assert list(o["alloc_units"][0]) == [2, 0, 4] and list(o["act_us"][0]) == [500, -1, 200]
    # replayed with rounds of 1000 us: round 1 finds everything released, b runs alone on 2 cores with its
    # 5 tokens (1000 + 500), round 2 finds the scenario drained
    o = oracle.replay_trace(pools, _arrays(rows, arrival=[0, 0, 0]), round_us=1000, max_rounds=8)
    assert list(o["alloc_units"][0]) == [2, 2, 4] and list(o["act_us"][0]) == [500, 1500, 200]
    assert o["occupancy"][0, :3].tolist() == [[2, 4], [2, 5], [0, 0]] and o["rounds_used"][0] == 3


def test_a_concurrency_pool_holds_the_amount_until_the_action_ends(oracle):
    # 8 cores, 10 units of memory, rounds of 1000 us.  Two actions of 2500 us, one core and 6 units each:
    # the second cannot start before the first has ended (6 + 6 > 10), i.e. in the round at 3000
    pools = [Pool(POOL_CPU, 8, 8), Pool(POOL_API, 10, 0, 0)]
    rows = [(0, 1, 1, 2500, 0, [(1, 6)])] * 2
    o = oracle.replay_trace(pools, _arrays(rows, arrival=[0, 0]), round_us=1000, max_rounds=12)
    assert list(o["act_us"][0]) == [2500, 3000 + 2500]
    assert o["occupancy"][0, :7].tolist() == [[1, 6]] * 6 + [[0, 0]] and o["rounds_used"][0] == 7


def test_a_quota_pool_counts_the_amounts_in_its_window(oracle):
    # pool 0: 5 tokens per 100 ms, pool 1: 8 cores, rounds of 10 ms.  a, b, c: one core for 1 ms and 2 tokens;
    # d: key pool 0, one token, 10 us; e: the same, arriving at 105 ms.
    # Round 0: a (2), b (4), c would make 6: the prefix ends, d waits behind c.  The tokens stay used although
    # a and b end: nothing moves until the window changes at 100 ms (round 10): c and d start, d's offset is 0
    # (amounts are booked after the key grants), used = 1 + 2.  e starts in round 11 at offset 3.
    pools = [Pool(POOL_API, 5, 0, 100_000), Pool(POOL_CPU, 8, 8)]
    rows = [(1, 1, 1, 1000, 0, [(0, 2)])] * 3 + [(0, 1, 1, 10, 0, [])] * 2
    o = oracle.replay_trace(pools, _arrays(rows, arrival=[0, 0, 0, 0, 105_000]), round_us=10_000, max_rounds=20)
    assert list(o["act_us"][0]) == [1000, 1000, 100_000 + 1000, 100_000 + 10, 5000 + 10]
    assert list(o["place_off"][0][3:]) == [0, 3]
    assert o["occupancy"][0, :12, 0].tolist() == [4] * 10 + [3, 4]
    assert o["rounds_used"][0] == 13                              # e ends at 110.01 ms: round 12 finds it gone


def test_entries_that_no_pool_can_serve_are_bad_records(oracle):
    pools = [Pool(POOL_CPU, 8, 8), Pool(POOL_API, 10, 0, 0), Pool(POOL_API, 4, 0, 50_000), Pool(POOL_GPU, 8, 8)]
    good = (0, 1, 1, 100, 0, [(1, 10), (2, 4)])
    assert oracle.schedule_batch(pools, _arrays([good]))["status"][0] == 0
    for side in ([(0, 1)], [(3, 1)], [(4, 1)], [(1, 0)], [(1, 11)], [(2, 1), (2, 5)]):
        o = oracle.schedule_batch(pools, _arrays([good, (0, 1, 1, 100, 0, side)]))
        assert o["status"][0] == 1 and o["n_selected"][0] == 0, side
    # the key pool itself cannot be named again
    assert oracle.schedule_batch(pools, _arrays([(1, 1, 1, 100, 0, [(1, 1)])]))["status"][0] == 1
    # "none" ignores the amount
    a = _arrays([good])
    a["side_pool"][1, 0, 0], a["side_units"][1, 0, 0] = NONE, 999
    assert oracle.schedule_batch(pools, a)["status"][0] == 0


POOLS = (Pool(POOL_CPU, 32, 8), Pool(POOL_GPU, 32, 8), Pool(POOL_API, 40, 0, 0), Pool(POOL_API, 25, 0, 200_000))


def _prefix_by_hand(pools, a, sc):
    """Length of the candidate prefix for single-level actions on fresh pools without GPU topology limits:
    running totals per pool, key units and further amounts alike."""
    used = [0] * len(pools)
    for i in range(int(a["n_actions"][sc])):
        add = [0] * len(pools)
        add[a["pool"][sc, i]] += int(a["unit"][sc, i] & 0x7F) * (int(a["level_mask"][sc, i]).bit_length())
        for e in range(a["side_pool"].shape[0]):
            if a["side_pool"][e, sc, i] != NONE:
                add[a["side_pool"][e, sc, i]] += int(a["side_units"][e, sc, i])
        if any(used[j] + add[j] > pools[j].capacity for j in range(len(pools)) if add[j]):
            return i
        used = [u + v for u, v in zip(used, add)]
    return int(a["n_actions"][sc])


@pytest.mark.parametrize("seed", range(4))
def test_all_single_level_rounds_schedule_exactly_the_prefix(oracle, seed):
    # with only one level per action nothing is chosen (Algorithm 1, the all-inelastic case): what is
    # scheduled is the candidate prefix, which a running total per pool gives.  Gang requests of one GPU
    # keep the chunk test out of it.
    w, a = random_round(500 + seed, 24, 80, POOLS, inelastic=1.0, replicas=0.0)
    a["level_mask"] = np.where(a["pool"] == 1, 1, a["level_mask"]).astype(np.uint32)
    a = add_side_costs(seed, a, POOLS, fraction=0.6)
    o = oracle.schedule_batch(POOLS, a)
    hit = 0
    for sc in range(24):
        n = _prefix_by_hand(POOLS, a, sc)
        assert np.all(o["alloc_units"][sc, :n] > 0) and np.all(o["alloc_units"][sc, n:] == 0), sc
        hit += n < a["n_actions"][sc]
    assert hit > 12


@pytest.mark.parametrize("seed", range(4))
def test_no_pool_is_overdrawn_and_elastic_actions_still_get_the_spare_units(oracle, seed):
    w, a = random_round(600 + seed, 24, 120, POOLS, max_mult=4)
    a = add_side_costs(seed, a, POOLS, fraction=0.5)
    o = oracle.schedule_batch(POOLS, a)
    b = {k: v for k, v in a.items() if not k.startswith("side_")}
    plain = oracle.schedule_batch(POOLS, b)
    sel = o["alloc_units"] > 0
    for j in (2, 3):
        key = np.where(sel & (a["pool"] == j), o["alloc_units"], 0).sum(axis=1)
        side = sum(np.where(sel & (a["side_pool"][e] == j), a["side_units"][e], 0).sum(axis=1) for e in range(2))
        assert np.all(key + side <= POOLS[j].capacity)
    assert np.any(o["n_selected"] < plain["n_selected"])          # the amounts did bind somewhere


# ------------------------------------------------------------------ CUDA path against the oracle
KEYS = ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us")


def _gpu_round(pools, a, n_side, **kw):
    import torch
    from paper_2603_13019_b200 import binding
    S, N = a["pool"].shape
    rnd = binding.Round(S, N, pools, side_costs=n_side, **kw)
    if kw.get("max_rounds", 0) > 0:
        out = rnd.replay_trace(binding.to_device(a))
    else:
        out = rnd.schedule_batch(binding.to_device(a))
    torch.cuda.synchronize()
    g = {k: v.cpu().numpy() for k, v in out.items()}
    rnd.destroy()
    return g


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(8))
def test_rounds_with_cost_vectors_match_oracle(oracle, seed):
    n_side = 1 + seed % 2
    pools = POOLS if seed < 6 else (Pool(POOL_API, 60, 0, 0), Pool(POOL_CPU, 64, 16), Pool(POOL_API, 30, 0, 50_000))
    # un-narrowed masks: the quota / concurrency pools get elastic key actions, which share what the
    # other pools' candidates leave
    w, a = random_round(700 + seed, 64, [200, 90, 700, 150, 4200, 60, 300, 120][seed], pools, max_mult=4,
                        narrow=seed % 3 == 0, busy_fraction=0.2 if seed % 2 else 0.0,
                        small_durations=0.3 if seed == 3 else 0.0)
    a = add_side_costs(seed, a, pools, n_side=n_side, fraction=0.5, max_share=[0.2, 0.05, 0.02, 0.3][seed % 4],
                       invalid=0.002 if seed in (1, 5) else 0.0)
    o = oracle.schedule_batch(pools, a)
    g = _gpu_round(pools, a, n_side)
    for k in KEYS:
        assert np.array_equal(o[k], g[k]), k
    assert (o["status"] == 0).sum() > 8 and (o["alloc_units"] > 0).sum() > 100
    if seed in (1, 5):
        assert (o["status"] == 1).sum() > 0


@pytest.mark.gpu
def test_a_round_created_with_cost_vectors_runs_without_them(oracle):
    w, a = random_round(11, 16, 100, POOLS, max_mult=4)
    g = _gpu_round(POOLS, a, 2)                                  # no side arrays handed over
    o = oracle.schedule_batch(POOLS, a)
    for k in KEYS:
        assert np.array_equal(o[k], g[k]), k


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(4))
def test_traces_with_cost_vectors_match_oracle(oracle, seed):
    pools = (Pool(POOL_CPU, 32, 8), Pool(POOL_GPU, 32, 8), Pool(POOL_API, 40, 0, 0), Pool(POOL_API, 25, 0, 200_000))
    w, a = random_round(800 + seed, 12, 160, pools, max_mult=4, narrow=seed % 2 == 0, small_durations=0.2)
    rng = np.random.default_rng(seed)
    a["arrival_us"] = np.cumsum(rng.integers(0, 5000, a["pool"].shape), axis=1).astype(np.int64)
    a = add_side_costs(seed, a, pools, n_side=2, fraction=0.6, max_share=0.3)
    o = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=1500)
    g = _gpu_round(pools, a, 2, round_us=10_000, max_rounds=1500)
    for k in KEYS + ("rounds_used", "occupancy"):
        assert np.array_equal(o[k], g[k]), k
    assert (o["alloc_units"] > 0).sum() > 300


@pytest.mark.gpu
def test_cfg4_with_cost_vectors_matches_oracle(oracle):
    from workloads import generate, make_workload
    w = make_workload("cfg4_vec", n_scenarios=48)
    a = generate(w)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    g = _gpu_round(w.pools, a, 2, depth=w.depth)
    for k in KEYS:
        assert np.array_equal(o[k], g[k]), k
    plain = oracle.schedule_batch(w.pools, {k: v for k, v in a.items() if not k.startswith("side_")}, depth=w.depth)
    assert (o["n_selected"] < plain["n_selected"]).sum() > 10      # the memory pool ends many prefixes early
