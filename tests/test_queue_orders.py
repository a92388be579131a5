"""Other queue orders (Section 4.2: the scheduling algorithm works with other ordering algorithms than
first come first served) and per-node CPU scheduling with trajectories pinned to nodes (Section 5.2).
CPU pins worked by hand; the GPU tests compare the CUDA path with the oracle."""
import numpy as np
import pytest

from workloads import POOL_API, POOL_CPU, POOL_GPU, Pool, add_trajectories, random_round

SJF, LJF, ARRIVAL = 1, 2, 3


def _arrays(rows, arrival=None):
    """rows: (pool, unit, mask, s, p); one scenario."""
    n = len(rows)
    return dict(pool=np.array([[r[0] for r in rows]], np.uint8), unit=np.array([[r[1] for r in rows]], np.uint8),
                level_mask=np.array([[r[2] for r in rows]], np.uint32), s_us=np.array([[r[3] for r in rows]], np.int64),
                p_us=np.array([[r[4] for r in rows]], np.int64),
                arrival_us=None if arrival is None else np.array([arrival], np.int64),
                n_actions=np.array([n], np.int32), gpu_busy=None)


def test_keys_and_ties_of_the_three_orders(oracle):
    pools = [Pool(POOL_CPU, 8, 8)]
    # least levels: a: r = 2 -> 10 + 100 / 2 = 60; b: r = 1 -> 60; c: r = 4 -> 0 + 90 / 4 = 22; d: r = 1 -> 300
    rows = [(0, 1, 0b1010, 10, 100), (0, 1, 0b1, 60, 0), (0, 1, 0b1000, 0, 90), (0, 1, 0b11, 100, 200)]
    a = _arrays(rows, arrival=[40, 10, 30, 10])
    assert list(oracle.order_queue(pools, a, SJF)[0]) == [2, 0, 1, 3]          # 22, 60 (a before b: queue order), 300
    assert list(oracle.order_queue(pools, a, LJF)[0]) == [3, 0, 1, 2]
    assert list(oracle.order_queue(pools, a, ARRIVAL)[0]) == [1, 3, 2, 0]      # 10 (b before d), 30, 40
    assert list(oracle.order_queue(pools, a, 0)[0]) == [0, 1, 2, 3]
    a["n_actions"][0] = 3                                                       # positions behind the queue map to themselves
    assert list(oracle.order_queue(pools, a, SJF)[0]) == [2, 0, 1, 3]
    assert list(oracle.order_queue(pools, a, LJF)[0]) == [0, 1, 2, 3]


def test_shortest_first_schedules_the_shortest_actions_that_fit(oracle):
    # 3 cores, five one-core actions of 50, 10, 40, 20, 30 us: first come first served takes the first three,
    # shortest first the three shortest (10, 20, 30), longest first 50, 40, 30; results stay at the actions' positions
    pools = [Pool(POOL_CPU, 3, 3)]
    a = _arrays([(0, 1, 1, t, 0) for t in (50, 10, 40, 20, 30)])
    assert list(oracle.schedule_batch(pools, a)["alloc_units"][0]) == [1, 1, 1, 0, 0]
    o = oracle.schedule_batch_ordered(pools, a, SJF)
    assert list(o["alloc_units"][0]) == [0, 1, 0, 1, 1] and list(o["act_us"][0]) == [-1, 10, -1, 20, 30]
    assert list(o["place_off"][0]) == [-1, 0, -1, 1, 2]                         # cores are handed out in the sorted order
    o = oracle.schedule_batch_ordered(pools, a, LJF)
    assert list(o["alloc_units"][0]) == [1, 0, 1, 0, 1] and list(o["place_off"][0]) == [0, -1, 1, -1, 2]


@pytest.mark.parametrize("policy", (SJF, LJF, ARRIVAL))
def test_order_is_a_stable_sort_and_the_round_is_the_plain_round_on_the_sorted_queue(oracle, policy):
    pools = (Pool(POOL_CPU, 24, 8), Pool(POOL_GPU, 16, 8), Pool(POOL_API, 9, 0, 0))
    w, a = random_round(40 + policy, 12, 70, pools, max_mult=4, small_durations=0.4)
    a["arrival_us"] = np.random.default_rng(policy).integers(0, 50, a["pool"].shape).astype(np.int64)
    perm = oracle.order_queue(pools, a, policy)
    o = oracle.schedule_batch_ordered(pools, a, policy, now_us=60)
    for sc in range(12):
        n = int(a["n_actions"][sc])
        pm = perm[sc, :n]
        assert sorted(pm) == list(range(n))
        r = np.array([int(m & -m).bit_length() for m in a["level_mask"][sc, :n].astype(np.int64)])
        T = a["s_us"][sc, :n] + a["p_us"][sc, :n] // np.maximum(r, 1)
        key = {SJF: T, LJF: -T, ARRIVAL: a["arrival_us"][sc, :n]}[policy][pm]
        assert np.all(np.diff(key) >= 0)
        assert np.all(np.diff(pm)[np.diff(key) == 0] > 0)                       # equal keys keep their queue order
        # the plain round on the permuted records gives the same schedule, position by position
        b = {k: (v[sc:sc + 1, :n][:, pm] if k in ("pool", "unit", "level_mask", "s_us", "p_us", "arrival_us") else None)
             for k, v in a.items()}
        b["n_actions"] = np.array([n], np.int32)
        b["gpu_busy"] = a["gpu_busy"][sc:sc + 1] if a["gpu_busy"] is not None else None
        plain = oracle.schedule_batch(pools, b, now_us=60)
        for k in ("alloc_units", "place_node", "place_off", "act_us"):
            assert np.array_equal(plain[k][0, :n], o[k][sc, :n][pm]), (sc, k)
        assert plain["n_selected"][0] == o["n_selected"][sc] and plain["total_act_us"][0] == o["total_act_us"][sc]


def test_replay_keeps_the_queue_in_the_policys_order(oracle):
    # one core, rounds of 10 ms.  a (30 ms) arrives at 0, b (50 ms) at 5 ms, c (10 ms) at 6 ms, d (10 ms) at 7 ms.
    # a runs until 30 ms.  First come first served: b at 30 (ends 80), c at 80, d at 90.
    # Shortest first: at 30 the queue is c, d, b (c before d: equal keys keep their arrival order): c 30-40,
    # d 40-50, b 50-100.  Longest first: b, c, d as they came.
    pools = [Pool(POOL_CPU, 1, 1)]
    a = _arrays([(0, 1, 1, 30_000, 0), (0, 1, 1, 50_000, 0), (0, 1, 1, 10_000, 0), (0, 1, 1, 10_000, 0)],
                arrival=[0, 5_000, 6_000, 7_000])
    fcfs = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=40)
    assert list(fcfs["act_us"][0]) == [30_000, 25_000 + 50_000, 74_000 + 10_000, 83_000 + 10_000]
    sjf = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=40, policy=SJF)
    assert list(sjf["act_us"][0]) == [30_000, 45_000 + 50_000, 24_000 + 10_000, 33_000 + 10_000]
    assert sjf["rounds_used"][0] == 11 and sjf["total_act_us"][0] < fcfs["total_act_us"][0]
    ljf = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=40, policy=LJF)
    assert list(ljf["act_us"][0]) == list(fcfs["act_us"][0])
    # a shorter action that arrives while the head does not fit becomes the head: 2 cores, x takes both for 30 ms,
    # y (2 cores, 20 ms) waits; z (1 core, 5 ms) arrives at 12 ms: shortest first puts it ahead of y, but it does
    # not fit either; at 30 ms z runs (ends 35), y has to wait for it (needs both cores): starts at 40
    pools = [Pool(POOL_CPU, 2, 2)]
    a = _arrays([(0, 2, 1, 30_000, 0), (0, 2, 1, 20_000, 0), (0, 1, 1, 5_000, 0)], arrival=[0, 1_000, 12_000])
    sjf = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=40, policy=SJF)
    assert list(sjf["act_us"][0]) == [30_000, 39_000 + 20_000, 18_000 + 5_000]
    fcfs = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=40)
    assert list(fcfs["act_us"][0]) == [30_000, 29_000 + 20_000, 38_000 + 5_000]


# ------------------------------------------------------------------ trajectories pinned to CPU nodes
def _traj(rows, traj, mem, node, free):
    a = _arrays(rows)
    a["trajectory"], a["traj_mem"] = np.array([traj], np.int32), np.array([mem], np.uint32)
    a["traj_node"], a["node_mem_free"] = np.array([node], np.int32), np.array([free], np.int64)
    return a


NODES = [Pool(POOL_CPU, 8, 8), Pool(POOL_CPU, 16, 8), Pool(POOL_GPU, 8, 8), Pool(POOL_CPU, 16, 8)]


def test_a_trajectory_goes_to_the_node_with_the_most_free_memory_and_stays_there(oracle):
    one = (0, 1, 1, 100, 0)
    # free memory 50 / 70 / - / 70: trajectory 0 (20) -> node 1 (most free, lower index of the tie), 50 left;
    # trajectory 1 (30) -> node 3 (70), 40 left; trajectory 0 again -> node 1, nothing more set aside;
    # trajectory 2 (45) -> node 0 (50 / 50 / 40: lower index), 5 left; the action without a trajectory keeps its pool
    a = _traj([one] * 5, [0, 1, 0, 2, -1], [20, 30, 20, 45, 9], [-1, -1, -1], [50, 70, 999, 70])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    assert list(o["pool"][0]) == [1, 3, 1, 0, 0] and o["n_admitted"][0] == 5
    assert list(o["traj_node"][0]) == [1, 3, 0] and list(o["node_mem_free"][0]) == [5, 50, 999, 40]


def test_nodes_without_the_cores_or_the_memory_are_filtered_out(oracle):
    # the action needs at least 4 x 3 = 12 cores (its least level; its largest, 20, fits no node and does not
    # matter): node 0 (8 cores) is out although it has the most memory
    a = _traj([(0, 4, 0b11100, 100, 0)], [0], [10], [-1], [90, 20, 999, 30])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    assert o["pool"][0, 0] == 3 and list(o["node_mem_free"][0]) == [90, 20, 999, 20]
    # the memory of the whole trajectory has to be free: 25 fits node 3 only
    a = _traj([(0, 1, 1, 100, 0)], [0], [25], [-1], [24, 20, 999, 30])
    assert oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])["pool"][0, 0] == 3
    # a pinned trajectory is not moved, whatever the memory says now; a GPU action is none of the CPU manager's
    a = _traj([(0, 1, 1, 100, 0), (2, 1 | 0x80, 1, 100, 0)], [0, 1], [25, 5], [0, -1], [0, 20, 999, 30])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    assert list(o["pool"][0]) == [0, 2] and list(o["traj_node"][0]) == [0, -1] and list(o["node_mem_free"][0]) == [0, 20, 999, 30]


def test_a_trajectory_that_finds_no_node_ends_the_admitted_queue(oracle):
    one = (0, 1, 1, 100, 0)
    a = _traj([one] * 4, [0, 1, 2, 0], [10, 80, 5, 10], [-1, -1, -1], [50, 60, 999, 70])
    o = oracle.pin_trajectories(NODES, a, a["traj_node"], a["node_mem_free"])
    # trajectory 0 -> node 3 (60 left); trajectory 1 needs 80: nowhere; what stands behind it waits as well
    assert o["n_admitted"][0] == 1 and list(o["traj_node"][0]) == [3, -1, -1]
    assert list(o["pool"][0]) == [3, 0, 0, 0] and list(o["node_mem_free"][0]) == [50, 60, 999, 60]


def test_replay_pins_trajectories_as_their_actions_arrive(oracle):
    # two nodes of 4 cores with 10 and 6 units of memory free, rounds of 10 ms, one-core actions.
    # a0 (trajectory 0, 8 units, 25 ms) arrives at 0: node 0 (most free), 2 left.  a1 (trajectory 1, 5 units, 12 ms,
    # its last action) at 1 ms: only node 1 has 5: 1 left.  a2 (trajectory 2, 4 units, 10 ms) at 2 ms finds no node
    # and waits outside the queue; a3 (trajectory 0 again, 5 ms, its last action) at 3 ms waits behind it although
    # its trajectory has a node.  a1 runs 10 .. 22; the round at 30 gives its 5 units back to node 1, a2 goes there
    # (6 >= 4), a3 to node 0; a3 ends at 35 and the round at 40 gives trajectory 0's 8 units back to node 0.
    pools = [Pool(POOL_CPU, 4, 4), Pool(POOL_CPU, 4, 4)]
    one = lambda t: (0, 1, 1, t, 0)
    a = _arrays([one(25_000), one(12_000), one(10_000), one(5_000)], arrival=[0, 1_000, 2_000, 3_000])
    a["trajectory"], a["traj_mem"] = np.array([[0, 1, 2, 0]], np.int32), np.array([[8, 5, 4, 8]], np.uint32)
    a["traj_last"] = np.array([[0, 1, 0, 1]], np.uint8)
    a["traj_node"], a["node_mem_free"] = np.full((1, 3), -1, np.int32), np.array([[10, 6]], np.int64)
    o = oracle.replay_trace_pinned(pools, a, round_us=10_000, max_rounds=30)
    assert list(o["pool"][0]) == [0, 1, 1, 0]
    assert list(o["act_us"][0]) == [25_000, 9_000 + 12_000, 28_000 + 10_000, 27_000 + 5_000]
    assert list(o["traj_node"][0]) == [-1, -1, 1] and list(o["node_mem_free"][0]) == [10, 2]
    assert o["rounds_used"][0] == 5 and o["occupancy"][0, :5].tolist() == [[1, 0], [1, 1], [1, 1], [1, 1], [0, 0]]
    # without the marks nothing is given back: a2 never finds a node, a3 never gets past it
    a["traj_last"][:] = 0
    o = oracle.replay_trace_pinned(pools, a, round_us=10_000, max_rounds=30)
    assert list(o["alloc_units"][0]) == [1, 1, 0, 0] and o["rounds_used"][0] == 30
    assert list(o["traj_node"][0]) == [0, 1, -1] and list(o["node_mem_free"][0]) == [2, 1]


# ------------------------------------------------------------------ CUDA path against the oracle
KEYS = ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us")
POOLS = (Pool(POOL_CPU, 64, 16), Pool(POOL_GPU, 32, 8), Pool(POOL_API, 40, 0, 0), Pool(POOL_CPU, 32, 8))


@pytest.mark.gpu
@pytest.mark.parametrize("seed,policy", [(0, SJF), (1, LJF), (2, ARRIVAL), (3, SJF), (4, LJF), (5, SJF), (6, SJF), (7, LJF), (8, ARRIVAL)])
def test_ordered_rounds_match_oracle(oracle, seed, policy):
    import torch
    from paper_2603_13019_b200 import binding
    # every tile size of the register sort (1 .. 32 elements per thread), queues below one element per thread,
    # the wide keys of the arrival order; tiny durations: many equal keys
    N = [300, 4200, 33, 1000, 64, 2048, 4096, 9000, 5000][seed]
    w, a = random_round(900 + seed, 24, N, POOLS, max_mult=4, narrow=seed != 3, small_durations=0.6 if seed in (0, 4) else 0.0,
                        busy_fraction=0.2 if seed % 2 else 0.0)
    a["arrival_us"] = np.random.default_rng(seed).integers(-50, 200, a["pool"].shape).astype(np.int64)
    o = oracle.schedule_batch_ordered(POOLS, a, policy, now_us=300)
    operm = oracle.order_queue(POOLS, a, policy)
    rnd = binding.Round(24, N, POOLS)
    dev = binding.to_device(a)
    perm = rnd.order_queue(dev, policy)
    out = rnd.schedule_batch_ordered(dev, policy, now_us=300)
    out2 = rnd.schedule_batch_ordered(dev, policy, now_us=300)      # the kept staging is reused
    torch.cuda.synchronize()
    assert np.array_equal(operm, perm.cpu().numpy())
    for res in (out, out2):
        for k in KEYS:
            assert np.array_equal(o[k], res[k].cpu().numpy()), k
    plain = oracle.schedule_batch(POOLS, a, now_us=300)
    assert not np.array_equal(plain["alloc_units"], o["alloc_units"])
    rnd.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(5))
def test_pinned_trajectories_match_oracle(oracle, seed):
    import torch
    from paper_2603_13019_b200 import binding
    N = [200, 1500, 31, 700, 4096][seed]
    w, a = random_round(950 + seed, 40, N, POOLS, max_mult=4, narrow=seed != 1)
    a = add_trajectories(seed, a, POOLS, max_traj=[16, 300, 5, 64, 900][seed], mem_hi=[64, 8, 64, 30, 4][seed],
                         pinned=0.3 if seed != 2 else 0.0)
    o = oracle.pin_trajectories(POOLS, a, a["traj_node"], a["node_mem_free"])
    rnd = binding.Round(40, N, POOLS)
    dev = binding.to_device(a)
    dev["traj_mem"] = dev["traj_mem"].view(torch.int32) if dev["traj_mem"].dtype != torch.int32 else dev["traj_mem"]
    out = rnd.pin_trajectories(dev)
    torch.cuda.synchronize()
    assert np.array_equal(o["pool"], out["pool"].cpu().numpy())
    assert np.array_equal(o["n_admitted"], out["n_admitted"].cpu().numpy())
    assert np.array_equal(o["traj_node"], dev["traj_node"].cpu().numpy())
    assert np.array_equal(o["node_mem_free"], dev["node_mem_free"].cpu().numpy())
    if seed != 2:
        assert (o["n_admitted"] < a["n_actions"]).sum() > 3 and (o["n_admitted"] == a["n_actions"]).sum() > 3
    # the pinned queue goes through the round: pool column from the pin, queue cut at n_admitted
    b = dict(a, pool=o["pool"], n_actions=o["n_admitted"])
    ob = oracle.schedule_batch(POOLS, b)
    devb = dict(dev, pool=out["pool"], n_actions=out["n_admitted"])
    g = rnd.schedule_batch(devb)
    torch.cuda.synchronize()
    for k in KEYS:
        assert np.array_equal(ob[k], g[k].cpu().numpy()), k
    rnd.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("seed,policy", [(0, SJF), (1, LJF), (2, SJF), (3, SJF), (4, LJF)])
def test_ordered_traces_match_oracle(oracle, seed, policy):
    import torch
    from paper_2603_13019_b200 import binding
    pools = [(Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 16, 8), Pool(POOL_API, 5, 0, 200_000)),
             (Pool(POOL_GPU, 40, 8),), (Pool(POOL_CPU, 40, 8), Pool(POOL_GPU, 8, 4), Pool(POOL_API, 3, 0, 0)),
             (Pool(POOL_CPU, 6, 3),), (Pool(POOL_CPU, 16, 4), Pool(POOL_GPU, 32, 8))][seed]
    N = [150, 200, 120, 400, 300][seed]
    w, a = random_round(970 + seed, 14, N, pools, max_mult=4, small_durations=0.3 if seed != 3 else 0.8,
                        replicas=0.5 if seed in (1, 4) else 0.0)
    rng = np.random.default_rng(seed)
    # bursts: many arrivals per round while actions last up to 0.5 s, so the queue is long and its order matters
    a["arrival_us"] = np.cumsum(rng.integers(0, [3000, 4000, 2500, 300, 3000][seed], a["pool"].shape), axis=1).astype(np.int64)
    o = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=5000, policy=policy)
    rnd = binding.Round(14, N, pools, round_us=10_000, max_rounds=5000)
    dev = binding.to_device(a)
    g = rnd.replay_trace(dev, policy=policy)
    g2 = rnd.replay_trace(dev, policy=policy)
    plain = rnd.replay_trace(dev)                                   # first come first served is untouched by the kept keys
    torch.cuda.synchronize()
    for res in (g, g2):
        for k in KEYS + ("rounds_used", "occupancy"):
            assert np.array_equal(o[k], res[k].cpu().numpy()), k
    of = oracle.replay_trace(pools, a, round_us=10_000, max_rounds=5000)
    for k in KEYS + ("rounds_used", "occupancy"):
        assert np.array_equal(of[k], plain[k].cpu().numpy()), k
    assert not np.array_equal(of["act_us"], o["act_us"])
    rnd.destroy()


@pytest.mark.gpu
@pytest.mark.parametrize("seed,policy", [(0, 0), (1, 0), (2, SJF), (3, 0), (4, LJF)])
def test_traces_with_trajectories_pinned_on_arrival_match_oracle(oracle, seed, policy):
    import torch
    from paper_2603_13019_b200 import binding
    pools = [(Pool(POOL_CPU, 16, 4), Pool(POOL_CPU, 8, 4), Pool(POOL_GPU, 16, 8)),
             (Pool(POOL_CPU, 6, 3), Pool(POOL_CPU, 6, 3), Pool(POOL_CPU, 12, 4)),
             (Pool(POOL_CPU, 16, 4), Pool(POOL_API, 6, 0, 0), Pool(POOL_CPU, 16, 8)),
             (Pool(POOL_CPU, 4, 4), Pool(POOL_CPU, 4, 4)),
             (Pool(POOL_CPU, 24, 8), Pool(POOL_GPU, 8, 8), Pool(POOL_CPU, 8, 8))][seed]
    N = [200, 300, 150, 400, 250][seed]
    w, a = random_round(990 + seed, 12, N, pools, max_mult=4, small_durations=0.3, replicas=0.0)
    rng = np.random.default_rng(seed)
    a["arrival_us"] = np.cumsum(rng.integers(0, [3000, 2000, 3000, 1500, 3000][seed], a["pool"].shape), axis=1).astype(np.int64)
    # memory is tight enough for arrivals to wait at the gate, in some scenarios for good
    a = add_trajectories(seed, a, pools, max_traj=[40, 25, 30, 60, 35][seed], mem_hi=40, pinned=0.0, mem_free_hi=700)
    o = oracle.replay_trace_pinned(pools, a, round_us=10_000, max_rounds=4000, policy=policy)
    rnd = binding.Round(12, N, pools, round_us=10_000, max_rounds=4000)
    dev = binding.to_device(a)
    dev["traj_mem"] = dev["traj_mem"].view(torch.int32)
    g = rnd.replay_trace_pinned(dev, policy=policy)
    torch.cuda.synchronize()
    for k in KEYS + ("rounds_used", "occupancy", "pool"):
        assert np.array_equal(o[k], g[k].cpu().numpy()), k
    assert np.array_equal(o["traj_node"], dev["traj_node"].cpu().numpy())
    assert np.array_equal(o["node_mem_free"], dev["node_mem_free"].cpu().numpy())
    assert (o["alloc_units"] > 0).sum() > 500 and (o["pool"] != a["pool"]).sum() > 30
    rnd.destroy()
