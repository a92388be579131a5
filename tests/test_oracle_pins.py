"""Pins of the CPU oracle against what the paper and plain mathematics fix.

Nothing here compares the oracle with itself: every expected value is a closed form, a
worked example that follows from the paper's rules, an exhaustive enumeration, or an
independent brute-force packing.
"""
import itertools
import os

import numpy as np
import pytest

GANG = 0x80
CPU, GPU, API = 0, 1, 2


# ------------------------------------------------------------------ helpers (independent)
def levels_of(unit, mask, pool_type=CPU, group=8):
    g, gang = unit & 0x7F, bool(unit & GANG) and pool_type == GPU
    out = []
    for r in range(1, 33):
        if mask >> (r - 1) & 1:
            k = g * r
            if gang and not (k & (k - 1) == 0 and k <= group):
                continue
            out.append(r)
    return g, gang, out


def requests_of(unit, r, pool_type=GPU):
    g, gang = unit & 0x7F, bool(unit & GANG)
    return [g * r] if gang else [g] * r


def can_pack(busy, sizes, group=8):
    """Brute force: can the aligned power-of-two requests be placed on the free GPUs?"""
    sizes = sorted(sizes, reverse=True)
    busy = list(busy)

    def rec(i):
        if i == len(sizes):
            return True
        z = sizes[i]
        seen = set()
        for node in range(len(busy)):
            for start in range(0, group, z):
                bits = ((1 << z) - 1) << start
                if busy[node] & bits:
                    continue
                key = (busy[node], start) if False else None
                busy[node] |= bits
                ok = rec(i + 1)
                busy[node] &= ~bits
                if ok:
                    return True
        return False

    return rec(0)


def brute_force_arrange(tasks, fits):
    """Exhaustive optimum under the tie order (sum T, sum units, (k_m..k_1) lexicographic).
    tasks: list of (unit, [r...], s, p); fits(choice of r per task) -> bool."""
    best = None
    for rs in itertools.product(*[t[1] for t in tasks]):
        if not fits(rs):
            continue
        T = sum(t[2] + t[3] // r for t, r in zip(tasks, rs))
        ks = [(t[0] & 0x7F) * r for t, r in zip(tasks, rs)]
        key = (T, sum(ks), tuple(reversed(ks)))
        if best is None or key < best[0]:
            best = (key, ks)
    return best


# ------------------------------------------------------------------ Eq. 1
def test_duration_closed_forms(oracle):
    assert oracle.duration(20000, 200000, 1) == 220000          # T_ori at one unit
    assert oracle.duration(20000, 200000, 8) == 45000
    assert oracle.duration(7, 10, 3) == 10                       # floor of the scalable part
    assert oracle.duration(-5, 1 << 50, 1) == (1 << 40)          # parameters clamped to [0, 2^40]
    rng = np.random.default_rng(0)
    for _ in range(200):
        s, p = int(rng.integers(0, 10**6)), int(rng.integers(0, 10**7))
        prev = None
        for r in range(1, 33):
            T = oracle.duration(s, p, r)
            assert prev is None or T <= prev                    # more units never slow an action
            prev = T
            # Eq. 1: T(m) = T_ori / (E(m) m) with 0 < E(m) <= 1  <=>  m T(m) >= T_ori (up to the floor)
            assert r * (T + 1) > s + p >= 0 and T >= 0
            assert r * T + (r - 1) >= s + p or s > 0


# ------------------------------------------------------------------ Section 5.3 chunks
def _parse_blocks(txt):
    if txt == "-":
        return []
    return sorted(tuple(int(x) for x in b.split(":")) for b in txt.split(","))


def _free_blocks_py(busy, group=8):
    out = []

    def rec(start, size):
        bits = ((1 << size) - 1) << start
        if busy & bits == 0:
            out.append((start, size))
        elif size > 1:
            rec(start, size // 2)
            rec(start + size // 2, size // 2)

    rec(0, group)
    return sorted(out)


def test_chunk_worked_examples(oracle):
    path = os.path.join(os.path.dirname(__file__), "golden", "chunk_examples.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        before, m, node, start, size, after, blocks = line.split()
        rc, gn, gs, gz, busy = oracle.chunk_alloc([int(before, 16)], int(m))
        if int(node) < 0:
            assert rc == -1
        else:
            assert (rc, gn, gs, gz) == (0, int(node), int(start), int(size))
            assert gs % gz == 0 and gz & (gz - 1) == 0          # legal chunk: aligned power of two
        assert busy[0] == int(after, 16)
        assert _free_blocks_py(int(busy[0])) == _parse_blocks(blocks)
        F = oracle.free_blocks([int(busy[0])])
        for lvl in range(4):
            assert F[lvl] == sum(1 for b in _parse_blocks(blocks) if b[1] == 1 << lvl)
        n += 1
    assert n >= 9


def test_chunk_alloc_prefers_smallest_block_then_lowest_position(oracle):
    # node 0 has a free 4-block, node 1 a free 2-block at 2 and node 2 a free 2-block at 0
    rc, node, start, size, busy = oracle.chunk_alloc([0x0F, 0xF3, 0xFC], 2)
    assert (rc, node, start, size) == (0, 1, 2, 2)
    rc, node, start, size, busy = oracle.chunk_alloc(list(busy), 2)
    assert (rc, node, start, size) == (0, 2, 0, 2)
    rc, node, start, size, busy = oracle.chunk_alloc(list(busy), 2)
    assert (rc, node, start, size) == (0, 0, 4, 2)              # split of the 4-block, low half


def test_chunks_fit_matches_bruteforce_packing(oracle):
    rng = np.random.default_rng(1)
    checked = {True: 0, False: 0}
    for _ in range(1500):
        nodes = int(rng.integers(1, 3))
        group = int(rng.choice([2, 4, 8]))
        busy = [int(rng.integers(0, 1 << group)) for _ in range(nodes)]
        n = [int(rng.integers(0, 5)), int(rng.integers(0, 4)), int(rng.integers(0, 3)), int(rng.integers(0, 2))]
        for lvl in range(4):
            if (1 << lvl) > group:
                n[lvl] = 0
        sizes = sum(([1 << lvl] * n[lvl] for lvl in range(4)), [])
        F = oracle.free_blocks(busy, group)
        expect = can_pack(busy, sizes, group)
        assert oracle.chunks_fit(n, F) == expect, (busy, n, F)
        checked[expect] += 1
    assert min(checked.values()) > 100


def test_encode_decode_bijection(oracle):
    N = [3, 2, 2, 1]
    seen = set()
    for d in range(N[3] + 1):
        for c in range(N[2] + 1):
            for b in range(N[1] + 1):
                for a in range(N[0] + 1):
                    j = oracle.encode([a, b, c, d], N)
                    assert j not in seen
                    seen.add(j)
                    assert list(oracle.decode(j, N)) == [a, b, c, d]
    assert seen == set(range(4 * 3 * 3 * 2))                     # collision free and dense
    assert oracle.encode([1, 0, 0, 0], N) == 1 and oracle.encode([0, 1, 0, 0], N) == 4


# ------------------------------------------------------------------ DPArrange
def _random_tasks(rng, m, pool_type, tiny):
    tasks = []
    for _ in range(m):
        if pool_type == GPU:
            if rng.random() < 0.5:
                unit, mask = 1 | GANG, int(rng.integers(1, 256)) & 0x8B or 1
            else:
                unit, mask = int(1 << rng.integers(0, 4)), int(rng.integers(1, 16))
        else:
            unit, mask = int(rng.integers(1, 3)), int(rng.integers(1, 64))
        s = int(rng.integers(0, 3)) if tiny else int(rng.integers(0, 1000))
        p = int(rng.integers(0, 9)) if tiny else int(rng.integers(0, 5000))
        tasks.append((unit, mask, s, p))
    return tasks


@pytest.mark.parametrize("tiny", [False, True])
def test_dp_basic_is_optimal_with_tie_order(oracle, tiny):
    rng = np.random.default_rng(2 + tiny)
    hits = 0
    for _ in range(300):
        m = int(rng.integers(1, 6))
        raw = _random_tasks(rng, m, CPU, tiny)
        U = int(rng.integers(1, 30))
        rc, value, alloc = oracle.dp_arrange([t[0] for t in raw], [t[1] for t in raw], [t[2] for t in raw],
                                             [t[3] for t in raw], pool_type=CPU, capacity=64, group=8, free_units=U)
        for q in range(1, m + 1):
            tasks = [(t[0], levels_of(t[0], t[1])[2], t[2], t[3]) for t in raw[:q]]
            best = brute_force_arrange(tasks, lambda rs: sum((t[0] & 0x7F) * r for t, r in zip(tasks, rs)) <= U)
            if best is None:
                assert rc != 0 and rc <= q
                break
            assert rc == 0 or rc > q
            assert value[q - 1] == best[0][0]
            assert list(alloc[q - 1, :q]) == best[1]
            hits += 1
    assert hits > 300


@pytest.mark.parametrize("tiny", [False, True])
def test_dp_gpu_is_optimal_with_tie_order_and_true_packing(oracle, tiny):
    rng = np.random.default_rng(4 + tiny)
    hits = 0
    for _ in range(160):
        m = int(rng.integers(1, 5))
        raw = _random_tasks(rng, m, GPU, tiny)
        nodes = int(rng.integers(1, 3))
        busy = [int(rng.integers(0, 256)) if rng.random() < 0.7 else 0 for _ in range(nodes)]
        rc, value, alloc = oracle.dp_arrange([t[0] for t in raw], [t[1] for t in raw], [t[2] for t in raw],
                                             [t[3] for t in raw], pool_type=GPU, capacity=8 * nodes, group=8, busy=busy)
        if rc == -1:
            continue
        for q in range(1, m + 1):
            tasks = [(t[0], levels_of(t[0], t[1], GPU)[2], t[2], t[3]) for t in raw[:q]]

            def fits(rs):
                sizes = sum((requests_of(t[0], r) for t, r in zip(tasks, rs)), [])
                return can_pack(busy, sizes)

            best = brute_force_arrange(tasks, fits)
            if best is None:
                assert rc != 0 and rc <= q
                break
            assert rc == 0 or rc > q
            assert value[q - 1] == best[0][0], (raw, busy, q)
            assert list(alloc[q - 1, :q]) == best[1], (raw, busy, q)
            hits += 1
    assert hits > 150


def test_dp_closed_form_cases(oracle):
    # everything fits at the top level: each task takes the smallest level reaching its
    # lowest duration (10 // 4 == 10 // 8 -> 4, not 8)
    unit, mask = [1, 1, 1], [0x8B, 0x8B, 0x0B]
    s, p = [5, 0, 3], [1000, 10, 0]
    rc, value, alloc = oracle.dp_arrange(unit, mask, s, p, pool_type=CPU, capacity=64, group=8, free_units=64)
    assert rc == 0 and list(alloc[2]) == [8, 8, 1]
    assert value[2] == (5 + 125) + (0 + 1) + 3
    # no spare unit: everything at its least level
    rc, value, alloc = oracle.dp_arrange(unit, mask, s, p, pool_type=CPU, capacity=64, group=8, free_units=3)
    assert rc == 0 and list(alloc[2]) == [1, 1, 1] and value[2] == 1005 + 10 + 3
    # prefix that cannot fit is reported
    rc, _, _ = oracle.dp_arrange(unit, mask, s, p, pool_type=CPU, capacity=64, group=8, free_units=2)
    assert rc == 3
    # one elastic task among inelastic ones with x spare units takes the largest level <= 1 + x
    for spare, expect in [(0, 1), (1, 2), (2, 2), (3, 4), (6, 4), (7, 8), (20, 8)]:
        rc, value, alloc = oracle.dp_arrange([1, 1, 1], [1, 0x8B, 1 << 2], [0, 0, 0], [50, 99991, 70],
                                             pool_type=CPU, capacity=64, group=8, free_units=1 + 1 + 3 + spare)
        assert rc == 0 and list(alloc[2]) == [1, expect, 3]


def test_dp_contiguous_convex_equals_greedy_marginal_allocation(oracle):
    # textbook: separable convex resource allocation is solved by repeatedly granting the unit
    # of largest marginal gain.  s + p // r is convex in r when r divides p throughout.
    rng = np.random.default_rng(7)
    for _ in range(60):
        m = int(rng.integers(2, 7))
        rmax = 6
        p = [int(rng.integers(1, 50)) * 60 for _ in range(m)]     # 60 = lcm(1..6)
        s = [int(rng.integers(0, 100)) for _ in range(m)]
        U = int(rng.integers(m, m * rmax + 1))
        r = [1] * m
        for _ in range(U - m):
            gains = [(p[i] // r[i] - p[i] // (r[i] + 1)) if r[i] < rmax else -1 for i in range(m)]
            i = int(np.argmax(gains))
            if gains[i] <= 0:
                break
            r[i] += 1
        greedy = sum(s[i] + p[i] // r[i] for i in range(m))
        rc, value, alloc = oracle.dp_arrange([1] * m, [(1 << rmax) - 1] * m, s, p, pool_type=CPU,
                                             capacity=256, group=8, free_units=U)
        assert rc == 0 and value[m - 1] == greedy


def test_gpu_operator_on_empty_nodes_equals_basic_operator(oracle):
    # with every node free, whole power-of-two chunks never fragment, so the chunk operator
    # must agree with the unit-count operator on value and allocation
    rng = np.random.default_rng(8)
    for _ in range(80):
        m = int(rng.integers(1, 9))
        mask = [int(rng.integers(1, 256)) & 0x8B or 1 for _ in range(m)]
        s = [int(rng.integers(0, 1000)) for _ in range(m)]
        p = [int(rng.integers(0, 9000)) for _ in range(m)]
        nodes = int(rng.integers(1, 4))
        rg, vg, ag = oracle.dp_arrange([1 | GANG] * m, mask, s, p, pool_type=GPU, capacity=8 * nodes, group=8,
                                       busy=[0] * nodes)
        rb, vb, ab = oracle.dp_arrange([1] * m, mask, s, p, pool_type=CPU, capacity=8 * nodes, group=8,
                                       free_units=8 * nodes)
        assert rg == rb
        q = m if rg == 0 else rg - 1
        assert np.array_equal(vg[:q], vb[:q]) and np.array_equal(ag[:q], ab[:q])


def test_state_pruning_changes_nothing(oracle):
    rng = np.random.default_rng(9)
    for _ in range(40):
        m = int(rng.integers(2, 9))
        raw = _random_tasks(rng, m, GPU, bool(rng.integers(0, 2)))
        busy = [int(rng.integers(0, 256)) if rng.random() < 0.5 else 0 for _ in range(3)]
        args = ([t[0] for t in raw], [t[1] for t in raw], [t[2] for t in raw], [t[3] for t in raw])
        a = oracle.dp_arrange(*args, pool_type=GPU, capacity=24, group=8, busy=busy, prune=True)
        b = oracle.dp_arrange(*args, pool_type=GPU, capacity=24, group=8, busy=busy, prune=False)
        assert a[0] == b[0]
        q = m if a[0] == 0 else max(a[0] - 1, 0)
        assert np.array_equal(a[1][:q], b[1][:q]) and np.array_equal(a[2][:q], b[2][:q])


# ------------------------------------------------------------------ estimate (Alg. 2)
def test_estimate_special_cases(oracle):
    rng = np.random.default_rng(10)
    n = 12
    s = rng.integers(0, 1000, n)
    p = rng.integers(0, 9000, n)
    T = s + p                                                     # least level r = 1
    # one slot: strictly sequential, completion times are prefix sums
    assert oracle.estimate([40], [1] * n, [1] * n, s, p, depth=1) == int(np.sum(40 + np.cumsum(T)))
    # more slots than remaining actions, all free at c: everyone starts at c
    assert oracle.estimate([25] * 20, [1] * n, [1] * n, s, p, depth=2) == int(np.sum(25 + T))
    # nothing remaining costs nothing
    assert oracle.estimate([1, 2, 3], [], [], [], [], depth=2) == 0
    # depth: the first remaining action may take its d-th level; the best depth wins
    one = oracle.estimate([0], [1, 1], [0x3, 0x3], [0, 0], [100, 100], depth=1)
    two = oracle.estimate([0], [1, 1], [0x3, 0x3], [0, 0], [100, 100], depth=2)
    assert one == 100 + 200 and two == 50 + 150
    # depth larger than the first action's level count stops early
    assert oracle.estimate([0], [1, 1], [0x1, 0x3], [0, 0], [100, 100], depth=3) == 100 + 200


def test_estimate_is_list_scheduling_on_free_slots(oracle):
    # independent statement: each remaining action, in order, starts on the slot that frees
    # first (earliest-available machine), slots tracked in a sorted list
    rng = np.random.default_rng(11)
    for _ in range(100):
        h = sorted(int(x) for x in rng.integers(0, 500, int(rng.integers(1, 9))))
        n = int(rng.integers(1, 30))
        s = rng.integers(0, 300, n)
        p = rng.integers(0, 900, n)
        mask = rng.integers(1, 16, n)
        best = None
        for d in (1, 2):
            lv0 = [r for r in range(1, 5) if mask[0] >> (r - 1) & 1]
            if len(lv0) < d:
                break
            slots, total = list(h), 0
            for i in range(n):
                lv = [r for r in range(1, 5) if mask[i] >> (r - 1) & 1]
                r = lv0[d - 1] if i == 0 else lv[0]
                slots.sort()
                done = slots[0] + int(s[i]) + int(p[i]) // r
                total += done
                slots[0] = done
            best = total if best is None else min(best, total)
        assert oracle.estimate(h, [1] * n, mask, s, p, depth=2) == best


# ------------------------------------------------------------------ Algorithm 1, closed forms
def _round(oracle, pools, rows, depth=2, busy=None, now=0):
    from workloads import Pool
    n = len(rows)
    a = dict(pool=np.array([[r[0] for r in rows]], np.uint8), unit=np.array([[r[1] for r in rows]], np.uint8),
             level_mask=np.array([[r[2] for r in rows]], np.uint32), s_us=np.array([[r[3] for r in rows]], np.int64),
             p_us=np.array([[r[4] for r in rows]], np.int64), arrival_us=None,
             n_actions=np.array([n], np.int32), gpu_busy=None if busy is None else np.array([busy], np.uint8))
    return oracle.schedule_batch([Pool(*p) for p in pools], a, depth=depth, now_us=now)


def test_eviction_closed_form_two_actions(oracle):
    # two identical actions, two cores, levels {1,2}, T(1) = s + p, T(2) = s + p/2, nothing else waits.
    # keep both: 2(s + p).  evict the second: (s + p/2) + best of {(s+p/2)+(s+p), (s+p/2)+(s+p/2)}
    # = 3s + 1.5p at depth 2, so eviction happens iff s < p/2; at depth 1 it never pays.
    pools = [(CPU, 2, 2, 0)]
    for s, p, evict in [(0, 1000, True), (499, 1000, True), (500, 1000, False), (800, 1000, False)]:
        o = _round(oracle, pools, [(0, 1, 3, s, p), (0, 1, 3, s, p)], depth=2)
        if evict:
            assert list(o["alloc_units"][0]) == [2, 0] and o["n_selected"][0] == 1
            assert o["act_us"][0, 0] == s + p // 2 and o["act_us"][0, 1] == -1
        else:
            assert list(o["alloc_units"][0]) == [1, 1] and o["total_act_us"][0] == 2 * (s + p)
        o1 = _round(oracle, pools, [(0, 1, 3, s, p), (0, 1, 3, s, p)], depth=1)
        assert list(o1["alloc_units"][0]) == [1, 1]


def test_head_candidate_is_never_evicted_and_shortcut(oracle):
    # three actions, one core each possible; eviction may strip the tail but keeps the head
    o = _round(oracle, [(CPU, 3, 3, 0)], [(0, 1, 7, 0, 900), (0, 1, 7, 0, 900), (0, 1, 7, 0, 900)])
    assert o["alloc_units"][0, 0] > 0
    # all candidates inelastic: selected as they are, least-required units, no eviction
    o = _round(oracle, [(CPU, 8, 4, 0)], [(0, 1, 1 << 2, 10, 100), (0, 2, 1 << 1, 10, 100), (0, 1, 1, 10, 100)])
    assert list(o["alloc_units"][0]) == [3, 4, 1] and o["n_selected"][0] == 3
    # candidate prefix is one prefix of the whole queue: the GPU action that does not fit
    # blocks the CPU action behind it
    o = _round(oracle, [(CPU, 8, 4, 0), (GPU, 8, 8, 0)],
               [(1, 8 | GANG, 1, 5, 50), (1, 1 | GANG, 1, 5, 50), (0, 1, 1, 5, 50)])
    assert list(o["alloc_units"][0]) == [8, 0, 0]
    # Eq. 2: ACT = time queued so far + execution
    o = _round(oracle, [(CPU, 8, 4, 0)], [(0, 1, 1, 10, 100)], now=1234)
    assert o["act_us"][0, 0] == 1234 + 110 and o["total_act_us"][0] == 1344


def test_cpu_placement_numa_first(oracle):
    # domains of 4 cores; 3 then 3 then 2 cores: the third fits no single domain's remainder of
    # the first two (1 + 1 free) but fits the untouched domain? there are only two domains, so
    # it spans them in ascending order
    o = _round(oracle, [(CPU, 8, 4, 0)], [(0, 1, 1 << 2, 1, 0), (0, 1, 1 << 2, 1, 0), (0, 1, 1 << 1, 1, 0)])
    assert list(o["alloc_units"][0]) == [3, 3, 2]
    assert list(o["place_node"][0]) == [0, 1, 0] and list(o["place_off"][0]) == [0, 4, 3]
    # best fit: 2 cores go to the domain with the fewest free cores that still fits
    o = _round(oracle, [(CPU, 12, 4, 0)], [(0, 1, 1 << 1, 1, 0), (0, 1, 1 << 1, 1, 0), (0, 1, 1 << 0, 1, 0)])
    assert list(o["place_node"][0]) == [0, 0, 1] and list(o["place_off"][0]) == [0, 2, 4]


def test_gpu_placement_order_and_preoccupation(oracle):
    # sizes placed large first; within a size by queue position; busy GPUs respected
    rows = [(0, 1 | GANG, 1, 1, 0), (0, 4 | GANG, 1, 1, 0), (0, 2 | GANG, 1, 1, 0), (0, 2, 2, 1, 0)]
    o = _round(oracle, [(GPU, 16, 8, 0)], rows, busy=[0x01, 0x00])
    assert list(o["alloc_units"][0]) == [1, 4, 2, 4]
    # 4-chunk -> node 0 block (4,4); 2-chunks (gang, then two replicas) -> (0,2) smallest block,
    # then node 1 split; the single GPU -> the leftover 1-block at (0,1)
    assert (o["place_node"][0, 1], o["place_off"][0, 1]) == (0, 4)
    assert (o["place_node"][0, 2], o["place_off"][0, 2]) == (0, 2)
    assert (o["place_node"][0, 3], o["place_off"][0, 3]) == (1, 0)
    assert (o["place_node"][0, 0], o["place_off"][0, 0]) == (0, 1)


def test_invalid_records_are_flagged(oracle):
    o = _round(oracle, [(CPU, 8, 4, 0)], [(0, 1, 0, 1, 1)])                    # empty level mask
    assert o["status"][0] == 1 and o["n_selected"][0] == 0
    o = _round(oracle, [(CPU, 8, 4, 0)], [(3, 1, 1, 1, 1)])                    # unknown pool
    assert o["status"][0] == 1
    o = _round(oracle, [(GPU, 8, 8, 0)], [(0, 3, 1, 1, 1)])                    # chunk of 3 GPUs
    assert o["status"][0] == 1
    o = _round(oracle, [(GPU, 8, 8, 0)], [(0, 1 | GANG, 0x4, 1, 1)])           # gang level 3 only
    assert o["status"][0] == 1


# ------------------------------------------------------------------ Algorithm 1, eviction loop worked by hand
def test_two_evictions_pay_and_the_third_does_not(oracle):
    # One core pool of 10, four candidates (s, p, levels), nothing else waits, depth 2:
    #   a1 (0, 3600, {1,4,6})   a2 (0, 2400, {1,4,6})   a3 (0, 1200, {3})   a4 (0, 3600, {3,4,6})
    # keep 4: least demand 8, two spare cores; the only level they reach is a4 at 4 (1200 -> 900):
    #         3600 + 2400 + 400 + 900 = 7300, nothing remains                        objective 7300
    # keep 3: a3 takes 3, seven cores for a1, a2: (6,1) = 600 + 2400 beats (4,1) = 3300 and (1,6) = 4000;
    #         completions {600, 2400, 400}; a4 waits: earliest slot 400, second level (4): 400 + 900
    #         3400 + 1300                                                            objective 4700
    # keep 2: (6,4) = 600 + 600; completions {600, 600}; a3 (one level, so only depth 1): 600 + 400 = 1000,
    #         a4 at its least level: 600 + 1200 = 1800;  1200 + 2800                 objective 4000
    # keep 1: a1 at 6 = 600; completions {600}; a2 at its second level (4): 600 + 600 = 1200, a3: 1600,
    #         a4: 2800 (depth 1 would give 3000 + 3400 + 4600);  600 + 5600          objective 6200
    # 7300 > 4700 > 4000 < 6200: two evictions are accepted, the third is not.  Comparing with the
    # initial 7300 would accept the third (6200 < 7300) and keep a1 alone; stopping after the first
    # accepted step would keep three.
    rows = [(0, 1, 0x29, 0, 3600), (0, 1, 0x29, 0, 2400), (0, 1, 0x04, 0, 1200), (0, 1, 0x2C, 0, 3600)]
    o = _round(oracle, [(CPU, 10, 10, 0)], rows, depth=2)
    assert list(o["alloc_units"][0]) == [6, 4, 0, 0]
    assert list(o["act_us"][0]) == [600, 600, -1, -1]
    assert o["n_selected"][0] == 2 and o["total_act_us"][0] == 1200
    # at depth 1 the step to three costs 3400 + (400 + 1200) = 5000 < 7300, the step to two stays 4000,
    # the step to one 600 + 11000: the same two evictions
    o = _round(oracle, [(CPU, 10, 10, 0)], rows, depth=1)
    assert list(o["alloc_units"][0]) == [6, 4, 0, 0]


def test_evicted_candidates_come_before_the_waiting_actions(oracle):
    # Two cores; candidates a1 (0, 2400, {1,2}), a2 (300, 2400, {1,2}); behind them waits w (0, 1200, {1}),
    # which does not fit (the prefix ends before it).  Depth 2.
    # keep 2: 2400 + 2700, completions {2400, 2700}, w: 2400 + 1200 = 3600             objective 8700
    # keep 1: a1 at 2 = 1200, completions {1200}; remaining = [a2, w] (evicted first):
    #         a2 is the first remaining action, so it may try its second level: 1200 + 1500 = 2700,
    #         then w: 2700 + 1200 = 3900;  1200 + 6600                                  objective 7800
    # 7800 < 8700: a2 is evicted.  With w ahead of a2 the first remaining action has one level only:
    # w 2400, a2 at its least level 2400 + 2700 = 5100, objective 1200 + 7500 = 8700, no eviction.
    rows = [(0, 1, 0x3, 0, 2400), (0, 1, 0x3, 300, 2400), (0, 1, 0x1, 0, 1200)]
    o = _round(oracle, [(CPU, 2, 2, 0)], rows, depth=2)
    assert list(o["alloc_units"][0]) == [2, 0, 0]
    assert o["act_us"][0, 0] == 1200 and o["n_selected"][0] == 1


def _replay(oracle, pools, rows, round_us, max_rounds, depth=2):
    from workloads import Pool
    n = len(rows)
    a = dict(pool=np.array([[r[0] for r in rows]], np.uint8), unit=np.array([[r[1] for r in rows]], np.uint8),
             level_mask=np.array([[r[2] for r in rows]], np.uint32), s_us=np.array([[r[3] for r in rows]], np.int64),
             p_us=np.array([[r[4] for r in rows]], np.int64), arrival_us=np.array([[r[5] for r in rows]], np.int64),
             n_actions=np.array([n], np.int32), gpu_busy=None)
    return oracle.replay_trace([Pool(*p) for p in pools], a, depth=depth, round_us=round_us, max_rounds=max_rounds)


def test_running_actions_of_the_same_pool_seed_the_completion_heap(oracle):
    # Rounds every 1000 us.  Pool 0 has three cores, pool 1 one core.  At t = 0: x (pool 0, one core, runs D)
    # and z (pool 1, one core, runs 1001) start.  At t = 1000 two actions y1, y2 = (600, 1000, {1,2}) that
    # arrived at 500 find two free cores on pool 0 and x still running there.
    # keep both: 1600 + 1600 = 3200.
    # keep y1 at 2 cores (1100): completions {D - 1000, 1100}; y2 at its second level:
    #     min(D - 1000, 1100) + 1100;  objective 2200 + min(D - 1000, 1100).
    # D = 1100: 2300 < 3200, y2 is evicted in this round and starts in the next.
    # D = 2100: 3300 >= 3200, both start with one core each.
    # Were the running action left out of the heap the objective would be 3300 for either D; were z's
    # completion (1 us after the round, but on the other pool) let in, it would be 2201 for either D.
    pools = [(CPU, 3, 3, 0), (CPU, 1, 1, 0)]
    for D, evicted in ((1100, True), (2100, False)):
        rows = [(0, 1, 1, D, 0, 0), (1, 1, 1, 1001, 0, 0), (0, 1, 3, 600, 1000, 500), (0, 1, 3, 600, 1000, 500)]
        o = _replay(oracle, pools, rows, 1000, 16)
        assert o["status"][0] == 0
        assert list(o["alloc_units"][0][:2]) == [1, 1] and list(o["act_us"][0][:2]) == [D, 1001]
        if evicted:
            # y1: waited 500, runs 1100 on two cores.  Round 2 (t = 2000): x is gone (finished 1100), y1 runs
            # until 2100 on two cores, one core is free: y2 is the only candidate, takes it, 1600 us:
            # completion 3600 - arrival 500
            assert list(o["alloc_units"][0][2:]) == [2, 1]
            assert list(o["act_us"][0][2:]) == [500 + 1100, 1500 + 1600]
        else:
            assert list(o["alloc_units"][0][2:]) == [1, 1]
            assert list(o["act_us"][0][2:]) == [500 + 1600, 500 + 1600]
        # occupancy after the scheduling of rounds 0 and 1
        assert list(o["occupancy"][0, 0]) == [1, 1]
        assert list(o["occupancy"][0, 1]) == [3, 1]


def test_objective_sums_saturate(oracle):
    # Two cores, n identical actions (2^40, 2^40, {1,2}): T(1) = 2^41, T(2) = 2^40 + 2^39.  The candidates
    # are the first two.  With both kept the n - 2 waiting actions start in pairs every 2^41 us: their
    # completions sum to about 2^41 (n/2)^2.  With one kept there is a single slot and the sum is about
    # 2^40 n^2, twice as much.
    # n = 3500: the first objective is about 2^62.6 and exact, the second passes 2^63 and is clamped to
    # INT64_MAX, which is not smaller: no eviction.  A sum that wrapped around instead would turn
    # negative and win.
    # n = 6000: both objectives are INT64_MAX; equal is not smaller, so again no eviction.
    for n in (3500, 6000):
        rows = [(0, 1, 0x3, 1 << 40, 1 << 40)] * n
        o = _round(oracle, [(CPU, 2, 2, 0)], rows, depth=2)
        assert o["status"][0] == 0 and o["n_selected"][0] == 2
        assert list(o["alloc_units"][0][:3]) == [1, 1, 0]
        assert list(o["act_us"][0][:3]) == [1 << 41, 1 << 41, -1]
        assert o["total_act_us"][0] == 1 << 42
    # parameters beyond 2^40 are clamped to it (R1), so this is the same round
    rows = [(0, 1, 0x3, 1 << 45, 1 << 62)] * 3500
    o = _round(oracle, [(CPU, 2, 2, 0)], rows, depth=2)
    assert list(o["alloc_units"][0][:3]) == [1, 1, 0] and o["total_act_us"][0] == 1 << 42


def test_quota_pool_reports_units_consumed_before_each_grant(oracle):
    # Section 5.1: three calls of 1, 2 and 3 tokens on a quota pool take tokens 0, 1..2 and 3..5
    o = _round(oracle, [(API, 10, 0, 1_000_000)], [(0, 1, 1, 5, 0), (0, 2, 1, 5, 0), (0, 3, 1, 5, 0), (0, 5, 1, 5, 0)])
    assert list(o["alloc_units"][0]) == [1, 2, 3, 0]                 # the fourth call needs 5 of the 4 left
    assert list(o["place_off"][0]) == [0, 1, 3, -1] and list(o["place_node"][0]) == [0, 0, 0, -1]
    # a concurrency-limited pool counts the same way within a round
    o = _round(oracle, [(API, 6, 0, 0)], [(0, 3, 1, 5, 0), (0, 2, 1, 5, 0), (0, 1, 1, 5, 0)])
    assert list(o["place_off"][0]) == [0, 3, 5]
