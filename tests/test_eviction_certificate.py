"""The CUDA path skips both estimates of an eviction step when the step cannot pay (same
allocation for the shorter prefix, evicted candidate not faster at the level the estimate tries).
This checks that claim on the CPU oracle's own pieces: DPArrange for the two prefixes and
estimate() for the two remaining lists, composed here as Algorithm 1, lines 8-14 compose them."""
import numpy as np

CPU = 0


def _dur(s, p, r):
    return int(s) + int(p) // int(r)


def _levels(mask):
    return [r for r in range(1, 33) if mask >> (r - 1) & 1]


def test_step_with_unchanged_allocation_never_lowers_the_objective(oracle):
    rng = np.random.default_rng(5)
    premise = checked = 0
    for trial in range(400):
        m = int(rng.integers(2, 7))
        n_wait = int(rng.integers(0, 12))
        n = m + n_wait
        mask = rng.integers(1, 16, n).astype(np.uint32)          # levels among {1,2,3,4}
        s = rng.integers(0, 400, n)
        p = rng.integers(0, 2000, n)
        unit = np.ones(n, np.uint8)
        need = sum(_levels(int(mk))[0] for mk in mask[:m])
        cap = need + int(rng.integers(0, 3 * m + 1))             # from tight to ample
        depth = int(rng.integers(1, 4))
        rc, value, alloc = oracle.dp_arrange(unit[:m], mask[:m], s[:m], p[:m], pool_type=CPU, capacity=cap,
                                             group=cap, free_units=cap)
        assert rc == 0
        for q in range(m, 1, -1):                                 # step from prefix q to q - 1
            kept, fewer = alloc[q - 1, :q], alloc[q - 2, :q - 1]
            lv = _levels(int(mask[q - 1]))
            tried = lv[min(depth, len(lv)) - 1]
            same = bool(np.array_equal(kept[:q - 1], fewer)) and \
                _dur(s[q - 1], p[q - 1], kept[q - 1]) <= _dur(s[q - 1], p[q - 1], tried)

            def objective(k, al):
                heap = [_dur(s[i], p[i], al[i]) for i in range(k)]
                return int(value[k - 1]) + oracle.estimate(heap, unit[k:], mask[k:], s[k:], p[k:], depth=depth)

            if same:
                premise += 1
                assert objective(q - 1, fewer) >= objective(q, kept), (trial, q)
            checked += 1
    assert premise > 100 and checked - premise > 100             # both kinds of step occurred
