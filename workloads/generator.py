"""Counter-based generator of scheduling-round inputs (see package docstring).

Record layout (structure of arrays, scenario-major, row stride = max_actions):

  pool        u8   index into the workload's pool list
  unit        u8   low 7 bits: unit multiplier g (units per multiplicity step);
                   bit 7 (GANG): on a GPU pool the g*r units of a level form ONE
                   contiguous aligned chunk; without it a level is r chunks of g
  level_mask  u32  bit (r-1) set  <=>  multiplicity r (1..32) is allowed
  s_us, p_us  i64  runtime parameters in microseconds (invariant / scalable part)
  arrival_us  i64  arrival time (replay workloads only, non-decreasing per row)
  n_actions   i32  per scenario
  gpu_busy    u8   per scenario x node (all GPU pools' nodes concatenated in pool
                   order): bit b set <=> GPU b of that node is occupied beforehand

Actions of one scenario are stored in queue (first-come first-served) order.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np

POOL_CPU, POOL_GPU, POOL_API = 0, 1, 2
GANG = 0x80

_U = np.uint64


@dataclass(frozen=True)
class Pool:
    type: int          # POOL_CPU | POOL_GPU | POOL_API
    capacity: int      # cores | GPUs | tokens per window (or concurrent calls)
    group: int         # CPU: cores per NUMA domain; GPU: GPUs per node; API: 0
    window_us: int = 0  # API quota period; 0 = concurrency limited


@dataclass(frozen=True)
class Workload:
    name: str
    n_scenarios: int
    max_actions: int
    pools: Tuple[Pool, ...]
    recipe: str
    base_seed: int = 0
    depth: int = 2
    round_us: int = 10_000
    replay: bool = False
    max_rounds: int = 0
    params: Dict[str, float] = field(default_factory=dict)

    @property
    def n_nodes(self) -> int:
        return sum(p.capacity // p.group for p in self.pools if p.type == POOL_GPU)


# --------------------------------------------------------------------------- RNG
def _splitmix64(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = x + _U(0x9E3779B97F4A7C15)
        z = (z ^ (z >> _U(30))) * _U(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> _U(27))) * _U(0x94D049BB133111EB)
        return z ^ (z >> _U(31))


class _Draws:
    """Random fields of a [scenario, action] grid; field ids select independent streams."""

    def __init__(self, base_seed: int, lo: int, hi: int, n_cols: int, salt: int = 0):
        sc = (np.arange(lo, hi, dtype=np.uint64) + _U(base_seed % (1 << 63)))[:, None]
        col = np.arange(n_cols, dtype=np.uint64)[None, :]
        with np.errstate(over="ignore"):
            h0 = _splitmix64(sc ^ (_U(salt) * _U(0x632BE59BD9B4E019)))
            self._h1 = _splitmix64(h0 ^ (col * _U(0xD1342543DE82EF95)))

    def bits(self, fid: int) -> np.ndarray:
        with np.errstate(over="ignore"):
            return _splitmix64(self._h1 + _U(fid) * _U(0xA24BAED4963EE407))

    def uniform(self, fid: int) -> np.ndarray:
        return ((self.bits(fid) >> _U(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)

    def normal(self, fid: int) -> np.ndarray:
        u1, u2 = self.uniform(fid), self.uniform(fid + 1)
        return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)

    def lognormal_us(self, fid: int, median: float, sigma: float) -> np.ndarray:
        v = np.exp(np.log(median) + sigma * self.normal(fid))
        return np.minimum(np.floor(v), float(1 << 40)).astype(np.int64)


# fixed field ids (two consecutive ids are consumed by a normal draw)
_F_POOL, _F_INEL, _F_LEVEL, _F_S, _F_P, _F_OUT, _F_SIZE, _F_ARR, _F_DUR, _F_BUSY = (
    1, 2, 3, 4, 6, 8, 9, 10, 11, 12)
_F_MEM, _F_TOKEN, _F_SERVICE, _F_RESTORE, _F_CTAG, _F_CUSE = 40, 41, 42, 43, 44, 45


def _pow2_mask(max_level: int) -> int:
    m, r = 0, 1
    while r <= max_level:
        m |= 1 << (r - 1)
        r *= 2
    return m


def _choose(u: np.ndarray, probs) -> np.ndarray:
    edges = np.cumsum(np.asarray(probs, dtype=np.float64))
    edges[-1] = 1.0 + 1e-9
    return np.searchsorted(edges, u, side="right").astype(np.uint8)


def _single_pow2_level(u: np.ndarray, n_levels: np.ndarray) -> np.ndarray:
    """mask with exactly one power-of-two multiplicity, index uniform in [0, n_levels)."""
    idx = np.minimum((u * n_levels).astype(np.int64), n_levels - 1)
    r = np.left_shift(np.int64(1), idx)
    return np.left_shift(np.uint32(1), (r - 1).astype(np.uint32)).astype(np.uint32)


# --------------------------------------------------------------------- recipes
def _mixed_round(w: Workload, d: _Draws, S: int, N: int):
    """Configs 0, 1, 4: independent single rounds over CPU / GPU(gang) / API pools."""
    P = w.params
    pool = _choose(d.uniform(_F_POOL), P["mix"])
    ptype = np.array([p.type for p in w.pools], dtype=np.int64)[pool]
    # highest power-of-two multiplicity per pool ("capped by pool")
    cap_level = np.array(
        [min(P["max_level"], 8 if p.type == POOL_GPU else P["max_level"]) if p.type != POOL_API else 1
         for p in w.pools], dtype=np.int64)[pool]
    n_levels = np.floor(np.log2(cap_level)).astype(np.int64) + 1
    full_mask = np.array([_pow2_mask(int(c)) for c in range(0, 33)], dtype=np.uint32)[cap_level]
    inelastic = (d.uniform(_F_INEL) < P["inelastic"]) | (ptype == POOL_API)
    one = _single_pow2_level(d.uniform(_F_LEVEL), n_levels)
    mask = np.where(inelastic, one, full_mask).astype(np.uint32)
    unit = np.where(ptype == POOL_GPU, 1 | GANG, 1).astype(np.uint8)
    s = d.lognormal_us(_F_S, 20_000.0, P["sigma_s"])
    p = d.lognormal_us(_F_P, 200_000.0, P["sigma_p"])
    if P.get("outliers", 0.0) > 0.0:
        big = d.uniform(_F_OUT) < P["outliers"]
        s = np.where(big, np.minimum(s * 100, 1 << 40), s)
        p = np.where(big, np.minimum(p * 100, 1 << 40), p)
    return dict(pool=pool, unit=unit, level_mask=mask, s_us=s, p_us=p, arrival_us=None)


def _topology_round(w: Workload, d: _Draws, S: int, N: int):
    """Config 3: one GPU pool, chunk size 1/2/4/8, elastic replica count 1..4."""
    P = w.params
    size_idx = _choose(d.uniform(_F_SIZE), P["size_probs"]).astype(np.int64)
    unit = np.left_shift(np.int64(1), size_idx).astype(np.uint8)            # g = chunk size, no GANG
    mask = np.full((S, N), (1 << int(P["max_replicas"])) - 1, dtype=np.uint32)
    s = d.lognormal_us(_F_S, 20_000.0, P["sigma_s"])
    p = d.lognormal_us(_F_P, 200_000.0, P["sigma_p"])
    return dict(pool=np.zeros((S, N), np.uint8), unit=unit, level_mask=mask, s_us=s, p_us=p,
                arrival_us=None)


def _replay_trace(w: Workload, d: _Draws, S: int, N: int):
    """Config 2: Poisson arrivals; CPU code execution (Pareto) and GPU reward model (uniform)."""
    P = w.params
    gap = np.floor(-np.log(d.uniform(_F_ARR)) * (1e6 / P["rate_per_s"])).astype(np.int64)
    arrival = np.cumsum(gap, axis=1)
    is_gpu = d.uniform(_F_POOL) >= P["cpu_fraction"]
    u = d.uniform(_F_DUR)
    t_cpu = np.minimum(np.floor(P["pareto_min_us"] * u ** (-1.0 / P["pareto_alpha"])), float(1 << 40))
    t_gpu = np.floor(P["gpu_lo_us"] + u * (P["gpu_hi_us"] - P["gpu_lo_us"]))
    t_cpu, t_gpu = t_cpu.astype(np.int64), t_gpu.astype(np.int64)
    s_gpu = t_gpu // 5
    s = np.where(is_gpu, s_gpu, t_cpu)
    p = np.where(is_gpu, t_gpu - s_gpu, 0)
    pool = is_gpu.astype(np.uint8)                                            # pool 0 CPU, 1 GPU
    unit = np.where(is_gpu, 1 | GANG, 1).astype(np.uint8)
    mask = np.where(is_gpu, _pow2_mask(8), 1).astype(np.uint32)
    return dict(pool=pool, unit=unit, level_mask=mask, s_us=s, p_us=p, arrival_us=arrival)


def _ablation_trace(w: Workload, d: _Draws, S: int, N: int):
    """Scheduling ablation (elastic against fixed degree of parallelism) on a coding-like trace:
    one CPU pool; short one-core code executions and long, parallelisable reward calculations
    (5 % serial part).  params["dop"] = 0 makes the reward calculations elastic over
    1, 2, 4, ..., 32 cores, any other value pins them to that many cores."""
    P = w.params
    gap = np.floor(-np.log(d.uniform(_F_ARR)) * (1e6 / P["rate_per_s"])).astype(np.int64)
    arrival = np.cumsum(gap, axis=1)
    reward = d.uniform(_F_POOL) < P["reward_fraction"]
    t_exec = np.minimum(np.floor(P["pareto_min_us"] * d.uniform(_F_DUR) ** (-1.0 / P["pareto_alpha"])),
                        float(1 << 40)).astype(np.int64)
    t_rew = d.lognormal_us(_F_S, P["reward_median_us"], P["reward_sigma"])
    s_rew = t_rew // 20
    s = np.where(reward, s_rew, t_exec)
    p = np.where(reward, t_rew - s_rew, 0)
    dop = int(P["dop"])
    rew_mask = _pow2_mask(32) if dop == 0 else 1 << (dop - 1)
    mask = np.where(reward, rew_mask, 1).astype(np.uint32)
    return dict(pool=np.zeros((S, N), np.uint8), unit=np.ones((S, N), np.uint8), level_mask=mask,
                s_us=s, p_us=p, arrival_us=arrival)


_RECIPES = {"mixed": _mixed_round, "topology": _topology_round, "replay": _replay_trace,
            "ablation": _ablation_trace}


def _busy_masks(w: Workload, lo: int, hi: int) -> Optional[np.ndarray]:
    """Pre-occupied GPUs as aligned chunks: every aligned block of 8, 4, 2, 1 GPUs is
    independently occupied with the same probability q, (1-q)^4 = 1 - busy_fraction."""
    frac = w.params.get("busy_fraction", 0.0)
    nodes = w.n_nodes
    if nodes == 0:
        return None
    out = np.zeros((hi - lo, nodes), dtype=np.uint8)
    if frac <= 0.0:
        return out
    q = 1.0 - (1.0 - frac) ** 0.25
    d = _Draws(w.base_seed, lo, hi, nodes * 15, salt=7)
    u = d.uniform(_F_BUSY).reshape(hi - lo, nodes, 15) < q
    k = 0
    for size in (8, 4, 2, 1):
        for start in range(0, 8, size):
            bits = np.uint8(((1 << size) - 1) << start)
            out |= np.where(u[:, :, k], bits, np.uint8(0))
            k += 1
    # nodes narrower than 8 GPUs: drop bits beyond the group
    col = 0
    for p in w.pools:
        if p.type == POOL_GPU:
            n = p.capacity // p.group
            out[:, col:col + n] &= np.uint8((1 << p.group) - 1)
            col += n
    return out


# ------------------------------------------------------------------- configs
_CPU_NUMA = 64
CONFIGS: Dict[str, Workload] = {
    # single round, one scenario, 64 actions, levels {1,2,4,8}
    "cfg0": Workload("cfg0", 1, 64, (Pool(POOL_CPU, 256, _CPU_NUMA), Pool(POOL_GPU, 8, 8)), "mixed",
                     params=dict(mix=(0.5, 0.5), max_level=8, inelastic=0.0, sigma_s=1.0, sigma_p=1.2)),
    # batched rounds, 4096 x 1024, CPU / GPU 8x8 / API 512 per second
    "cfg1": Workload("cfg1", 4096, 1024,
                     (Pool(POOL_CPU, 4096, _CPU_NUMA), Pool(POOL_GPU, 64, 8), Pool(POOL_API, 512, 0, 1_000_000)),
                     "mixed", params=dict(mix=(0.60, 0.25, 0.15), max_level=16, inelastic=0.20,
                                          sigma_s=1.5, sigma_p=1.5)),
    # trace replay, 256 x 20000, Poisson 50/s, 10 ms rounds
    "cfg2": Workload("cfg2", 256, 20000, (Pool(POOL_CPU, 256, _CPU_NUMA), Pool(POOL_GPU, 8, 8)), "replay",
                     replay=True, max_rounds=60_000,
                     params=dict(rate_per_s=50.0, cpu_fraction=0.70, pareto_alpha=1.3, pareto_min_us=5_000.0,
                                 gpu_lo_us=50_000.0, gpu_hi_us=800_000.0)),
    # topology constrained GPU pool, 1024 x 2048, 64 nodes x 8, 30 % pre-occupied
    "cfg3": Workload("cfg3", 1024, 2048, (Pool(POOL_GPU, 512, 8),), "topology",
                     params=dict(size_probs=(0.4, 0.3, 0.2, 0.1), max_replicas=4, busy_fraction=0.30,
                                 sigma_s=1.0, sigma_p=1.2)),
    # large mixed, 16384 x 4096, four pools
    "cfg4": Workload("cfg4", 16384, 4096,
                     (Pool(POOL_CPU, 8192, _CPU_NUMA), Pool(POOL_GPU, 128, 8),
                      Pool(POOL_API, 1000, 0, 1_000_000), Pool(POOL_API, 200, 0, 1_000_000)),
                     "mixed", params=dict(mix=(0.50, 0.25, 0.15, 0.10), max_level=32, inelastic=0.35,
                                          sigma_s=2.0, sigma_p=2.0, outliers=0.01)),
}


# cfg4 with cost vectors (Section 4.1): a concurrency pool of 2048 memory units is added; every action of
# the core pool asks 1 .. 32 units of it beside its cores, and three in ten GPU actions one token of the
# second quota pool (a tool call made while the service runs)
CONFIGS["cfg4_vec"] = Workload("cfg4_vec", 16384, 4096, CONFIGS["cfg4"].pools + (Pool(POOL_API, 2048, 0, 0),), "mixed",
                               params=dict(CONFIGS["cfg4"].params, mix=(0.50, 0.25, 0.15, 0.10, 0.0), side_costs=2,
                                           mem_pool=4, mem_max=32, token_pool=3, token_fraction=0.3))
# cfg1 with the service cache of the GPU pool (Section 5.3): 6 services (24 instances with the four chunk sizes), every GPU remembers two instances,
# restoration takes 0.5 .. 4 s, two thirds of the entries start filled
CONFIGS["cfg1_cache"] = Workload("cfg1_cache", 4096, 1024, CONFIGS["cfg1"].pools, "mixed",
                                 params=dict(CONFIGS["cfg1"].params, cache_slots=2, n_services=6,
                                             restore_lo_us=500_000.0, restore_hi_us=4_000_000.0, cache_fill=0.67))


def _ablation(dop: int, cores: int = 256, rate_per_s: float = 110.0, name: Optional[str] = None) -> Workload:
    return Workload(name or ("abl_dop%d" % dop if dop else "abl_elastic"), 64, 4000, (Pool(POOL_CPU, cores, _CPU_NUMA),),
                    "ablation", replay=True, max_rounds=12_000,
                    params=dict(rate_per_s=rate_per_s, reward_fraction=0.20, pareto_alpha=1.3, pareto_min_us=5_000.0,
                                reward_median_us=4_000_000.0, reward_sigma=1.0, dop=dop))


def ablation_sweep():
    """The capacity and load sweeps of the scheduling ablation: the same trace recipe at 0.5x, 1x and
    2x the cores and at 0.5x, 1x and 2x the arrival rate (the rate stands in for the batch size of
    the paper's sweep: more trajectories in flight submit more actions per second), each for the
    elastic policy and the two fixed degrees of parallelism.  Yields (cores, rate, policy, workload)."""
    for cores, rate in ((128, 110.0), (256, 110.0), (512, 110.0), (256, 55.0), (256, 220.0)):
        for dop in (0, 4, 16):
            pol = "dop%d" % dop if dop else "elastic"
            yield cores, rate, pol, _ablation(dop, cores, rate, "abl_%s_c%d_r%d" % (pol, cores, int(rate)))


# scheduling ablation on a synthetic coding-like trace: elastic 1..32 against fixed DoP 4 and 16
for _d in (0, 4, 16):
    _w = _ablation(_d)
    CONFIGS[_w.name] = _w


def make_workload(name: str, n_scenarios: Optional[int] = None, max_actions: Optional[int] = None,
                  base_seed: Optional[int] = None) -> Workload:
    """A named configuration, optionally shrunk (same recipe, fewer scenarios / actions)."""
    w = CONFIGS[name]
    kw = {}
    if n_scenarios is not None:
        kw["n_scenarios"] = int(n_scenarios)
    if max_actions is not None:
        kw["max_actions"] = int(max_actions)
    if base_seed is not None:
        kw["base_seed"] = int(base_seed)
    if not kw:
        return w
    from dataclasses import replace
    return replace(w, **kw)


def generate(w: Workload, lo: int = 0, hi: Optional[int] = None) -> Dict[str, Optional[np.ndarray]]:
    """Input arrays of scenarios [lo, hi) of workload `w` (host numpy arrays, C contiguous)."""
    hi = w.n_scenarios if hi is None else hi
    S, N = hi - lo, w.max_actions
    d = _Draws(w.base_seed, lo, hi, N)
    a = _RECIPES[w.recipe](w, d, S, N)
    a["n_actions"] = np.full(S, N, dtype=np.int32)
    a["gpu_busy"] = _busy_masks(w, lo, hi)
    for k in ("pool", "unit", "level_mask", "s_us", "p_us", "arrival_us"):
        if a[k] is not None:
            a[k] = np.ascontiguousarray(a[k])
    P = w.params
    if P.get("side_costs", 0):                       # further entries of the cost vectors
        ptype = np.array([p.type for p in w.pools], dtype=np.int64)[a["pool"]]
        sp = np.full((int(P["side_costs"]), S, N), 0xFF, np.uint8)
        su = np.zeros((int(P["side_costs"]), S, N), np.uint16)
        cpu = ptype == POOL_CPU
        sp[0] = np.where(cpu, P["mem_pool"], 0xFF)
        su[0] = np.where(cpu, 1 + (d.uniform(_F_MEM) * P["mem_max"]).astype(np.int64), 0)
        tok = (ptype == POOL_GPU) & (d.uniform(_F_TOKEN) < P["token_fraction"])
        sp[1] = np.where(tok, P["token_pool"], 0xFF)
        su[1] = np.where(tok, 1, 0)
        a["side_pool"], a["side_units"] = sp, su
    if P.get("cache_slots", 0):                      # services and the cache state of the GPU pools
        K = int(P["cache_slots"])
        a["service"] = (d.uniform(_F_SERVICE) * P["n_services"]).astype(np.uint16)
        a["restore_us"] = (P["restore_lo_us"] + d.uniform(_F_RESTORE) * (P["restore_hi_us"] - P["restore_lo_us"])).astype(np.int64)
        # a node's GPUs start with the same instances (what earlier whole-node or aligned runs left behind)
        dc = _Draws(w.base_seed, lo, hi, w.n_nodes * K, salt=7)
        inst = (dc.uniform(_F_CTAG) * P["n_services"]).astype(np.int64) * 8 + (dc.bits(_F_SERVICE) % _U(4)).astype(np.int64)
        tag = np.where(dc.uniform(_F_CUSE) < P["cache_fill"], inst + 1, 0).astype(np.uint32)
        use = -(dc.bits(_F_CUSE + 1) % _U(1_000_000)).astype(np.int64)
        per_gpu = lambda x: np.ascontiguousarray(np.broadcast_to(x.reshape(S, w.n_nodes, 1, K), (S, w.n_nodes, 8, K))).reshape(S, -1)
        a["cache_tag"], a["cache_use"] = per_gpu(tag), per_gpu(use)
    return a


# ------------------------------------------------- randomized rounds for tests
def random_round(seed: int, n_scenarios: int, max_actions: int, pools: Tuple[Pool, ...],
                 *, contiguous_levels: float = 0.3, max_mult: int = 8, inelastic: float = 0.25,
                 small_durations: float = 0.0, busy_fraction: float = 0.0, ragged: bool = True,
                 replicas: float = 0.5, narrow: bool = True) -> Tuple[Workload, Dict[str, Optional[np.ndarray]]]:
    """Adversarial little rounds for parity and property tests: arbitrary level masks
    (power-of-two sets, contiguous ranges, random subsets), mixed gang/replica GPU
    requests, ragged action counts, optional tiny durations (forces ties) and
    pre-occupied GPUs.  With narrow=False the masks are left as drawn: replica requests with up
    to max_mult multiplicities, gang requests whose masks hold unusable levels among usable
    ones (and sometimes none, which makes the record invalid), elastic quota actions."""
    rng = np.random.Generator(np.random.PCG64(seed))
    S, N = n_scenarios, max_actions
    w = Workload(f"random{seed}", S, N, tuple(pools), "random", base_seed=seed,
                 params=dict(busy_fraction=busy_fraction))
    pool = rng.integers(0, len(pools), size=(S, N)).astype(np.uint8)
    ptype = np.array([p.type for p in pools])[pool]
    kind = rng.random((S, N))
    r_hi = rng.integers(1, max_mult + 1, size=(S, N))
    r_lo = np.minimum(rng.integers(1, max_mult + 1, size=(S, N)), r_hi)
    contiguous = ((np.int64(1) << r_hi) - 1) & ~((np.int64(1) << (r_lo - 1)) - 1)
    pow2 = np.array([_pow2_mask(int(c)) for c in range(0, 33)], dtype=np.int64)[r_hi]
    subset = rng.integers(1, 1 << max_mult, size=(S, N))
    mask = np.where(kind < contiguous_levels, contiguous, np.where(kind < 0.8, pow2, subset))
    single = np.int64(1) << (rng.integers(0, max_mult, size=(S, N)))
    mask = np.where(rng.random((S, N)) < inelastic, single, mask)
    unit = np.ones((S, N), dtype=np.int64)
    is_gpu = ptype == POOL_GPU
    rep = is_gpu & (rng.random((S, N)) < replicas)
    grp = np.array([max(p.group, 1) for p in pools], dtype=np.int64)[pool]
    unit = np.where(rep, np.minimum(np.int64(1) << rng.integers(0, 4, size=(S, N)), grp), unit)
    unit = np.where(is_gpu & ~rep, 1 | GANG, unit)
    # gang requests need power-of-two levels <= GPUs per node; replicas keep few multiplicities
    if narrow:
        gang_ok = np.array([_pow2_mask(int(c)) for c in range(0, 33)], dtype=np.int64)[np.minimum(grp, 32)]
        mask = np.where(is_gpu & ~rep, mask & gang_ok, mask)
        mask = np.where(is_gpu & ~rep & (mask == 0), 1, mask)
        mask = np.where(rep, mask & 0xF, mask)
        mask = np.where(rep & (mask == 0), 1, mask)
        mask = np.where(ptype == POOL_API, 1, mask)
    else:
        # most gang records keep a usable level (one GPU); the few that do not are invalid records
        mask = np.where(is_gpu & ~rep & (rng.random((S, N)) < 0.97), mask | 1, mask)
    if small_durations > 0.0:
        tiny = rng.random((S, N)) < small_durations
    else:
        tiny = np.zeros((S, N), dtype=bool)
    s = np.where(tiny, rng.integers(0, 4, size=(S, N)), rng.integers(0, 50_000, size=(S, N)))
    p = np.where(tiny, rng.integers(0, 12, size=(S, N)), rng.integers(0, 500_000, size=(S, N)))
    n_act = rng.integers(0, N + 1, size=S).astype(np.int32) if ragged else np.full(S, N, np.int32)
    a = dict(pool=pool, unit=unit.astype(np.uint8), level_mask=mask.astype(np.uint32),
             s_us=s.astype(np.int64), p_us=p.astype(np.int64), arrival_us=None, n_actions=n_act)
    a["gpu_busy"] = _busy_masks(w, 0, S)
    for k in ("pool", "unit", "level_mask", "s_us", "p_us"):
        a[k] = np.ascontiguousarray(a[k])
    return w, a


def add_side_costs(seed: int, arrays: Dict[str, Optional[np.ndarray]], pools: Tuple[Pool, ...], n_side: int = 2,
                   fraction: float = 0.5, max_share: float = 0.2, invalid: float = 0.0) -> Dict[str, Optional[np.ndarray]]:
    """Further entries of the actions' cost vectors (Section 4.1): returns a copy of `arrays` with
    "side_pool" (uint8, 0xff = none) and "side_units" (uint16), both [n_side][scenario][action].  An entry
    names a quota / concurrency pool other than the action's own with an amount of up to max_share of its
    capacity; `invalid` is the probability of an entry being drawn without these restrictions."""
    rng = np.random.Generator(np.random.PCG64(seed))
    S, N = arrays["pool"].shape
    api = [j for j, p in enumerate(pools) if p.type == POOL_API]
    sp = np.full((n_side, S, N), 0xFF, np.uint8)
    su = np.zeros((n_side, S, N), np.uint16)
    caps = np.array([p.capacity for p in pools], dtype=np.int64)
    for e in range(n_side):
        if not api:
            break
        k = np.array(api, dtype=np.int64)[rng.integers(0, len(api), size=(S, N))]
        on = (rng.random((S, N)) < fraction) & (k != arrays["pool"])
        amount = 1 + (rng.random((S, N)) * np.maximum(caps[k] * max_share - 1, 0)).astype(np.int64)
        wild = rng.random((S, N)) < invalid
        k = np.where(wild, rng.integers(0, len(pools) + 1, size=(S, N)), k)
        amount = np.where(wild, rng.integers(0, 3, size=(S, N)) * caps[np.minimum(k, len(pools) - 1)], amount)
        sp[e] = np.where(on | wild, k, 0xFF).astype(np.uint8)
        su[e] = np.where(on | wild, np.minimum(amount, 65535), 0).astype(np.uint16)
    out = dict(arrays)
    out["side_pool"], out["side_units"] = sp, su
    return out


def add_trajectories(seed: int, arrays: Dict[str, Optional[np.ndarray]], pools: Tuple[Pool, ...], max_traj: int,
                     fraction: float = 0.9, mem_hi: int = 64, pinned: float = 0.3,
                     mem_free_hi: int = 600) -> Dict[str, Optional[np.ndarray]]:
    """Trajectories for the per-node CPU scheduling (Section 5.2): returns a copy of `arrays` with "trajectory"
    (int32 per action, -1 = none), "traj_mem" (uint32, memory of the whole trajectory), "traj_last" (uint8, marks
    the last action of nine in ten trajectories), and the state
    "traj_node" ([scenario][max_traj], a fraction already pinned to a random CPU pool) and "node_mem_free"
    ([scenario][pool])."""
    rng = np.random.Generator(np.random.PCG64(seed))
    S, N = arrays["pool"].shape
    cpu = np.array([j for j, p in enumerate(pools) if p.type == POOL_CPU], dtype=np.int64)
    traj = np.where(rng.random((S, N)) < fraction, rng.integers(0, max_traj, size=(S, N)), -1).astype(np.int32)
    per_traj_mem = rng.integers(0, mem_hi + 1, size=(S, max_traj))
    mem = np.take_along_axis(per_traj_mem, np.maximum(traj, 0).astype(np.int64), axis=1).astype(np.uint32)
    node = np.where(rng.random((S, max_traj)) < pinned, cpu[rng.integers(0, len(cpu), size=(S, max_traj))], -1).astype(np.int32)
    out = dict(arrays)
    out["trajectory"], out["traj_mem"], out["traj_node"] = traj, mem, node
    out["node_mem_free"] = rng.integers(0, mem_free_hi + 1, size=(S, len(pools))).astype(np.int64)
    # the last action of most trajectories is marked (a trace gives the memory back when it ends)
    last = np.zeros((S, N), np.uint8)
    n_act = arrays["n_actions"]
    for sc in range(S):
        seen = set()
        for i in range(int(n_act[sc]) - 1, -1, -1):
            t = int(traj[sc, i])
            if t >= 0 and t not in seen:
                seen.add(t)
                last[sc, i] = 1
    out["traj_last"] = np.where(rng.random((S, N)) < 0.9, last, 0).astype(np.uint8)
    return out


def contiguous_replica_round(seed: int, n_scenarios: int, max_actions: int, nodes: int, max_mult: int,
                             *, small_durations: float = 0.0, busy_fraction: float = 0.3
                             ) -> Tuple[Workload, Dict[str, Optional[np.ndarray]]]:
    """Rounds on one fragmented GPU pool whose actions all ask for replicas (chunks of 1, 2, 4 or 8
    GPUs with the probabilities of config 3) with CONTIGUOUS multiplicities lo..hi, hi up to
    max_mult: many candidates with many upgrade steps each.  Tiny durations make the floor of the
    duration model break the monotony of the gains and produce ties."""
    rng = np.random.Generator(np.random.PCG64(seed))
    S, N = n_scenarios, max_actions
    pools = (Pool(POOL_GPU, 8 * nodes, 8),)
    w = Workload(f"contig{seed}", S, N, pools, "random", base_seed=seed, params=dict(busy_fraction=busy_fraction))
    unit = (1 << rng.choice(4, size=(S, N), p=[0.4, 0.3, 0.2, 0.1])).astype(np.uint8)
    hi = rng.integers(1, max_mult + 1, size=(S, N))
    lo = np.where(rng.random((S, N)) < 0.8, 1, np.minimum(2, hi))
    mask = (((np.int64(1) << hi) - 1) & ~((np.int64(1) << (lo - 1)) - 1)).astype(np.uint32)
    tiny = rng.random((S, N)) < small_durations
    s = np.where(tiny, rng.integers(0, 4, (S, N)), rng.integers(0, 50_000, (S, N))).astype(np.int64)
    p = np.where(tiny, rng.integers(0, 40, (S, N)), rng.integers(0, 500_000, (S, N))).astype(np.int64)
    a = dict(pool=np.zeros((S, N), np.uint8), unit=unit, level_mask=mask, s_us=s, p_us=p, arrival_us=None,
             n_actions=np.full(S, N, np.int32))
    a["gpu_busy"] = _busy_masks(w, 0, S)
    return w, a
