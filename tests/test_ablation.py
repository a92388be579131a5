"""Scheduling ablation on the synthetic coding-like trace: elastic allocation (1..32 cores)
against fixed degrees of parallelism 4 and 16, all through the same scheduler.  The paper
reports the elastic policy ahead of both fixed ones; on this seeded trace the oracle shows the
same order, and the CUDA replay reproduces the oracle bit for bit."""
import numpy as np
import pytest

from workloads import generate, make_workload

NAMES = ("abl_elastic", "abl_dop4", "abl_dop16")


def _mean_act(o):
    act = o["act_us"]
    return float(act[act >= 0].mean())


def test_elastic_beats_fixed_dop_on_the_oracle(oracle):
    means = {}
    for name in NAMES:
        w = make_workload(name, n_scenarios=3, max_actions=2500)
        o = oracle.replay_trace(w.pools, generate(w), depth=w.depth, round_us=w.round_us,
                                max_rounds=w.max_rounds, want_occupancy=False)
        assert np.all(o["status"] == 0) and np.all(o["n_selected"] == 2500)
        means[name] = _mean_act(o)
    assert means["abl_elastic"] < means["abl_dop4"] < means["abl_dop16"]
    assert means["abl_dop16"] > 2.0 * means["abl_elastic"]


@pytest.mark.gpu
@pytest.mark.parametrize("name", NAMES)
def test_ablation_replay_matches_oracle(oracle, name):
    import torch
    from paper_2603_13019_b200 import binding
    w = make_workload(name, n_scenarios=6, max_actions=1500)
    a = generate(w)
    o = oracle.replay_trace(w.pools, a, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds)
    rnd = binding.Round(6, 1500, w.pools, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds)
    out = rnd.replay_trace(binding.to_device(a))
    torch.cuda.synchronize()
    for k in ("status", "n_selected", "total_act_us", "alloc_units", "place_node", "place_off", "act_us",
              "rounds_used", "occupancy"):
        assert np.array_equal(o[k], out[k].cpu().numpy()), k
    rnd.destroy()


@pytest.mark.gpu
def test_sweep_points_match_oracle(oracle):
    # two corners of the capacity / load sweeps (half the cores; twice the arrival rate), all policies
    import torch
    from dataclasses import replace
    from paper_2603_13019_b200 import binding
    from workloads import ablation_sweep
    for cores, rate, pol, w in ablation_sweep():
        if (cores, rate) not in ((128, 110.0), (256, 220.0)):
            continue
        w = replace(w, n_scenarios=3, max_actions=1200)
        a = generate(w)
        o = oracle.replay_trace(w.pools, a, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds)
        rnd = binding.Round(3, 1200, w.pools, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds)
        out = rnd.replay_trace(binding.to_device(a))
        torch.cuda.synchronize()
        for k in ("status", "n_selected", "total_act_us", "alloc_units", "act_us", "rounds_used", "occupancy"):
            assert np.array_equal(o[k], out[k].cpu().numpy()), (w.name, k)
        rnd.destroy()
