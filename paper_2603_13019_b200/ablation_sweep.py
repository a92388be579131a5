"""Capacity and load sweeps of the scheduling ablation (paper Section 6.4, "Impact of scheduling") on the
synthetic coding-like trace: elastic allocation against fixed degrees of parallelism 4 and 16, through
the device-resident trace replay.

    python -m paper_2603_13019_b200.ablation_sweep [--scenarios 16]

Prints one line per (cores, arrival rate): mean action completion time of the three policies and the
ratios to the elastic one.  Needs a GPU; there is no CPU path."""
from __future__ import annotations

import argparse
import os
import sys
from dataclasses import replace

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main():
    import torch
    from paper_2603_13019_b200 import binding, build
    from workloads import ablation_sweep, generate

    ap = argparse.ArgumentParser()
    ap.add_argument("--scenarios", type=int, default=16)
    args = ap.parse_args()
    build.build()
    rows = {}
    for cores, rate, pol, w in ablation_sweep():
        w = replace(w, n_scenarios=args.scenarios)
        a = generate(w)
        rnd = binding.Round(w.n_scenarios, w.max_actions, w.pools, depth=w.depth, round_us=w.round_us,
                            max_rounds=w.max_rounds)
        out = rnd.replay_trace(binding.to_device(a))
        torch.cuda.synchronize()
        act = out["act_us"]
        done = act >= 0
        rows.setdefault((cores, rate), {})[pol] = (float(act[done].double().mean().item()) / 1e6,
                                                   float(done.double().mean().item()))
        rnd.destroy()
    print("cores  rate/s  elastic_s  dop4_s  dop16_s  dop4/elastic  dop16/elastic  (share of actions finished)")
    for (cores, rate), r in rows.items():
        e, d4, d16 = r["elastic"], r["dop4"], r["dop16"]
        print(f"{cores:5d}  {rate:6.0f}  {e[0]:9.3f}  {d4[0]:6.3f}  {d16[0]:7.3f}  {d4[0] / e[0]:12.2f}  {d16[0] / e[0]:13.2f}"
              f"  ({e[1]:.2f} {d4[1]:.2f} {d16[1]:.2f})")


if __name__ == "__main__":
    main()
