"""Writes tests/golden/cfg0_schedule.txt: the oracle's schedule of the smallest named
configuration (one scenario, 64 actions, seed 0).  Calls only the oracle and the input
generator; rerun after a justified change of the oracle and review the diff."""
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

import oracle  # noqa: E402
from workloads import CONFIGS, generate  # noqa: E402


def main() -> None:
    w = CONFIGS["cfg0"]
    a = generate(w)
    o = oracle.schedule_batch(w.pools, a, depth=w.depth)
    with open(os.path.join(HERE, "cfg0_schedule.txt"), "w") as f:
        f.write("# oracle schedule of cfg0 (seed 0): action pool unit mask s_us p_us | alloc node off act_us\n")
        for i in range(w.max_actions):
            f.write("%d %d %d %d %d %d | %d %d %d %d\n" % (
                i, a["pool"][0, i], a["unit"][0, i], a["level_mask"][0, i], a["s_us"][0, i], a["p_us"][0, i],
                o["alloc_units"][0, i], o["place_node"][0, i], o["place_off"][0, i], o["act_us"][0, i]))
        f.write("# total_act_us %d n_selected %d\n" % (o["total_act_us"][0], o["n_selected"][0]))


if __name__ == "__main__":
    main()
