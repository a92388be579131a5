#!/usr/bin/env python
"""Benchmark of the batched elastic scheduling round on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg4] [--impl ours|reference]

A step is one call of tangram_schedule_batch over one batch of synthetic scenarios (every
row of the hot path: duration model, candidate prefix, per-pool selection, placement,
predicted completion times).  Prints ONE JSON line:
  value      actions scheduled per second with inputs resident in HBM (device time, CUDA events)
  e2e        the same through host buffers (host->device and device->host copies timed)
  roofline   algorithmic bytes of a step / measured duration of the step, against the measured HBM
             copy peak; per kernel interval the DRAM bytes ncu counted for it over its own duration
  cpu_baseline  the CPU oracle timed on this machine's cores over a bounded sample
With --impl reference the oracle itself is timed (bounded sample per step) on the host cores.
N > 1 runs one independent replica per GPU (scenarios are independent, no collective on the
data path); timing is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import CONFIGS, generate, make_workload  # noqa: E402

ALGO_BYTES_PER_ACTION = 42        # 22 B read (pool, unit, mask, s, p) + 20 B written (alloc, node, off, act)
METRIC = "actions scheduled/sec (1xB200)"
# DRAM bytes per pending action (dram__bytes_read.sum + dram__bytes_write.sum of one launch / actions of the
# launch) from the ncu capture summarised under profiles/ (cfg4 shape, 2048
# scenarios); traffic grows in proportion to the actions, so a launch's traffic is this times its actions.
# The k_stream interval of the per-kernel timing holds k_fill as well (it runs beside it), the k_finish interval
# k_easy and the certified pools' k_place (beside it), the k_place interval the solver-side pools' placement.
NCU_BYTES_PER_ACTION = {"cfg4": {"k_head": 1.72, "k_stream": 11.70 + 22.48, "k_solve": 1.54, "k_sims": 2.46,
                                 "k_finish": 1.88 + 1.90 + 0.55, "k_place": 0.02 + 0.23}}
NCU_TRAFFIC_SOURCE = "ncu on 2048 scenarios of the same shape, scaled by actions (profiles/)"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def _oracle_call(w, arrays, lo, hi):
    import oracle
    K = int(w.params.get("cache_slots", 0))
    if w.replay:
        return oracle.replay_trace(w.pools, arrays, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds,
                                   lo=lo, hi=hi, want_occupancy=False, cache_slots=K)
    return oracle.schedule_batch(w.pools, arrays, depth=w.depth, lo=lo, hi=hi, cache_slots=K)


def _oracle_throughput(w, arrays, target_s: float, threads: int):
    """Times the oracle, as it stands, on a bounded sample of scenarios; returns (actions/s, sample text)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    oracle.build()
    S = arrays["pool"].shape[0]
    probe = min(S, 2 * threads)
    t0 = time.perf_counter()
    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(lambda sc: _oracle_call(w, arrays, sc, sc + 1), range(probe)))
    dt = time.perf_counter() - t0
    n = int(min(S, max(probe, target_s / max(dt / probe, 1e-9))))
    chunk = max(1, n // (threads * 8))
    starts = list(range(0, n, chunk))
    t0 = time.perf_counter()
    with ThreadPoolExecutor(threads) as ex:
        list(ex.map(lambda lo: _oracle_call(w, arrays, lo, min(n, lo + chunk)), starts))
    dt = time.perf_counter() - t0
    acts = int(arrays["n_actions"][:n].sum())
    return acts / dt, f"first {n} of {S} scenarios of {w.name} ({acts} pending actions), {threads} threads, {dt:.1f} s"


def run_reference(args, w, rank: int):
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    S = min(w.n_scenarios, 256 if w.max_actions >= 4096 else 1024)
    arrays = generate(w, 0, S)
    target = 20.0 / max(args.steps + args.warmup, 1)
    vals, sample = [], ""
    for it in range(args.warmup + args.steps):
        v, sample = _oracle_throughput(w, arrays, target, threads)
        if it >= args.warmup:
            vals.append(v)
    value = float(np.mean(vals))
    acts = S * w.max_actions
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "actions/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": None, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": w.name, "scenarios": w.n_scenarios, "actions_per_scenario": w.max_actions,
                       "note": "CPU oracle on host cores, bounded sample per step"},
            "cpu_baseline": {"value": value, "unit": "actions/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "actions/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps (default: 100 for the single-round configs that take milliseconds, 5 otherwise)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="cfg4", choices=list(CONFIGS))
    ap.add_argument("--scenarios", type=int, default=0, help="override the number of scenarios (smaller runs)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--order", type=int, default=0, choices=[0, 1, 2, 3],
                    help="queue order of a single-round config: 0 first come first served, 1 shortest first, 2 longest first, 3 arrival")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.steps <= 0:
        args.steps = 100 if args.config in ("cfg0", "cfg1", "cfg4", "cfg4_vec", "cfg1_cache") and args.impl == "ours" else 5
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = make_workload(args.config, n_scenarios=args.scenarios or None)

    if args.impl == "reference":
        run_reference(args, w, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2603_13019_b200 import binding, build
    if local_rank == 0:
        build.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    torch.cuda.set_device(local_rank)
    binding.load_library()

    # each rank schedules its own batch of scenarios (seed = base + global scenario id)
    S, N = w.n_scenarios, w.max_actions
    lo = rank * S
    chunk = max(1, min(S, (64 << 20) // N))
    parts = [generate(w, lo + c, lo + min(S, c + chunk)) for c in range(0, S, chunk)]
    # per-action and per-scenario arrays are scenario-major; the cost-vector planes are [entry][scenario][action]
    arrays = {k: (None if parts[0][k] is None else np.concatenate([p[k] for p in parts], axis=1 if k.startswith("side_") else 0))
              for k in parts[0]}
    del parts

    cpu = None
    if rank == 0 and not args.no_cpu_baseline and not args.order:   # the oracle leg times the first-come-first-served round
        threads = os.cpu_count() or 1
        v, sample = _oracle_throughput(w, arrays, 15.0, threads)
        v1, sample1 = _oracle_throughput(w, arrays, 5.0, 1)
        cpu = {"value": v, "unit": "actions/s", "cores": threads, "kind": "oracle", "sample": sample,
               "one_thread": {"value": v1, "unit": "actions/s", "cores": 1, "sample": sample1}}

    dev = binding.to_device(arrays)
    extras = dict(cache_slots=int(w.params.get("cache_slots", 0)), side_costs=int(w.params.get("side_costs", 0)))
    rnd = binding.Round(S, N, w.pools, depth=w.depth, round_us=w.round_us, max_rounds=w.max_rounds, **extras)
    res = rnd.new_result(replay=w.replay)
    stream = torch.cuda.current_stream()
    if args.order and not w.replay:                # the round on the sorted queue (sort, gather, round, scatter)
        _plain = rnd.schedule_batch
        rnd.schedule_batch = lambda a_, now_, res_, st_: rnd.schedule_batch_ordered(a_, args.order, now_, res_, st_)
    if w.replay:                                   # a step of a replay workload = the whole trace
        _sb = rnd.schedule_batch
        rnd.schedule_batch = lambda a_, now_, res_, st_: rnd.replay_trace(a_, res_, st_)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        rnd.schedule_batch(dev, 0, res, stream)
    sync_all()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    rnd.set_profiling(True)
    launches0 = rnd.kernel_launches
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        rnd.schedule_batch(dev, 0, res, stream)
    e1.record(stream)
    sync_all()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    ktimes = rnd.kernel_times()
    launches = rnd.kernel_launches - launches0
    rnd.set_profiling(False)
    act = res["act_us"]
    mean_act = float(act[act >= 0].double().mean().item()) if bool((act >= 0).any().item()) else None
    status_bad = int((res["status"] != 0).sum().item())
    n_sel = int(res["n_selected"].sum().item())

    # end to end through host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e and not any(extras.values()) and not args.order:          # cost vectors and the service cache take device buffers only
        hrnd = binding.Round(S, N, w.pools, depth=w.depth, host_buffers=True, round_us=w.round_us,
                             max_rounds=w.max_rounds)
        hin = binding.to_device(arrays, pin=True)
        hres = hrnd.new_result(replay=w.replay)
        if w.replay:
            hrnd.schedule_batch = lambda a_, now_, res_, st_: hrnd.replay_trace(a_, res_, st_)
        for _ in range(2):
            hrnd.schedule_batch(hin, 0, hres, stream)
        sync_all()
        k_e2e = max(1, min(args.steps, 5))
        h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0.record(stream)
        for _ in range(k_e2e):
            hrnd.schedule_batch(hin, 0, hres, stream)
        h1.record(stream)
        sync_all()
        ems = h0.elapsed_time(h1)
        h2d = sum(t.numel() * t.element_size() for t in hin.values() if t is not None)
        d2h = sum(t.numel() * t.element_size() for t in hres.values())
        e2e = {"ms": ems, "steps": k_e2e, "h2d": h2d, "d2h": d2h}
        hrnd.destroy()

    if world > 1:
        tmax = torch.tensor([ms, e2e["ms"] if e2e else 0.0], device="cuda", dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        ms = float(tmax[0].item())
        if e2e:
            e2e["ms"] = float(tmax[1].item())

    if rank == 0:
        acts = S * N * world
        peak, which = _peaks()
        per_step = {k: v[0] / max(v[1], 1) for k, v in ktimes.items() if v[1]}     # ms of each kernel interval per step
        longest = max(per_step.items(), key=lambda kv: kv[1]) if per_step else ("", 0.0)
        # The roofline fraction is that of the whole step: the algorithmic bytes of one round (42 B per
        # pending action) over the step's duration.  Beside it, per kernel interval, the DRAM bytes that ncu
        # counted for it (scaled by actions) over its own duration.
        step_ms = ms / args.steps
        achieved = ALGO_BYTES_PER_ACTION * S * N / (step_ms * 1e-3) / 1e9
        ncu = NCU_BYTES_PER_ACTION.get(w.name, {})
        on_traffic = {k: {"ms": per_step[k], "dram_bytes": ncu[k] * S * N,
                          "achieved_on_traffic_gbs": ncu[k] * S * N / (per_step[k] * 1e-3) / 1e9,
                          "frac_of_peak": ncu[k] * S * N / (per_step[k] * 1e-3) / 1e9 / peak}
                      for k in per_step if k in ncu and per_step[k] > 0}
        traffic = sum(ncu.values()) * S * N if ncu else None
        line = {
            "metric": METRIC, "value": acts * args.steps / (ms * 1e-3), "unit": "actions/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": w.name, "scenarios_per_gpu": S, "actions_per_scenario": N,
                       "pools": [[p.type, p.capacity, p.group, p.window_us] for p in w.pools], "depth": w.depth,
                       "queue_order": args.order,
                       "l2": "inputs+outputs %.0f MB per step, larger than L2" % (ALGO_BYTES_PER_ACTION * S * N / 1e6)
                       if ALGO_BYTES_PER_ACTION * S * N > 126e6 else "working set below L2; no flush",
                       "parallelism": "independent replicas" if world > 1 else "single GPU",
                       "selected_actions": n_sel, "scenarios_with_status": status_bad,
                       "mean_act_us": mean_act},
            "clocks": clocks,
            "e2e": None if e2e is None else {"value": acts * e2e["steps"] / (e2e["ms"] * 1e-3), "unit": "actions/s",
                                             "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                                             "ms_per_step": e2e["ms"] / e2e["steps"]},
            "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": "whole step (%s)" % ", ".join(sorted(per_step)),
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "frac_nominal_8TBs": achieved / 8000.0,
                         "traffic": traffic,
                         "traffic_source": NCU_TRAFFIC_SOURCE if traffic else None,
                         "peak_source": which, "longest_kernel": longest[0],
                         "kernel_ms": per_step, "per_kernel": on_traffic},
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    rnd.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
