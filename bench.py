#!/usr/bin/env python
"""Benchmark of the batched WWW.Serve network step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path over one batch: advance -> gossip (on the steps its
cadence selects) -> dispatch -> duel-and-judge -> settle.  Metric: simulated requests
dispatched and settled per second.  One JSON line is printed by rank 0.

Multi-GPU (`torchrun`, one process per GPU): replicas are independent, so every rank runs its
own set of replicas (weak scaling, no data-path collective); timing is the max over ranks.
`--impl reference` times the CPU oracle, as it stands, on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "simulated requests dispatched+settled per second"
UNIT = "requests/s"
DEFAULT_WORKLOAD = "adversarial16k"          # the largest single-GPU configuration


# DRAM traffic (read + write) of one k_gossip_merge pass over one replica, from the ncu capture
# summarised in profiles/k_gossip_merge_adversarial16k_1replica.md; a launch over Rp replicas is
# Rp such passes back to back (replica-major grid), so traffic scales with the replica count.
NCU_MERGE_TRAFFIC = {"n_peers": 16384, "fanout_k": 4, "flags": 3, "bytes_per_replica": 2.1897e9 + 2.1133e9}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in out.strip().splitlines():
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def step_args(wl, s, phase=0):
    """(first, count, now_ms, gossip) of global step s; the request stream is reused cyclically
    while simulated time keeps growing.  Gossip runs on the steps `phase`, `phase` + cadence, ...:
    the timed steps start on a gossip step, so K timed steps hold ceil(K / cadence) rounds whatever
    the warm-up count (never fewer than the workload's cadence asks for)."""
    n = wl.n_steps
    cyc, k = divmod(s, n)
    first = k * wl.batch
    cnt = min(wl.batch, wl.n_requests - first)
    t_end = int(wl.requests["t_ms"][0, -1]) + 1
    return first, cnt, cyc * t_end + wl.step_now_ms(k), (s - phase) % wl.gossip_every == 0


def algorithmic_bytes(wl, stats_delta):
    """Bytes the method must move (stated in the design notes):
    gossip round: 2 * 8 * N^2 per replica (every view entry read once and written once; the
    k+1 readers of a row share it through L2 because the merge walks the matrix by column panels);
    request path: 8 B record + 26 B result, plus a 256 B view window per request that offloads."""
    st = wl.settings
    gossip_round = 2 * 8 * st.n_peers ** 2 * st.n_replicas
    offloaded = stats_delta["n_delegated"] + stats_delta["n_fallback_local"] + stats_delta["n_failed"]
    req = stats_delta["n_requests"] * (8 + 26) + offloaded * 256
    return gossip_round, req


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2603_20661_b200 import synth
    from paper_2603_20661_b200.binding import Network, STAT_NAMES

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    from paper_2603_20661_b200.sharding import max_over_ranks, replica_shard, sum_counters
    wl0 = synth.make_workload(args.workload, seed=args.seed, n_replicas=args.replicas)
    Rp = wl0.settings.n_replicas
    # weak scaling: every rank runs the configuration's full replica count, on its own replica indices
    off, _ = replica_shard(world * Rp, world, rank)
    wl = synth.make_workload(args.workload, seed=args.seed, replica_offset=off, n_replicas=args.replicas)
    if args.batch:
        wl.batch = args.batch
    wl.settings.flags |= (8 if args.push_pull else 0) | (4 if args.greedy else 0)
    st = wl.settings
    net = Network(st, wl.peers, wl.batch, device=dev)
    net.bind_requests(wl.requests, scores=False)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    reduce_max, reduce_sum_vec = max_over_ranks, sum_counters

    W, K = args.warmup, args.steps
    s = 0
    for _ in range(W):
        f, c, now, g = step_args(wl, s, W)
        net.step(f, c, now, g or s == 0); s += 1        # a gossip round in the warm-up whatever the phase
    stats0 = net.stats()[-1].copy()
    launches0 = net.kernel_launches()

    # ---- timed region A: device-resident inputs --------------------------------------------
    sampler = ClockSampler(local) if rank == 0 else None
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler:
        sampler.start()
        time.sleep(0.5)                                # nvidia-smi needs a moment before its first sample
    barrier()
    ev0.record()
    for _ in range(K):
        net.step(*step_args(wl, s, W)); s += 1
    ev1.record()
    barrier()
    ms = reduce_max(ev0.elapsed_time(ev1))
    launches = net.kernel_launches() - launches0
    stats1 = net.stats()[-1].copy()
    delta = {k: int(b) - int(a) for k, a, b in zip(STAT_NAMES, stats0, stats1)}
    total_requests = int(reduce_sum_vec(np.array([delta["n_requests"]], np.uint64))[0])
    value = total_requests / (ms * 1e-3)

    # a second, identical timed region: reported beside the first one so that a disturbed run shows
    barrier()
    ev0.record()
    for _ in range(K):
        net.step(*step_args(wl, s, W)); s += 1
    ev1.record()
    barrier()
    ms_repeat = reduce_max(ev0.elapsed_time(ev1))

    # ---- region B: same K steps with per-kernel events (roofline of the dominant kernel) ---
    net.profile(True)
    stats_b0 = net.stats()[-1].copy()
    for _ in range(K):
        net.step(*step_args(wl, s, W)); s += 1
    prof = net.profile_read()
    net.profile(False)
    clocks = sampler.stop() if sampler else None     # sampled over region A and its instrumented repeat
    stats_b1 = net.stats()[-1].copy()
    delta_b = {k: int(b) - int(a) for k, a, b in zip(STAT_NAMES, stats_b0, stats_b1)}
    peak, peak_kind = measured_peaks()
    g_bytes, req_bytes = algorithmic_bytes(wl, delta_b)
    total_ms = sum(v[0] for v in prof.values())
    dom = max(prof, key=lambda k: prof[k][0])
    kernels = {k: {"ms_per_launch": v[0] / v[1], "launches": v[1], "share": v[0] / total_ms} for k, v in prof.items()}

    def roof(kernel, bytes_per_launch):
        if kernel not in prof:
            return None
        t = prof[kernel][0] / prof[kernel][1] * 1e-3
        ach = bytes_per_launch / t / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_source": peak_kind, "traffic": None, "bytes_per_launch": bytes_per_launch,
                "ms_per_launch": t * 1e3}

    roof_merge = roof("k_gossip_merge", g_bytes)
    if roof_merge and (st.n_peers, st.fanout_k, st.flags) == tuple(NCU_MERGE_TRAFFIC[k] for k in ("n_peers", "fanout_k", "flags")):
        roof_merge["traffic"] = NCU_MERGE_TRAFFIC["bytes_per_replica"] * Rp
    if roof_merge:      # context: bytes a merge without L2 reuse would move (k+1 rows read, one written)
        roof_merge["bytes_per_launch_without_reuse"] = (st.fanout_k + 2) * 8 * st.n_peers ** 2 * st.n_replicas
    roof_req = roof("k_step_fused", req_bytes / max(1, prof.get("k_step_fused", (0, 1))[1]))
    roofline = roof_merge if dom == "k_gossip_merge" else roof_req
    # the whole timed region A against HBM: algorithmic bytes of its gossip rounds and requests over its duration
    g_a, req_a = algorithmic_bytes(wl, delta)
    rounds_a = delta["rounds"] // Rp
    step_bytes = g_a * rounds_a + req_a
    whole = {"bound": "hbm", "achieved": step_bytes / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
             "frac": step_bytes / (ms * 1e-3) / 1e9 / peak, "bytes_per_step": step_bytes / K,
             "what": "all kernels of the K timed steps (gossip at its cadence + dispatch + duel + settle), algorithmic bytes"}
    # requests/s of dispatch+duel+settle alone (advance, fused step, fold, block commit), from the same events
    t_req = sum(prof[k][0] for k in ("k_advance", "k_step_fused", "k_fold", "k_fifo") if k in prof)
    req_only = {"value": delta_b["n_requests"] / (t_req * 1e-3), "unit": UNIT, "ms_per_step": t_req / K,
                "kernels": "k_advance + k_step_fused + k_fold (block commit included), summed CUDA-event time"}

    # ---- region S: the same K steps through the six separate calls ------------------------------
    for _ in range(min(W, 3)):                 # first use of the separate kernels loads their code: keep that untimed
        net.run_step(*step_args(wl, s, W)); s += 1
    while (s - W) % wl.gossip_every:
        net.step(*step_args(wl, s, W)); s += 1
    stats_s0 = net.stats()[-1].copy()
    barrier()
    ev0.record()
    for _ in range(K):
        net.run_step(*step_args(wl, s, W)); s += 1
    ev1.record()
    barrier()
    ms_six = reduce_max(ev0.elapsed_time(ev1))
    req_six = int(reduce_sum_vec(np.array([int(net.stats()[-1][0]) - int(stats_s0[0])], np.uint64))[0])
    six = {"value": req_six / (ms_six * 1e-3), "unit": UNIT, "ms_per_step": ms_six / K,
           "entry": "wwws_advance_time, wwws_gossip_round, wwws_dispatch_batch, wwws_duel_judge, wwws_settle_credits"}

    # ---- region C: end to end through host buffers ---------------------------------------------
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    Q = wl.n_requests
    io = {"origin": pin(wl.requests["origin"].view(np.int32)), "len_in": pin(wl.requests["len_in"].view(np.int16)),
          "len_out": pin(wl.requests["len_out"].view(np.int16)),
          "exec_a": torch.empty((Rp, Q), dtype=torch.int32).pin_memory(),
          "exec_b": torch.empty((Rp, Q), dtype=torch.int32).pin_memory(),
          "judges": torch.empty((Rp, Q, 4), dtype=torch.int32).pin_memory(),
          "outcome": torch.empty((Rp, Q), dtype=torch.uint8).pin_memory(),
          "flags": torch.empty((Rp, Q), dtype=torch.uint8).pin_memory()}
    for _ in range(min(W, 3)):
        net.step_host(io, *step_args(wl, s, W)); s += 1
    while (s - W) % wl.gossip_every:           # start the timed steps on a gossip step, as region A did
        net.step_host(io, *step_args(wl, s, W)); s += 1
    stats_c0 = net.stats()[-1].copy()
    barrier()
    ev0.record()
    for _ in range(K):
        tot = net.step_host(io, *step_args(wl, s, W)); s += 1
    ev1.record()
    barrier()
    ms_e2e = reduce_max(ev0.elapsed_time(ev1))
    req_e2e = int(reduce_sum_vec(np.array([int(tot[0]) - int(stats_c0[0])], np.uint64))[0])
    h2d = Rp * wl.batch * 8
    d2h = Rp * wl.batch * 26 + 8 * len(STAT_NAMES)

    line = None
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "ms_per_step_repeat": ms_repeat / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u64 views, i64 ledgers, fp32 scores", "data": "synthetic",
            "config": {"workload": args.workload, "n_peers": st.n_peers, "n_replicas_per_gpu": Rp,
                       "requests_per_step_per_gpu": Rp * wl.batch, "batch_overridden": bool(args.batch), "flags": st.flags, "gossip_every": wl.gossip_every, "gossip_phase": "first timed step",
                       "fanout_k": st.fanout_k, "entry": "wwws_step (fused dispatch+duel+settle)",
                       "l2": ("inputs larger than L2 (view buffers %.1f GB per GPU)" % (2 * 8 * st.n_peers ** 2 * Rp / 1e9)
                              if 2 * 8 * st.n_peers ** 2 * Rp > 126e6 else
                              "inputs smaller than L2 and not flushed: this workload is a launch-latency case, not a bandwidth one")},
            "clocks": clocks,
            "e2e": {"value": req_e2e / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / K, "entry": "wwws_step_host, pinned host buffers (mapped: the kernels read requests from and write results to them)"},
            "gpu_launches": launches,
            "roofline": roofline,
            "roofline_request_path": roof_req,
            "dispatch_duel_settle_only": req_only,
            "six_separate_calls": six,
            "whole_step_roofline": whole,
            "roofline_gossip_merge": roof_merge,
            "kernels": kernels,
            "step_mix": {k: delta[k] for k in ("n_requests", "n_delegated", "n_duel", "n_probes", "rounds")},
        }
    net.close()
    if world > 1:
        dist.destroy_process_group()
    return line


def oracle_run(workload, seed, steps, warmup, replicas=1, first_replica=0):
    """Time the CPU oracle, as it stands, on `replicas` replicas of the workload: `warmup`
    untimed steps, then `steps` timed ones.  Returns (requests/s, seconds, description)."""
    from oracle import Oracle
    from paper_2603_20661_b200 import synth
    wl = synth.slice_replicas(synth.make_workload(workload, seed=seed), first_replica, first_replica + replicas)
    o = Oracle(wl.settings, wl.peers)
    o.bind_requests(wl.requests)
    s = 0
    for _ in range(warmup):
        f, c, now, g = step_args(wl, s, warmup); o.run_step(f, c, now, g); s += 1
    n0 = o.stats_dict()["n_requests"]
    t0 = time.perf_counter()
    for _ in range(steps):
        f, c, now, g = step_args(wl, s, warmup); o.run_step(f, c, now, g); s += 1
    dt = time.perf_counter() - t0
    n = o.stats_dict()["n_requests"] - n0
    rounds = sum(1 for k in range(steps) if k % wl.gossip_every == 0)
    desc = (f"{replicas} replica(s) of {workload}, {steps} steps of {wl.batch} requests with {rounds} gossip round(s), "
            f"single thread")
    o.close()
    return n / dt, dt, desc


def _oracle_worker(job):
    workload, seed, steps, replica = job
    v, dt, _ = oracle_run(workload, seed, steps, 0, 1, replica)
    return v * dt, dt


def oracle_all_cores(workload, seed, steps):
    """One independent oracle instance per host core, each on its own replica (replicas share
    nothing); processes are started with `spawn`.  Returns (requests/s, workers, seconds)."""
    import multiprocessing as mp
    from paper_2603_20661_b200 import synth
    wl = synth.make_workload(workload, seed=seed, n_requests=1)
    view_bytes = 2 * 8 * wl.settings.n_peers ** 2 + (64 << 20)
    try:
        import psutil
        fit = max(1, int(psutil.virtual_memory().available * 0.6 // view_bytes))
    except ImportError:
        fit = 4
    workers = max(1, min(os.cpu_count() or 1, wl.settings.n_replicas, fit))
    t0 = time.perf_counter()
    with mp.get_context("spawn").Pool(workers) as pool:
        out = pool.map_async(_oracle_worker, [(workload, seed, steps, r) for r in range(workers)]).get(timeout=240)
    wall = time.perf_counter() - t0
    return sum(n for n, _ in out) / max(dt for _, dt in out), workers, wall


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores (1 thread), bounded sample."""
    if int(os.environ.get("RANK", "0")) != 0:
        return None
    from paper_2603_20661_b200 import synth
    wl = synth.make_workload(args.workload, seed=args.seed, n_replicas=1, n_requests=1000)
    K, W = args.steps, args.warmup
    # keep the whole run to a few minutes: the oracle's gossip round costs O(k N^2) on one core
    big = wl.settings.n_peers >= 8192
    W_eff = min(W, wl.gossip_every) if big else W
    K_eff = min(K, 2 * wl.gossip_every) if big else K
    v, dt, desc = oracle_run(args.workload, args.seed, K_eff, W_eff, 1)
    cb = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc}
    return {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": K_eff,
            "warmup": W_eff, "ms_per_step": dt / K_eff * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u64 views, i64 ledgers, fp32 scores", "data": "synthetic",
            "config": {"workload": args.workload, "sample": desc}, "cpu_baseline": cb,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--replicas", type=int, default=None, help="override the workload's replica count (profiling)")
    ap.add_argument("--push-pull", action="store_true", help="gossip as a full pairwise exchange (flag 8)")
    ap.add_argument("--greedy", action="store_true", help="greedy dispatch rule instead of the proportional draw (flag 4)")
    ap.add_argument("--batch", type=int, default=None, help="override requests per replica per step (saturation runs)")
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing legs")
    ap.add_argument("--no-cpu-all-cores", action="store_true", help="skip the one-oracle-per-core timing leg")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        line = run_reference(args)
        if line:
            print(json.dumps(line))
        return
    line = run_gpu(args)
    if line is not None:
        if args.gpus == 1 and not args.no_cpu_baseline:
            from paper_2603_20661_b200 import synth
            ge = synth.make_workload(args.workload, n_replicas=1, n_requests=1000).gossip_every
            v, dt, desc = oracle_run(args.workload, args.seed, ge, 0, 1)
            if not args.no_cpu_all_cores:
                try:
                    va, workers, wall = oracle_all_cores(args.workload, args.seed, ge)
                    line["cpu_baseline_all_cores"] = {
                        "value": va, "unit": UNIT, "cores": workers, "kind": "oracle", "wall_seconds": wall,
                        "sample": f"{workers} independent oracle instances, one replica each, same steps"}
                except Exception as e:          # a baseline leg must never cost the GPU result
                    line["cpu_baseline_all_cores"] = {"unavailable": repr(e)}
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
                                    "seconds": dt}
        print(json.dumps(line))


if __name__ == "__main__":
    main()
