#!/usr/bin/env python
"""Benchmark of the batched WWW.Serve network step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole path over one batch: advance -> gossip (on the steps its
cadence selects) -> dispatch -> duel-and-judge -> settle.  Metric: simulated requests
dispatched and settled per second.  One JSON line is printed by rank 0.

Multi-GPU: replicas are independent, so every rank runs its own set of replicas (weak
scaling, no data-path collective; only counters and the max-over-ranks time are reduced).
`--gpus N` with N > 1 starts N ranks itself (one process per GPU through torch.distributed.run)
unless it already runs under such a launcher (WORLD_SIZE set).
`--impl reference` times the CPU oracle, as it stands, on a bounded sample of the workload.
"""
from __future__ import annotations

import argparse
import glob
import hashlib
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
EXTRA_LEGS = ("zipf1k", "churn4k")           # also timed, compactly, by the default run
TARGET_FRAC = 0.6                            # the stated goal for dispatch+settle: 60 % of HBM bandwidth
N_SM, ISSUE_PER_SM = 148, 4                  # warp instructions an SM can issue per cycle: one per scheduler


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def read_counter_files():
    """Counters taken from ncu captures: `profiles/*_counters.txt`, one capture per file, `key: value`
    lines (kernel, workload, commit, source file and its sha256 at the time of the capture, figures)."""
    out = []
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*_counters.txt"))):
        rec = {"file": os.path.relpath(path, ROOT)}
        with open(path) as f:
            for ln in f:
                if ln.startswith("#") or ":" not in ln:
                    continue
                k, v = ln.split(":", 1)
                rec[k.strip()] = v.strip()
        out.append(rec)
    return out


def source_unchanged(rec):
    """True if the kernel's source file still has the digest recorded with the capture."""
    src = rec.get("source")
    if not src or "source_sha256" not in rec:
        return False
    try:
        with open(os.path.join(ROOT, src), "rb") as f:
            return hashlib.sha256(f.read()).hexdigest() == rec["source_sha256"]
    except OSError:
        return False


def find_counters(kernel, **match):
    """The capture of `kernel` whose keys equal `match`; `workload` also matches a name listed in the
    capture's `applies_to` (the same kernel at the same launch size on a network small enough to profile)."""
    for rec in read_counter_files():
        if rec.get("kernel") != kernel:
            continue
        ok = True
        for k, v in match.items():
            if k == "workload" and str(v) in rec.get("applies_to", "").replace(",", " ").split():
                continue
            ok = ok and str(rec.get(k)) == str(v)
        if ok:
            return rec
    return None


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
        time.sleep(0.5)                                # nvidia-smi needs a moment before its first sample
        return self

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
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm), "reasons": sorted(reasons)}


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
    """Bytes the method must move.
    Gossip round: 2 * 8 * N^2 per replica (every view entry read once and written once; the k+1
    readers of a row share it through L2 because the merge walks the matrix by column panels).
    Request path: 8 B record + 26 B result, plus a 256 B view window per request that offloads."""
    st = wl.settings
    gossip_round = 2 * 8 * st.n_peers ** 2 * st.n_replicas
    offloaded = stats_delta["n_delegated"] + stats_delta["n_fallback_local"] + stats_delta["n_failed"]
    req = stats_delta["n_requests"] * (8 + 26) + offloaded * 256
    return gossip_round, req


REQUEST_KERNELS = ("k_advance", "k_step_fused", "k_fold", "k_fifo")


class Leg:
    """One workload on this rank's GPU: the network, its step counter and the timed regions."""

    def __init__(self, args, name, dev, world, rank, batch=None, warmup=None):
        import torch
        from paper_2603_20661_b200 import synth
        from paper_2603_20661_b200.binding import Network
        from paper_2603_20661_b200.sharding import replica_shard
        self.torch, self.dev, self.world, self.rank, self.name = torch, dev, world, rank, name
        wl0 = synth.make_workload(name, seed=args.seed, n_replicas=args.replicas)
        self.Rp = wl0.settings.n_replicas
        # weak scaling: every rank runs the configuration's full replica count, on its own replica indices
        off, _ = replica_shard(world * self.Rp, world, rank)
        self.wl = synth.make_workload(name, seed=args.seed, replica_offset=off, n_replicas=args.replicas)
        if batch:
            self.wl.batch = batch
        self.wl.settings.flags |= (8 if args.push_pull else 0) | (4 if args.greedy else 0)
        self.net = Network(self.wl.settings, self.wl.peers, self.wl.batch, device=dev)
        self.net.bind_requests(self.wl.requests, scores=False)
        if args.step_kernel:
            self.net.set_option(1, args.step_kernel)
        if args.stream_run:
            self.net.set_option(2, args.stream_run)
        if args.host_io:
            self.net.set_option(4, args.host_io)
        if args.overlap is not None:
            self.net.set_option(3, args.overlap)
        self.W, self.s = (args.warmup if warmup is None else warmup), 0
        for _ in range(self.W):
            f, c, now, g = step_args(self.wl, self.s, self.W)
            self.net.step(f, c, now, g or self.s == 0); self.s += 1     # a gossip round in the warm-up whatever the phase
        self.align()

    def close(self):
        self.net.close()
        self.net = None
        self.torch.cuda.empty_cache()

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize(self.dev)

    def totals(self):
        from paper_2603_20661_b200.binding import STAT_NAMES
        return dict(zip(STAT_NAMES, (int(v) for v in self.net.stats()[-1])))

    def align(self, call=None):
        """Run untimed steps until the next step is a gossip step, as the first timed region starts."""
        call = call or self.net.step
        while (self.s - self.W) % self.wl.gossip_every:
            call(*step_args(self.wl, self.s, self.W)); self.s += 1

    def timed(self, K, call=None, repeats=1):
        """`repeats` back-to-back regions of K steps, each bracketed by CUDA events on the launching
        stream, barrier + synchronize on both sides of the whole; returns the per-region times (ms,
        max over ranks) and the counter deltas of all regions together."""
        from paper_2603_20661_b200.sharding import max_over_ranks
        torch = self.torch
        call = call or self.net.step
        before = self.totals()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(repeats + 1)]
        self.barrier()
        ev[0].record()
        for i in range(repeats):
            for _ in range(K):
                call(*step_args(self.wl, self.s, self.W)); self.s += 1
            ev[i + 1].record()
        self.barrier()
        ms = [max_over_ranks(ev[i].elapsed_time(ev[i + 1])) for i in range(repeats)]
        after = self.totals()
        return ms, {k: after[k] - before[k] for k in after}

    def profiled(self, K):
        """K steps with per-kernel events: {kernel: (summed ms, launches)} and the counter deltas."""
        before = self.totals()
        self.net.profile(True)
        for _ in range(K):
            self.net.step(*step_args(self.wl, self.s, self.W)); self.s += 1
        prof = self.net.profile_read()
        self.net.profile(False)
        after = self.totals()
        return prof, {k: after[k] - before[k] for k in after}


def rooflines(leg, prof, delta_b, sm_mhz, counters_workload=None):
    """HBM roofline of the gossip merge and of the request kernel, and the issue-slot roofline of
    the request kernel (warp instructions per request from the ncu capture on record)."""
    st, wl = leg.wl.settings, leg.wl
    peak, peak_kind = measured_peaks()
    g_bytes, req_bytes = algorithmic_bytes(wl, delta_b)

    def roof(kernel, bytes_per_launch):
        if kernel not in prof:
            return None
        t = prof[kernel][0] / prof[kernel][1] * 1e-3
        ach = bytes_per_launch / t / 1e9
        return {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                "peak_source": peak_kind, "traffic": None, "bytes_per_launch": bytes_per_launch, "ms_per_launch": t * 1e3}

    merge = roof("k_gossip_merge", g_bytes)
    if merge:
        rec = find_counters("k_gossip_merge", n_peers=st.n_peers, fanout_k=st.fanout_k, flags=st.flags & ~4)
        if rec and source_unchanged(rec):      # DRAM bytes of one replica's pass; a launch is Rp such passes back to back
            merge["traffic"] = float(rec["dram_bytes_per_replica_round"]) * leg.Rp
            merge["traffic_from_profile"] = rec["file"]
        elif rec:
            merge["traffic_from_profile"] = rec["file"] + " (kernel source changed since: traffic withheld)"
        merge["bytes_per_launch_without_reuse"] = (st.fanout_k + 2) * 8 * st.n_peers ** 2 * st.n_replicas
    launches = max(1, prof.get("k_step_fused", (0, 1))[1])
    req = roof("k_step_fused", req_bytes / launches)
    if req:
        req["target_frac"] = TARGET_FRAC
        req["target_met"] = bool(req["frac"] >= TARGET_FRAC)
        per_launch = delta_b["n_requests"] / launches
        rate = per_launch / (req["ms_per_launch"] * 1e-3)
        req["requests_per_launch"] = per_launch
        req["requests_per_s"] = rate
        rec = find_counters("k_step_fused", workload=counters_workload or leg.name)
        if rec and sm_mhz:
            ipr = float(rec["warp_instructions_per_request"])
            req["issue"] = {"bound": "alu", "warp_instr_per_request": ipr,
                            "active_lanes": float(rec.get("active_lanes_per_instruction", "nan")),
                            "issue_frac": ipr * rate / (N_SM * ISSUE_PER_SM * sm_mhz * 1e6),
                            "peak": "148 SMs x 4 warp instructions per cycle x the SM clock sampled in this run",
                            "sm_mhz": sm_mhz, "source": rec["file"],
                            "source_current": source_unchanged(rec), "commit": rec.get("commit")}
    t_req = sum(prof[k][0] for k in REQUEST_KERNELS if k in prof)
    return merge, req, t_req


def run_compact_leg(args, name, dev, world, rank, sampler_index):
    """A secondary workload: value, time per step and the rooflines of its two main kernels."""
    leg = Leg(args, name, dev, world, rank)
    K = args.steps
    sampler = ClockSampler(sampler_index).start() if rank == 0 else None
    ms, delta = leg.timed(K)
    leg.align()
    prof, delta_b = leg.profiled(K)
    clocks = sampler.stop() if sampler else {"sm_mhz": None}
    merge, req, t_req = rooflines(leg, prof, delta_b, clocks.get("sm_mhz"))
    from paper_2603_20661_b200.sharding import sum_counters
    total = int(sum_counters(np.array([delta["n_requests"]], np.uint64))[0])
    out = {"workload": name, "value": total / (ms[0] * 1e-3), "unit": UNIT, "ms_per_step": ms[0] / K,
           "requests_per_step_per_gpu": leg.Rp * leg.wl.batch,
           "gossip_merge": {k: merge[k] for k in ("frac", "ms_per_launch", "achieved")} if merge else None,
           "request_path": ({"frac": req["frac"], "ms_per_launch": req["ms_per_launch"], "requests_per_s": req["requests_per_s"],
                             "issue_frac": req.get("issue", {}).get("issue_frac"),
                             "warp_instr_per_request": req.get("issue", {}).get("warp_instr_per_request")} if req else None),
           "dispatch_duel_settle_only_ms_per_step": t_req / K, "sm_mhz": clocks.get("sm_mhz")}
    g_a, req_a = algorithmic_bytes(leg.wl, delta)
    out["whole_step_hbm_frac"] = (g_a * (delta["rounds"] // leg.Rp) + req_a) / (ms[0] * 1e-3) / 1e9 / measured_peaks()[0]
    leg.close()
    return out


SATURATED_BATCH = {"adversarial16k": 100000, "churn4k": 50000, "zipf1k": 10000}


def run_saturated_leg(args, name, dev, world, rank, sampler_index):
    """The request kernel alone on launches large enough to fill the GPU (the workload's whole request
    stream of every replica in one step), on a fresh network so that the request mix is the workload's
    own: the configurations' step sizes leave the kernel latency-bound, this is its throughput."""
    leg = Leg(args, name, dev, world, rank, batch=SATURATED_BATCH[name], warmup=3)
    sampler = ClockSampler(sampler_index).start() if rank == 0 else None
    prof, delta_b = leg.profiled(3)
    clocks = sampler.stop() if sampler else {"sm_mhz": None}
    _, req, _ = rooflines(leg, prof, delta_b, clocks.get("sm_mhz"), counters_workload=name + "_saturated")
    leg.close()
    if req:
        req["workload"] = name
        req["batch_per_replica"] = SATURATED_BATCH[name]
        req["offloaded_fraction"] = (delta_b["n_delegated"] + delta_b["n_fallback_local"] + delta_b["n_failed"]) / max(1, delta_b["n_requests"])
    return req


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2603_20661_b200.binding import STAT_NAMES
    from paper_2603_20661_b200.sharding import sum_counters

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE is {world}")
    if torch.cuda.device_count() <= local:
        raise SystemExit(f"bench.py: rank {rank} needs cuda:{local} but only {torch.cuda.device_count()} device(s) are visible")
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    leg = Leg(args, args.workload, dev, world, rank, batch=args.batch)
    wl, st, Rp, net = leg.wl, leg.wl.settings, leg.Rp, leg.net
    K, W = args.steps, args.warmup
    launches0 = net.kernel_launches()

    # ---- region A: exactly K steps, device-resident inputs: the headline value --------------------
    sampler = ClockSampler(local).start() if rank == 0 else None
    ms_a, delta = leg.timed(K)
    ms = ms_a[0]
    launches = net.kernel_launches() - launches0
    total_requests = int(sum_counters(np.array([delta["n_requests"]], np.uint64))[0])
    value = total_requests / (ms * 1e-3)
    clocks = sampler.stop() if sampler else None

    # ---- sustained: the same region repeated back to back for about a second of device time (each
    # repeat a whole number of gossip periods, so that all repeats hold the same work)
    sustained, clocks_sustained = None, None
    if args.sustain_s > 0:
        leg.align()
        k_rep = K if K % wl.gossip_every == 0 else K * wl.gossip_every
        reps = int(min(400, max(3, np.ceil(args.sustain_s * 1e3 / max(ms * k_rep / K, 1e-3)))))
        sampler = ClockSampler(local).start() if rank == 0 else None
        ms_rep, _ = leg.timed(k_rep, repeats=reps)
        clocks_sustained = sampler.stop() if sampler else None
        per_step = [m / k_rep for m in ms_rep]
        sustained = {"repeats": len(ms_rep), "steps_per_repeat": k_rep, "device_seconds": sum(ms_rep) * 1e-3,
                     "ms_per_step_median": statistics.median(per_step), "ms_per_step_min": min(per_step),
                     "ms_per_step_max": max(per_step),
                     "value_at_median": Rp * wl.batch * world / (statistics.median(per_step) * 1e-3),
                     "clocks": clocks_sustained}

    # ---- region B: K steps with per-kernel events (rooflines of the dominant kernel and of the request path)
    leg.align()
    sampler = ClockSampler(local).start() if rank == 0 else None
    prof, delta_b = leg.profiled(K)
    clocks_profiled = sampler.stop() if sampler else None
    peak, peak_kind = measured_peaks()
    total_ms = sum(v[0] for v in prof.values())
    dom = max(prof, key=lambda k: prof[k][0])
    kernels = {k: {"ms_per_launch": v[0] / v[1], "launches": v[1], "share": v[0] / total_ms} for k, v in prof.items()}
    sm_mhz = (clocks_profiled or {}).get("sm_mhz") or (clocks or {}).get("sm_mhz")     # the clock while these kernels were timed
    roof_merge, roof_req, t_req = rooflines(leg, prof, delta_b, sm_mhz)
    roofline = roof_merge if dom == "k_gossip_merge" else roof_req
    # the whole timed region A against HBM: algorithmic bytes of its gossip rounds and requests over its duration
    g_a, req_a = algorithmic_bytes(wl, delta)
    step_bytes = g_a * (delta["rounds"] // Rp) + req_a
    whole = {"bound": "hbm", "achieved": step_bytes / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
             "frac": step_bytes / (ms * 1e-3) / 1e9 / peak, "bytes_per_step": step_bytes / K,
             "what": "all kernels of the K timed steps (gossip at its cadence + dispatch + duel + settle), algorithmic bytes"}
    req_only = {"value": delta_b["n_requests"] / (t_req * 1e-3), "unit": UNIT, "ms_per_step": t_req / K,
                "kernels": "k_advance + k_step_fused + k_fold (block commit included), summed CUDA-event time"}

    # ---- region S: the same K steps through the six separate calls ------------------------------
    for _ in range(3):                         # first use of the separate kernels loads their code: keep that untimed
        net.run_step(*step_args(wl, leg.s, W)); leg.s += 1
    leg.align()
    ms_six, d_six = leg.timed(K, call=net.run_step)
    req_six = int(sum_counters(np.array([d_six["n_requests"]], np.uint64))[0])
    six = {"value": req_six / (ms_six[0] * 1e-3), "unit": UNIT, "ms_per_step": ms_six[0] / K,
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
    host_step = lambda *a: net.step_host(io, *a)
    for _ in range(3):
        host_step(*step_args(wl, leg.s, W)); leg.s += 1
    leg.align(host_step)
    ms_e2e, d_e2e = leg.timed(K, call=host_step)
    req_e2e = int(sum_counters(np.array([d_e2e["n_requests"]], np.uint64))[0])
    h2d = Rp * wl.batch * 8
    d2h = Rp * wl.batch * 26 + 8 * len(STAT_NAMES)

    line = None
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u64 views, i64 ledgers, fp32 scores", "data": "synthetic",
            "config": {"workload": args.workload, "n_peers": st.n_peers, "n_replicas_per_gpu": Rp,
                       "requests_per_step_per_gpu": Rp * wl.batch, "batch_overridden": bool(args.batch), "flags": st.flags, "gossip_every": wl.gossip_every, "gossip_phase": "first timed step",
                       "fanout_k": st.fanout_k, "entry": "wwws_step (fused dispatch+duel+settle)",
                       "l2": ("inputs larger than L2 (view buffers %.1f GB per GPU)" % (2 * 8 * st.n_peers ** 2 * Rp / 1e9)
                              if 2 * 8 * st.n_peers ** 2 * Rp > 126e6 else
                              "inputs smaller than L2 and not flushed: this workload is a launch-latency case, not a bandwidth one")},
            "clocks": clocks,
            "sustained": sustained,
            "e2e": {"value": req_e2e / (ms_e2e[0] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e[0] / K, "entry": "wwws_step_host, pinned host buffers"},
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
    leg.close()
    del io
    # ---- the other large configurations, compactly (default run only) ---------------------------
    if args.legs and args.workload == DEFAULT_WORKLOAD and not args.batch:
        legs = [run_compact_leg(args, name, dev, world, rank, local) for name in EXTRA_LEGS]
        sat = run_saturated_leg(args, args.workload, dev, world, rank, local)
        if line is not None:
            line["other_workloads"] = legs
            line["roofline_request_path_saturated"] = sat
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
        f, c, now, g = step_args(wl, s, warmup); o.run_step(f, c, now, g or s == 0); s += 1
    n0 = o.stats_dict()["n_requests"]
    t0 = time.perf_counter()
    for _ in range(steps):
        f, c, now, g = step_args(wl, s, warmup); o.run_step(f, c, now, g); s += 1
    dt = time.perf_counter() - t0
    n = o.stats_dict()["n_requests"] - n0
    rounds = sum(1 for k in range(steps) if k % wl.gossip_every == 0)
    desc = (f"{replicas} replica(s) of {workload}, {warmup} untimed step(s), then {steps} steps of {wl.batch} requests "
            f"per replica with {rounds} gossip round(s), single thread")
    o.close()
    return n / dt, dt, desc


def _oracle_worker(job):
    workload, seed, steps, replica = job
    v, dt, _ = oracle_run(workload, seed, steps, 1, 1, replica)
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


def launcher_command(argv, n, port=None):
    """The command that starts `n` ranks of this script on this node, one per GPU."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port or 29500 + os.getpid() % 2000), os.path.abspath(__file__)]
    return cmd + list(argv)


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
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
    ap.add_argument("--step-kernel", type=int, default=0, help="force the fused step's kernel (WWWS_OPT_STEP_KERNEL)")
    ap.add_argument("--stream-run", type=int, default=0, help="requests per warp of the streaming kernel (WWWS_OPT_STREAM_RUN)")
    ap.add_argument("--host-io", type=int, default=0, help="wwws_step_host path: 0 by batch size, 1 mapped direct, 2 staged (WWWS_OPT_HOST_IO)")
    ap.add_argument("--overlap", type=int, default=None, help="mask of launches that may overlap their predecessor (WWWS_OPT_LAUNCH_OVERLAP)")
    ap.add_argument("--sustain-s", type=float, default=1.0, help="device seconds of the repeated timed region (0 skips it)")
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--no-legs", dest="legs", action="store_false", help="skip the compact legs on the other large workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing legs")
    ap.add_argument("--no-cpu-all-cores", action="store_true", help="skip the one-oracle-per-core timing leg")
    args = ap.parse_args(argv)
    if args.warmup < 3:
        args.warmup = 3
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be >= 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher yet: start one rank per GPU and let rank 0 print the line
        if args.impl == "ours":
            import torch
            if torch.cuda.device_count() < args.gpus:
                raise SystemExit(f"bench.py: --gpus {args.gpus} but {torch.cuda.device_count()} CUDA device(s) are visible")
        raise SystemExit(subprocess.call(launcher_command(argv, args.gpus)))
    if args.impl == "reference":
        line = run_reference(args)
        if line:
            print(json.dumps(line))
        return
    line = run_gpu(args)
    if line is not None:
        if args.gpus == 1 and not args.no_cpu_baseline:
            from paper_2603_20661_b200 import synth
            wl = synth.make_workload(args.workload, n_requests=1000)
            # the large networks are timed on two replicas (the cost is linear in replicas), the others on one
            reps = 2 if wl.settings.n_replicas >= 2 and wl.settings.n_peers >= 2048 else 1
            ge = wl.gossip_every
            v, dt, desc = oracle_run(args.workload, args.seed, ge, 1, reps)
            if not args.no_cpu_all_cores:
                try:
                    va, workers, wall = oracle_all_cores(args.workload, args.seed, ge)
                    line["cpu_baseline_all_cores"] = {
                        "value": va, "unit": UNIT, "cores": workers, "kind": "oracle", "wall_seconds": wall,
                        "sample": f"{workers} independent oracle instances, one replica each, one untimed step, then the same steps"}
                except Exception as e:          # a baseline leg must never cost the GPU result
                    line["cpu_baseline_all_cores"] = {"unavailable": repr(e)}
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc,
                                    "seconds": dt}
        print(json.dumps(line))


if __name__ == "__main__":
    main()
