"""Seeded synthetic networks and request streams (inputs only).

This module builds the *inputs* of a simulated WWW.Serve network: per-peer
hidden parameters and policies, a request stream, and the scalar settings of a
run.  It contains none of the method's arithmetic (no scoring, sampling,
merging or settlement) and loads no native code, so both the CUDA path and the
independent CPU checker can be fed from it.

Shapes follow the paper's experiments where it gives them: a handful to
thousands of heterogeneous providers, Poisson arrivals with hot and idle
origins (Appendix "Experimental Settings", Table of request schedules), the
standard policy constants (offload 80 %, accept 80 %, target utilisation 70 %)
and duel rates of 5-25 % (Section "Overhead of Duel-and-Judge Mechanism").
The prompts of the paper's runs come from a public dataset; only their length
distribution matters to the simulation, and lengths are drawn here from a
lognormal law instead.

Everything is generated with ``numpy.random.Generator(PCG64(seed))``.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional

import numpy as np

WINDOW = 32  # candidate-window width (peers per block of the id ring)


@dataclasses.dataclass
class Settings:
    """Scalar settings of one network; mirrors the C-ABI configuration record."""
    n_peers: int
    n_replicas: int
    replica_offset: int = 0
    seed: int = 0
    fanout_k: int = 2
    gossip_tries: int = 8
    max_probes: int = 6
    n_judges: int = 3
    p_duel_ppm: int = 50_000
    p_noise_ppm: int = 0
    p_leave_ppm: int = 0
    p_join_ppm: int = 0
    p_prio_active_ppm: int = 500_000
    prio_window_ms: int = 60_000
    util_window_ms: int = 10_000
    cap_ref_tok_s: int = 2000
    slo_num: int = 2
    slo_den: int = 1
    hop_ms: int = 0
    init_stale_max: int = 0
    flags: int = 3            # bit0 reputation factor, bit1 load factor
    reward_R: int = 100
    reward_add: int = 40
    penalty_P: int = 70
    rank_cdf: Optional[np.ndarray] = None   # uint32 thresholds, None = uniform


@dataclasses.dataclass
class Workload:
    """A complete seeded input set: settings, peers, requests, step structure."""
    name: str
    settings: Settings
    peers: Dict[str, np.ndarray]      # each [n_replicas, n_peers]
    requests: Dict[str, np.ndarray]   # each [n_replicas, n_requests]
    batch: int                        # requests per replica per step
    gossip_every: int                 # steps between gossip rounds
    finalize_every: int = 1           # steps between ledger finalizations

    @property
    def n_requests(self) -> int:
        return int(self.requests["origin"].shape[1])

    @property
    def n_steps(self) -> int:
        return (self.n_requests + self.batch - 1) // self.batch

    def step_now_ms(self, step: int) -> int:
        """Simulated time at which step `step` runs: arrival time of its last request."""
        last = min((step + 1) * self.batch, self.n_requests) - 1
        return int(self.requests["t_ms"][0, last])


PEER_FIELDS = {
    "cap_true_tok_s": np.uint32, "quality_fx": np.uint32, "credit0": np.int64,
    "stake_pm": np.uint16, "offload_util_pm": np.uint16, "accept_util_pm": np.uint16,
    "offload_ppm": np.uint32, "accept_ppm": np.uint32,
    "misreport_mul": np.uint8, "prio_flag": np.uint8, "online0": np.uint8,
}
REQUEST_FIELDS = {"origin": np.uint32, "t_ms": np.uint32, "len_in": np.uint16, "len_out": np.uint16}


def _quality_to_fx(q: np.ndarray) -> np.ndarray:
    return np.minimum(np.floor(q * 4294967296.0), 4294967295.0).astype(np.uint32)


def default_peers(rng: np.random.Generator, n_replicas: int, n_peers: int, *,
                  capacity: str = "lognormal", offload_util_pm: int = 700,
                  prio_prob: float = 0.0, adversary_frac: float = 0.0) -> Dict[str, np.ndarray]:
    shape = (n_replicas, n_peers)
    if capacity == "lognormal":
        cap = np.exp(rng.normal(math.log(2000.0), 0.5, shape))
    elif capacity == "tiers":
        cap = 2000.0 * (2.0 ** rng.integers(0, 4, shape))
    else:
        raise ValueError(capacity)
    cap = np.clip(np.rint(cap), 1, 2 ** 31 - 1).astype(np.uint32)
    q = rng.random(shape)
    mis = np.ones(shape, np.uint8)
    if adversary_frac > 0:
        adv = rng.random(shape) < adversary_frac
        q = np.where(adv, rng.random(shape) * 0.3, q)
        mis = np.where(adv, 4, 1).astype(np.uint8)
    prio = (rng.random(shape) < prio_prob).astype(np.uint8) if prio_prob > 0 else np.zeros(shape, np.uint8)
    return {
        "cap_true_tok_s": cap,
        "quality_fx": _quality_to_fx(q),
        "credit0": np.full(shape, 10_000, np.int64),
        "stake_pm": np.full(shape, 1000, np.uint16),
        "offload_util_pm": np.full(shape, offload_util_pm, np.uint16),
        "accept_util_pm": np.full(shape, 700, np.uint16),
        "offload_ppm": np.full(shape, 800_000, np.uint32),
        "accept_ppm": np.full(shape, 800_000, np.uint32),
        "misreport_mul": mis,
        "prio_flag": prio,
        "online0": np.ones(shape, np.uint8),
    }


def _lengths(rng: np.random.Generator, shape, median: float) -> np.ndarray:
    x = np.exp(rng.normal(math.log(median), 0.8, shape))
    return np.clip(np.rint(x), 1, 8192).astype(np.uint16)


def poisson_times_ms(rng: np.random.Generator, n: int, rate_per_s: float) -> np.ndarray:
    gaps = rng.exponential(1.0 / rate_per_s, n)
    return np.minimum(np.floor(np.cumsum(gaps) * 1000.0), 2 ** 32 - 1).astype(np.uint32)


def mmpp_times_ms(rng: np.random.Generator, n: int, rates=(50.0, 500.0), sojourn_s: float = 10.0) -> np.ndarray:
    """Two-state Markov-modulated Poisson arrivals (bursty)."""
    out = np.empty(n, np.float64)
    t, state, i = 0.0, 0, 0
    t_switch = rng.exponential(sojourn_s)
    while i < n:
        gap = rng.exponential(1.0 / rates[state])
        if t + gap >= t_switch:
            t = t_switch
            state ^= 1
            t_switch = t + rng.exponential(sojourn_s)
            continue
        t += gap
        out[i] = t
        i += 1
    return np.minimum(np.floor(out * 1000.0), 2 ** 32 - 1).astype(np.uint32)


def default_requests(rng: np.random.Generator, n_replicas: int, n_peers: int, n_requests: int,
                     t_ms: np.ndarray, hot_prob: float = 0.25) -> Dict[str, np.ndarray]:
    """Origins: every peer is hot (4x arrival weight) with probability `hot_prob`."""
    origin = np.empty((n_replicas, n_requests), np.uint32)
    for r in range(n_replicas):
        w = np.where(rng.random(n_peers) < hot_prob, 4.0, 1.0)
        cdf = np.cumsum(w / w.sum())
        origin[r] = np.minimum(np.searchsorted(cdf, rng.random(n_requests), side="right"), n_peers - 1)
    shape = (n_replicas, n_requests)
    return {
        "origin": origin,
        "t_ms": np.ascontiguousarray(np.broadcast_to(t_ms.astype(np.uint32), shape)),
        "len_in": _lengths(rng, shape, 512.0),
        "len_out": _lengths(rng, shape, 256.0),
    }


def zipf_rank_cdf(n_ranks: int, s: float = 1.1) -> np.ndarray:
    p = 1.0 / np.arange(1, n_ranks + 1, dtype=np.float64) ** s
    c = np.cumsum(p / p.sum())
    return np.minimum(np.floor(c * 4294967296.0), 4294967295.0).astype(np.uint32)


CONFIG_NAMES = ("tiny", "tiers64", "zipf1k", "churn4k", "adversarial16k")


def make_workload(name: str, *, seed: int = 0, n_replicas: Optional[int] = None,
                  n_requests: Optional[int] = None, n_peers: Optional[int] = None,
                  replica_offset: int = 0) -> Workload:
    """One of the five seeded configurations; sizes can be overridden to get
    reduced cases of the same shape (fewer replicas / requests / peers)."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    if name == "tiny":
        N, Rp, Q = n_peers or 8, n_replicas or 1, n_requests or 1000
        st = Settings(N, Rp, fanout_k=2, p_duel_ppm=50_000)
        peers = default_peers(rng, Rp, N, offload_util_pm=700)
        t = poisson_times_ms(rng, Q, 20.0)
        wl = Workload(name, st, peers, default_requests(rng, Rp, N, Q, t), batch=50, gossip_every=1)
    elif name == "tiers64":
        N, Rp, Q = n_peers or 64, n_replicas or 1, n_requests or 100_000
        st = Settings(N, Rp, fanout_k=3, p_duel_ppm=100_000)
        peers = default_peers(rng, Rp, N, capacity="tiers", offload_util_pm=700, prio_prob=0.2)
        t = poisson_times_ms(rng, Q, 400.0 * N / 64)
        wl = Workload(name, st, peers, default_requests(rng, Rp, N, Q, t), batch=500, gossip_every=1)
    elif name == "zipf1k":
        N, Rp, Q = n_peers or 1024, n_replicas or 256, n_requests or 10_000
        st = Settings(N, Rp, fanout_k=4, p_duel_ppm=50_000,
                      rank_cdf=zipf_rank_cdf((N + WINDOW - 1) // WINDOW))
        peers = default_peers(rng, Rp, N, offload_util_pm=0)
        t = poisson_times_ms(rng, Q, 2.5 * N)
        wl = Workload(name, st, peers, default_requests(rng, Rp, N, Q, t), batch=500, gossip_every=2)
    elif name == "churn4k":
        N, Rp, Q = n_peers or 4096, n_replicas or 64, n_requests or 50_000
        st = Settings(N, Rp, fanout_k=4, p_duel_ppm=50_000, init_stale_max=5,
                      p_leave_ppm=60_000, p_join_ppm=60_000)
        peers = default_peers(rng, Rp, N, offload_util_pm=0)
        t = mmpp_times_ms(rng, Q)
        wl = Workload(name, st, peers, default_requests(rng, Rp, N, Q, t), batch=1000, gossip_every=5)
    elif name == "adversarial16k":
        N, Rp, Q = n_peers or 16_384, n_replicas or 16, n_requests or 100_000
        st = Settings(N, Rp, fanout_k=4, p_duel_ppm=200_000, p_noise_ppm=100_000)
        peers = default_peers(rng, Rp, N, offload_util_pm=0, adversary_frac=0.10)
        t = poisson_times_ms(rng, Q, 2.5 * N)
        wl = Workload(name, st, peers, default_requests(rng, Rp, N, Q, t), batch=1000, gossip_every=10)
    else:
        raise ValueError(f"unknown workload {name!r}; choose from {CONFIG_NAMES}")
    wl.settings.seed = seed
    wl.settings.replica_offset = replica_offset
    return wl


# Request schedules shaped like the paper's Table of experimental settings: per node
# (relative capacity, [(interval end in s, mean inter-arrival time in s), ...]) over 750 s.
# Only the schedule shapes are taken from the table; capacities are relative service rates
# chosen here (the table names models and GPUs, not token rates).
PAPER_SETTINGS = {
    "setting1": [(1.0, [(300, 5), (750, 20)]), (1.0, [(750, 20)]), (1.0, [(750, 20)]), (1.0, [(450, 20), (750, 5)])],
    "setting2": [(1.0, [(300, 4), (750, 20)]), (1.0, [(750, 20)]), (0.7, [(750, 30)]), (0.7, [(450, 30), (750, 6)])],
    "setting3": [(4.0, [(300, 2), (750, 6)]), (1.0, [(750, 15)]), (0.7, [(750, 30)]), (1.0, [(450, 15), (750, 5)])],
    "setting4": [(1.0, [(750, 9)]), (1.0, [(450, 6), (750, 12)]), (1.0, [(300, 6), (750, 12)]), (1.0, [(450, 12), (750, 6)]),
                 (0.8, [(750, 12)]), (0.8, [(450, 10), (750, 20)]), (0.7, [(300, 20), (750, 10)]), (0.7, [(300, 20), (750, 10)])],
}


def make_paper_setting(name: str, *, seed: int = 0, n_replicas: int = 64, offload: bool = True,
                       base_capacity: int = 1000, batch: int = 8) -> Workload:
    """A small network with piecewise-Poisson per-node arrivals (hot and idle phases that differ
    across nodes), long generations (median 6,000 output tokens, capped at 8,192 like the paper's
    runs) and the paper's standard policy; `offload=False` gives the single-node baseline in
    which every node serves only its own users.  All replicas share the arrival stream and differ
    in request lengths and in the protocol's random draws."""
    nodes = PAPER_SETTINGS[name]
    rng = np.random.default_rng(np.random.PCG64(seed))
    times, origins = [], []
    for node, (_, schedule) in enumerate(nodes):
        t, start = 0.0, 0.0
        for end, gap in schedule:
            t = max(t, start)
            while True:
                t += rng.exponential(gap)
                if t >= end:
                    break
                times.append(t); origins.append(node)
            start = end
    order = np.argsort(np.array(times), kind="stable")
    t_ms = np.floor(np.array(times)[order] * 1000.0).astype(np.uint32)
    origin = np.array(origins, np.uint32)[order]
    N, Q = len(nodes), len(order)
    shape = (n_replicas, N)
    st = Settings(N, n_replicas, seed=seed, fanout_k=2, p_duel_ppm=50_000, n_judges=2, cap_ref_tok_s=base_capacity,
                  flags=3 | 16)
    cap = np.array([int(round(c * base_capacity)) for c, _ in nodes], np.uint32)
    peers = default_peers(rng, n_replicas, N, offload_util_pm=700)
    peers["cap_true_tok_s"] = np.ascontiguousarray(np.broadcast_to(cap, shape))
    if not offload:
        peers["offload_ppm"] = np.zeros(shape, np.uint32)
    rshape = (n_replicas, Q)
    requests = {"origin": np.ascontiguousarray(np.broadcast_to(origin, rshape)),
                "t_ms": np.ascontiguousarray(np.broadcast_to(t_ms, rshape)),
                "len_in": np.clip(np.rint(np.exp(rng.normal(math.log(300.0), 0.5, rshape))), 1, 8192).astype(np.uint16),
                "len_out": np.clip(np.rint(np.exp(rng.normal(math.log(6000.0), 0.5, rshape))), 1, 8192).astype(np.uint16)}
    return Workload(name, st, peers, requests, batch=batch, gossip_every=1)


SWEEP_AXES = ("stake", "accept", "offload")


def make_policy_sweep(*, seed: int = 0, replicas_per_axis: int = 32, n_requests: int = 4000, batch: int = 500) -> Workload:
    """The ablation on user-level policies as one batched run: a requester-only node 0 and four
    providers (nodes 1-4), pure stake-proportional selection, and three groups of replicas that
    differ in one policy each, every replica an independent repetition:

      stake    stakes 1:2:3:4 (per-mille of credit 250, 500, 750, 1000), everybody accepts;
      accept   equal stakes, acceptance frequencies 0.25, 0.5, 0.75, 1.0, at most three probes;
      offload  requests arrive at the providers themselves, offloading frequencies 0.25 .. 1.0.

    `wl.axis[r]` names the group of replica r (index into SWEEP_AXES)."""
    rng = np.random.default_rng(np.random.PCG64(seed))
    N, Rp, Q = 5, 3 * replicas_per_axis, n_requests
    st = Settings(N, Rp, seed=seed, fanout_k=2, p_duel_ppm=100_000, max_probes=3, n_judges=1, flags=0)
    shape = (Rp, N)
    axis = np.repeat(np.arange(3), replicas_per_axis)
    ramp = np.array([0, 0.25, 0.5, 0.75, 1.0])
    cap = np.full(shape, 2000, np.uint32); cap[axis != 2, 0] = 0            # node 0 only issues requests
    stake = np.full(shape, 1000, np.uint16); stake[axis == 0] = (1000 * ramp).astype(np.uint16); stake[axis == 0, 0] = 1000
    accept = np.full(shape, 1_000_000, np.uint32); accept[axis == 1] = (1e6 * ramp).astype(np.uint32)
    offload = np.full(shape, 1_000_000, np.uint32); offload[axis == 2] = (1e6 * ramp).astype(np.uint32)
    peers = {
        "cap_true_tok_s": cap, "quality_fx": _quality_to_fx(rng.random(shape)),
        "credit0": np.full(shape, 10 ** 9, np.int64), "stake_pm": stake,
        "offload_util_pm": np.zeros(shape, np.uint16), "accept_util_pm": np.full(shape, 1001, np.uint16),
        "offload_ppm": offload, "accept_ppm": accept,
        "misreport_mul": np.ones(shape, np.uint8), "prio_flag": np.zeros(shape, np.uint8), "online0": np.ones(shape, np.uint8),
    }
    origin = np.zeros((Rp, Q), np.uint32)
    origin[axis == 2] = rng.integers(1, N, (replicas_per_axis, Q))
    t = poisson_times_ms(rng, Q, 20.0)
    rq = {"origin": origin, "t_ms": np.ascontiguousarray(np.broadcast_to(t, (Rp, Q))),
          "len_in": _lengths(rng, (Rp, Q), 512.0), "len_out": _lengths(rng, (Rp, Q), 256.0)}
    wl = Workload("policy_sweep", st, peers, rq, batch=batch, gossip_every=4)
    wl.axis = axis
    return wl


def slice_replicas(wl: Workload, r0: int, r1: int) -> Workload:
    """The same workload restricted to replicas [r0, r1); randomness stays keyed
    by the global replica index through `replica_offset`."""
    st = dataclasses.replace(wl.settings, n_replicas=r1 - r0,
                             replica_offset=wl.settings.replica_offset + r0)
    return Workload(wl.name, st,
                    {k: np.ascontiguousarray(v[r0:r1]) for k, v in wl.peers.items()},
                    {k: np.ascontiguousarray(v[r0:r1]) for k, v in wl.requests.items()},
                    wl.batch, wl.gossip_every, wl.finalize_every)
