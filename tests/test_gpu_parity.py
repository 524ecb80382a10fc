"""GPU parity: the CUDA library against the CPU oracle, bit for bit, through the C-ABI.

Views, ledgers, queues, executor choices, duel pairings, judge panels, outcomes and
counters must be identical; fp32 scores within 1e-5 relative.
"""
import os

import numpy as np
import pytest

from oracle import Oracle
from paper_2603_20661_b200 import synth
from tests.helpers import assert_same_state, make_net, requester_first

pytestmark = pytest.mark.gpu


def _pair(wl, max_batch=None):
    from paper_2603_20661_b200.binding import Network
    g = Network(wl.settings, wl.peers, max_batch or wl.batch)
    g.bind_requests(wl.requests)
    o = Oracle(wl.settings, wl.peers)
    o.bind_requests(wl.requests)
    return g, o


CASES = [
    ("tiny", {}, None),
    ("tiers64", dict(n_requests=6000), None),
    ("zipf1k", dict(n_replicas=3, n_requests=2500), None),
    ("churn4k", dict(n_replicas=2, n_requests=6000, n_peers=1100), None),      # ragged last block (1100 = 34*32+12)
    ("adversarial16k", dict(n_replicas=2, n_requests=3000, n_peers=2048), None),
]


@pytest.mark.parametrize("name,kw,steps", CASES, ids=[c[0] for c in CASES])
def test_six_calls_match_oracle_after_every_call(name, kw, steps):
    wl = synth.make_workload(name, **kw)
    g, o = _pair(wl)
    n = wl.n_steps if steps is None else steps
    assert_same_state(g, o, "after create")
    for s in range(n):
        first = s * wl.batch
        cnt = min(wl.batch, wl.n_requests - first)
        gossip = s % wl.gossip_every == 0
        full = s < 3 or s == n - 1          # compare after every call early on, then once per step
        for sim in (g, o):
            sim.advance_time(wl.step_now_ms(s))
        if full:
            assert_same_state(g, o, f"step {s} advance", views=False)
        if gossip:
            g.gossip_round(); o.gossip_round()
            if full or s % 7 == 0:
                assert_same_state(g, o, f"step {s} gossip")
        g.dispatch_batch(first, cnt); o.dispatch_batch(first, cnt)
        if full:
            assert_same_state(g, o, f"step {s} dispatch", upto=first + cnt, views=False, stats=False)
        g.duel_judge(); o.duel_judge()
        if full:
            assert_same_state(g, o, f"step {s} duel", upto=first + cnt, views=False, stats=False)
        g.settle_credits(True); o.settle_credits(True)
        assert_same_state(g, o, f"step {s} settle", upto=first + cnt, views=False)
    assert_same_state(g, o, "end", upto=wl.n_requests)
    assert o.error() == 0
    sd = g.stats_dict()
    assert sd["n_requests"] == wl.settings.n_replicas * wl.n_requests
    assert sd["credit_total"] == int(wl.peers["credit0"].sum())


@pytest.mark.parametrize("name,kw,steps", CASES, ids=[c[0] for c in CASES])
def test_six_calls_with_thread_kernels_match_oracle(name, kw, steps):
    """The thread-per-request implementation of the separate dispatch and duel calls, forced on."""
    wl = synth.make_workload(name, **kw)
    g, o = _pair(wl)
    g.set_option(0, 2)
    for s in range(wl.n_steps):
        first = s * wl.batch
        cnt = min(wl.batch, wl.n_requests - first)
        for sim in (g, o):
            sim.advance_time(wl.step_now_ms(s))
            if s % wl.gossip_every == 0:
                sim.gossip_round()
            sim.dispatch_batch(first, cnt)
        if s < 3:
            assert_same_state(g, o, f"step {s} dispatch", upto=first + cnt, views=False, stats=False)
        g.duel_judge(); o.duel_judge()
        if s < 3:
            assert_same_state(g, o, f"step {s} duel", upto=first + cnt, views=False, stats=False)
        g.settle_credits(s % 2 == 0); o.settle_credits(s % 2 == 0)
        if s < 3 or s % 5 == 0:
            assert_same_state(g, o, f"step {s} settle", upto=first + cnt, views=False)
    assert_same_state(g, o, "end", upto=wl.n_requests)


@pytest.mark.parametrize("name,kw,steps", CASES, ids=[c[0] for c in CASES])
def test_fused_step_matches_oracle(name, kw, steps):
    wl = synth.make_workload(name, **kw)
    g, o = _pair(wl)
    for s in range(wl.n_steps):
        first = s * wl.batch
        cnt = min(wl.batch, wl.n_requests - first)
        gossip = s % wl.gossip_every == 0
        fin = s % 3 != 1                     # leave some blocks pending across steps
        g.step(first, cnt, wl.step_now_ms(s), gossip, fin)
        o.run_step(first, cnt, wl.step_now_ms(s), gossip, fin)
        if s < 2 or s % 5 == 0:
            assert_same_state(g, o, f"fused step {s}", upto=first + cnt, views=gossip)
    assert_same_state(g, o, "fused end", upto=wl.n_requests)


STEP_KERNELS = {"8_lanes": 1, "4_lanes": 2, "thread": 3, "stream": 4}


@pytest.mark.parametrize("batch,flags,kernel,run", [
    (250, 3, "8_lanes", 0), (1500, 3, "4_lanes", 0), (5000, 3, "thread", 0), (10000, 3, "thread", 0),
    (250, 7, "8_lanes", 0), (1500, 7, "4_lanes", 0), (1500, 19, "4_lanes", 0), (5000, 7, "thread", 0),
    (250, 3, "stream", 32), (1500, 3, "stream", 64), (5000, 3, "stream", 0), (5000, 3, "stream", 512), (10000, 3, "stream", 96),
    (10000, 3, "stream", 0), (1500, 7, "stream", 64), (5000, 19, "stream", 160), (5000, 0, "stream", 0), (1500, 35, "stream", 2048),
    (5000, 3, None, 0), (10000, 3, None, 0)],
    ids=lambda v: str(v))
def test_fused_step_with_every_kernel_matches_oracle(batch, flags, kernel, run):
    """The fused step has four implementations with identical results (8 or 4 lanes per request,
    one thread per request, streaming phases with runs of `run` requests per warp); each is forced
    on here, and left to the launch size in the last two cases: 8 replicas x batch = 2,000 /
    12,000 / 40,000 / 80,000 requests per launch."""
    wl = synth.make_workload("zipf1k", n_replicas=8, n_requests=2 * batch, n_peers=300)
    wl.batch = batch
    wl.settings.flags = flags
    wl.settings.p_duel_ppm = 150_000
    g, o = _pair(wl)
    if kernel:
        g.set_option(1, STEP_KERNELS[kernel])
        g.set_option(2, run)
        g.set_option(3, 15 if batch % 1000 else 0)   # launches overlapped with their predecessor's tail, or plain
    for s in range(2):
        g.step(s * batch, batch, wl.step_now_ms(s), s == 0, s == 1)
        o.run_step(s * batch, batch, wl.step_now_ms(s), s == 0, s == 1)
        assert_same_state(g, o, f"batch {batch} step {s}", upto=(s + 1) * batch, views=s == 0)
    assert o.stats_dict()["n_duel"] > 0.05 * o.stats_dict()["n_delegated"] > 0


@pytest.mark.parametrize("case", ["all_duels_four_judges", "one_probe", "nobody_accepts", "all_local", "ragged_window", "no_scores"])
def test_streaming_kernel_corner_cases_match_oracle(case):
    """The streaming kernel where its queues are stressed: every delegated request a duel with four
    judges (the draw queue recirculates), a probe budget of one, nobody accepting (all fall back),
    nobody offloading (everything goes straight to the finish queue), a last candidate block of 12."""
    kw = dict(n_replicas=3, n_requests=3000, n_peers=300)
    if case == "ragged_window":
        kw["n_peers"] = 44
    wl = synth.make_workload("zipf1k", **kw)
    wl.batch = 1500
    st = wl.settings
    if case == "all_duels_four_judges":
        st.p_duel_ppm, st.n_judges, st.p_noise_ppm = 1_000_000, 4, 200_000
    elif case == "one_probe":
        st.max_probes, st.p_duel_ppm = 1, 400_000
    elif case == "nobody_accepts":
        wl.peers["accept_ppm"][:] = 0
    elif case == "all_local":
        wl.peers["offload_ppm"][:] = 0
    elif case == "ragged_window":
        st.rank_cdf = None
        st.p_duel_ppm = 500_000
    g, o = _pair(wl)
    if case == "no_scores":
        g.bind_requests(wl.requests, scores=False)
    g.set_option(1, 4)
    for s in range(2):
        g.set_option(2, (96, 0)[s])
        g.step(s * 1500, 1500, wl.step_now_ms(s), s == 0, True)
        o.run_step(s * 1500, 1500, wl.step_now_ms(s), s == 0, True)
        assert_same_state(g, o, f"{case} step {s}", upto=(s + 1) * 1500, views=s == 0, scores=case != "no_scores")


@pytest.mark.parametrize("pinned,mode", [(True, 1), (True, 2), (True, 0), (False, 0)],
                         ids=["mapped_direct", "pinned_staged", "pinned_by_size", "pageable_staged"])
def test_step_host_roundtrip_matches_oracle(pinned, mode):
    """Host buffers both ways: page-locked buffers used by the kernels directly, and staged copies
    (second stream beside the kernels) from page-locked or pageable buffers."""
    import torch
    from paper_2603_20661_b200.binding import Network
    wl = synth.make_workload("zipf1k", n_replicas=2, n_requests=1500, n_peers=256)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    g = Network(wl.settings, wl.peers, wl.batch)
    Rp, Q = wl.settings.n_replicas, wl.n_requests
    # device arrays start as garbage: everything must arrive through the host copies
    g.bind_requests({k: np.full((Rp, Q), 7, v.dtype) for k, v in wl.requests.items()}, scores=False)
    g.set_option(4, mode)
    direct = pinned and mode != 2                    # 2 x 500 requests per step: small enough for the direct path
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    io = {"origin": pin(torch.from_numpy(wl.requests["origin"].view(np.int32).copy())),
          "len_in": pin(torch.from_numpy(wl.requests["len_in"].view(np.int16).copy())),
          "len_out": pin(torch.from_numpy(wl.requests["len_out"].view(np.int16).copy())),
          "exec_a": pin(torch.full((Rp, Q), -9, dtype=torch.int32)),
          "exec_b": pin(torch.full((Rp, Q), -9, dtype=torch.int32)),
          "judges": pin(torch.full((Rp, Q, 4), -9, dtype=torch.int32)),
          "outcome": pin(torch.zeros((Rp, Q), dtype=torch.uint8)),
          "flags": pin(torch.zeros((Rp, Q), dtype=torch.uint8))}
    for s in range(wl.n_steps):
        first = s * wl.batch
        tot = g.step_host(io, first, wl.batch, wl.step_now_ms(s), s % wl.gossip_every == 0)
        o.run_step(first, wl.batch, wl.step_now_ms(s), s % wl.gossip_every == 0)
        assert np.array_equal(tot, o.stats()[-1])
    ro = o.results()
    for k in ("exec_a", "exec_b", "judges", "outcome", "flags"):
        assert np.array_equal(io[k].numpy(), ro[k]), k
    # the bound device arrays hold the results only on the copying path
    assert_same_state(g, o, "host path end", upto=None if direct else Q)


def test_determinism_and_replica_sharding():
    """Same seed twice gives the same bytes; replicas [2,4) run alone (replica_offset = 2)
    give the same results as inside the 4-replica network."""
    from paper_2603_20661_b200.binding import Network
    wl = synth.make_workload("churn4k", n_replicas=4, n_requests=3000, n_peers=512)
    outs = []
    for _ in range(2):
        g = Network(wl.settings, wl.peers, wl.batch); g.bind_requests(wl.requests)
        for s in range(wl.n_steps):
            g.step(s * wl.batch, wl.batch, wl.step_now_ms(s), s % wl.gossip_every == 0)
        outs.append((g.results(), g.view(), g.table("credit"), g.stats()))
        g.close()
    for k in outs[0][0]:
        assert np.array_equal(outs[0][0][k], outs[1][0][k])
    assert np.array_equal(outs[0][1], outs[1][1]) and np.array_equal(outs[0][3], outs[1][3])
    half = synth.slice_replicas(wl, 2, 4)
    g = Network(half.settings, half.peers, half.batch); g.bind_requests(half.requests)
    for s in range(half.n_steps):
        g.step(s * half.batch, half.batch, half.step_now_ms(s), s % half.gossip_every == 0)
    res = g.results()
    for k in res:
        assert np.array_equal(res[k], outs[0][0][k][2:4])
    assert np.array_equal(g.view(), outs[0][1][2:4]) and np.array_equal(g.table("credit"), outs[0][2][2:4])
    assert np.array_equal(g.stats()[:2], outs[0][3][2:4])


@pytest.mark.parametrize("n_peers,k,churn", [(1100, 4, 60_000), (300, 2, 0), (40, 1, 200_000)])
def test_push_pull_gossip_matches_oracle(n_peers, k, churn):
    """Full pairwise exchange (flag 8): reverse lists + merge over a variable number of rows."""
    wl = synth.make_workload("churn4k", n_replicas=2, n_requests=4000, n_peers=n_peers)
    wl.settings.flags |= 8
    wl.settings.fanout_k = k
    wl.settings.p_leave_ppm = wl.settings.p_join_ppm = churn
    g, o = _pair(wl)
    for s in range(wl.n_steps):
        first = s * wl.batch
        g.advance_time(wl.step_now_ms(s)); o.advance_time(wl.step_now_ms(s))
        for _ in range(2):                       # two rounds per step
            g.gossip_round(); o.gossip_round()
        assert_same_state(g, o, f"push-pull step {s} gossip")
        g.dispatch_batch(first, wl.batch); o.dispatch_batch(first, wl.batch)
        g.duel_judge(); o.duel_judge()
        g.settle_credits(True); o.settle_credits(True)
    assert_same_state(g, o, "push-pull end", upto=wl.n_requests)


@pytest.mark.parametrize("n_peers,k,churn,stale", [(1024, 4, 60_000, 5), (1100, 4, 60_000, 0), (300, 2, 0, 3), (40, 1, 200_000, 0),
                                                   (2100, 3, 30_000, 2)])
def test_gossip_rounds_on_uniform_and_ragged_rows_match_oracle(n_peers, k, churn, stale):
    """Several gossip rounds per step on row lengths that are and are not a multiple of the
    panel width (1100 peers pad to 1120 columns, 2100 to 2112), with churn and stale initial views."""
    wl = synth.make_workload("churn4k", n_replicas=3, n_requests=4000, n_peers=n_peers)
    wl.settings.fanout_k = k
    wl.settings.p_leave_ppm = wl.settings.p_join_ppm = churn
    wl.settings.init_stale_max = stale
    g, o = _pair(wl)
    for s in range(4):
        g.advance_time(wl.step_now_ms(s)); o.advance_time(wl.step_now_ms(s))
        for _ in range(3):
            g.gossip_round(); o.gossip_round()
        assert_same_state(g, o, f"gossip x3, step {s}")
        first = s * wl.batch
        g.dispatch_batch(first, wl.batch); o.dispatch_batch(first, wl.batch)
        g.duel_judge(); o.duel_judge()
        g.settle_credits(True); o.settle_credits(True)
    assert_same_state(g, o, "gossip x3, end", upto=4 * wl.batch)
    assert g.stats_dict()["rounds"] == 3 * 12


@pytest.mark.parametrize("name,kw", [("tiny", {}), ("tiers64", dict(n_requests=5000)),
                                     ("zipf1k", dict(n_replicas=3, n_requests=2500, n_peers=200))])
def test_fifo_queueing_matches_oracle(name, kw):
    """Exact intra-batch queueing (flag 16) through both call paths, with duels and heavy contention."""
    wl = synth.make_workload(name, **kw)
    wl.settings.flags |= 16
    wl.settings.p_duel_ppm = 300_000
    g, o = _pair(wl)
    g2 = _pair(wl)[0]
    for s in range(wl.n_steps):
        first = s * wl.batch
        cnt = min(wl.batch, wl.n_requests - first)
        gossip = s % wl.gossip_every == 0
        g.step(first, cnt, wl.step_now_ms(s), gossip, s % 2 == 0)
        g2.run_step(first, cnt, wl.step_now_ms(s), gossip, s % 2 == 0)
        o.run_step(first, cnt, wl.step_now_ms(s), gossip, s % 2 == 0)
        if s < 3 or s % 4 == 0:
            assert_same_state(g, o, f"fifo fused step {s}", upto=first + cnt, views=False)
            assert_same_state(g2, o, f"fifo six-call step {s}", upto=first + cnt, views=False)
    assert_same_state(g, o, "fifo fused end", upto=wl.n_requests)
    assert_same_state(g2, o, "fifo six-call end", upto=wl.n_requests)
    base = synth.make_workload(name, **kw)
    assert o.stats_dict()["sum_latency_ms"] > 0


@pytest.mark.parametrize("seed", range(int(os.environ.get("WWWS_FUZZ_SEEDS", "24"))))
def test_random_configurations_match_oracle(seed):
    """Seeded random small networks: sizes, fanout, judges, probe budget, probabilities, all
    combinations of the behaviour flags, skewed ranks, misreporting, churn, stale initial views;
    alternating call paths; everything compared after every step."""
    from paper_2603_20661_b200.binding import Network
    rng = np.random.default_rng(1000 + seed)
    N = int(rng.choice([2, 3, 9, 31, 32, 33, 64, 97, 200, 513]))
    Rp = int(rng.integers(1, 4))
    B = int(rng.choice([1, 7, 60, 120, 3500, 9000]))       # the large ones reach the streaming step kernel when the kernel is chosen by launch size
    Q = max(360, 3 * B)
    n_blk = (N + 31) // 32
    kw = dict(fanout_k=int(rng.integers(1, 5)), gossip_tries=int(rng.integers(1, 9)), max_probes=int(rng.integers(1, 8)),
              n_judges=int(rng.integers(1, 5)), p_duel_ppm=int(rng.choice([0, 100_000, 1_000_000])),
              p_noise_ppm=int(rng.choice([0, 250_000])), p_leave_ppm=int(rng.choice([0, 150_000])),
              p_join_ppm=int(rng.choice([0, 400_000])), hop_ms=int(rng.integers(0, 50)),
              init_stale_max=int(rng.integers(0, 8)), flags=int(rng.integers(0, 64)),
              util_window_ms=int(rng.choice([1000, 10_000])), slo_num=int(rng.integers(1, 4)), slo_den=int(rng.integers(1, 3)),
              reward_R=int(rng.integers(1, 200)), reward_add=int(rng.integers(1, 50)), penalty_P=int(rng.integers(50, 120)))
    if rng.random() < 0.5:
        kw["rank_cdf"] = synth.zipf_rank_cdf(int(rng.integers(1, n_blk + 2)), 1.1)
    shape = (Rp, N)
    peers = {"cap_true_tok_s": rng.integers(0, 9000, shape) * (rng.random(shape) > 0.05),
             "quality_fx": rng.integers(0, 2 ** 32, shape, dtype=np.uint64), "credit0": rng.integers(0, 3000, shape),
             "stake_pm": rng.integers(0, 1001, shape), "offload_util_pm": rng.choice([0, 300, 700, 1001], shape),
             "accept_util_pm": rng.choice([0, 500, 900, 1001], shape), "offload_ppm": rng.integers(0, 1_000_001, shape),
             "accept_ppm": rng.integers(0, 1_000_001, shape), "misreport_mul": rng.integers(1, 5, shape),
             "prio_flag": rng.integers(0, 2, shape), "online0": (rng.random(shape) > 0.1).astype(np.uint8)}
    st, pa, rq = make_net(N, Rp, Q, seed=seed, peers=peers, origin=rng.integers(0, N, (Rp, Q)), **kw)
    rq["len_in"] = rng.integers(1, 8193, (Rp, Q)).astype(np.uint16)
    rq["len_out"] = rng.integers(1, 8193, (Rp, Q)).astype(np.uint16)
    g = Network(st, pa, B); g.bind_requests(rq)
    g.set_option(0, 1 + seed % 2)                # six-call path: warp-per-request / thread-per-request kernels in turn
    g.set_option(1, (0, 3, 4)[seed % 3])         # fused step: by launch size / one thread per request / streaming phases
    if seed % 3 == 2:
        g.set_option(2, int(rng.choice([0, 32, 64, 224])))
    o = Oracle(st, pa); o.bind_requests(rq)
    assert_same_state(g, o, f"seed {seed} create")
    first, step = 0, 0
    while first < Q and step < 40:
        cnt = min(B, Q - first)
        args = (first, cnt, 900 * (step + 1), step % 2 == 0, step % 3 != 2)
        (g.step if step % 2 else g.run_step)(*args)
        o.run_step(*args)
        assert_same_state(g, o, f"seed {seed} step {step} (N={N}, flags={kw['flags']})", upto=first + cnt)
        first += cnt; step += 1
    g.close()


def test_many_replicas_of_a_tiny_network_match_oracle():
    """20,000 replicas of a 3-peer network (the replica axis is a grid dimension of every kernel):
    gossip, a 4-lane launch (one request per replica) and a one-thread launch (three per replica)."""
    from paper_2603_20661_b200.binding import Network
    Rp, N, Q = 20_000, 3, 4
    rng = np.random.default_rng(17)
    st, pa, rq = make_net(N, Rp, Q, seed=9, fanout_k=2, p_duel_ppm=500_000, n_judges=1, p_leave_ppm=50_000, p_join_ppm=300_000,
                          origin=rng.integers(0, N, (Rp, Q)),
                          peers={"cap_true_tok_s": rng.integers(0, 4000, (Rp, N)), "quality_fx": rng.integers(0, 2 ** 32, (Rp, N), dtype=np.uint64),
                                 "accept_ppm": rng.integers(0, 1_000_001, (Rp, N))})
    g = Network(st, pa, 3); g.bind_requests(rq)
    o = Oracle(st, pa); o.bind_requests(rq)
    for s, (first, cnt) in enumerate(((0, 1), (1, 3))):
        g.step(first, cnt, 500 * (s + 1), True)
        o.run_step(first, cnt, 500 * (s + 1), True)
        assert_same_state(g, o, f"many replicas step {s}", upto=first + cnt)
    g.close()


def test_edge_cases_match_oracle():
    """Degenerate networks: two peers, a single request, everybody offline, nobody willing,
    requester-only origin, ragged window, duel probability one with tiny candidate sets."""
    from paper_2603_20661_b200.binding import Network
    rng = np.random.default_rng(5)
    cases = []
    cases.append(make_net(2, n_requests=64, seed=1, p_duel_ppm=1_000_000))                       # never a challenger
    cases.append(make_net(3, n_requests=64, seed=2, p_duel_ppm=1_000_000, n_judges=4))          # never a judge
    cases.append(make_net(4, n_requests=1, seed=3))
    cases.append(make_net(33, n_requests=200, seed=4, origin=rng.integers(0, 33, 200), p_duel_ppm=500_000))
    cases.append(make_net(40, n_requests=200, seed=5, origin=rng.integers(0, 40, 200),
                          peers={"online0": np.zeros(40, np.uint8)}))                            # all dropped
    cases.append(make_net(40, n_requests=200, seed=6, origin=rng.integers(0, 40, 200),
                          peers={"accept_ppm": 0}))                                              # all fallback
    cases.append(make_net(12, n_requests=300, seed=7, p_duel_ppm=1_000_000, n_judges=2, max_probes=2,
                          peers=requester_first(12, accept_ppm=500_000, credit0=10 ** 7)))       # failed (-4)
    cases.append(make_net(64, n_requests=300, seed=8, origin=rng.integers(0, 64, 300), p_duel_ppm=300_000,
                          p_noise_ppm=500_000, hop_ms=25, flags=0, p_leave_ppm=200_000, p_join_ppm=500_000,
                          peers={"stake_pm": rng.integers(0, 1001, 64), "credit0": rng.integers(0, 300, 64),
                                 "prio_flag": 1, "misreport_mul": rng.integers(1, 5, 64)}))
    # greedy rule, with ties (equal stakes) and refusals
    cases.append(make_net(70, n_requests=400, seed=9, origin=rng.integers(0, 70, 400), flags=3 | 4, p_duel_ppm=400_000,
                          peers={"accept_ppm": 600_000, "stake_pm": rng.integers(1, 4, 70) * 300}))
    # majority validation under heavy churn: some blocks stay open
    cases.append(make_net(31, n_requests=300, seed=12, origin=rng.integers(0, 31, 300), flags=3 | 32, p_duel_ppm=300_000,
                          p_leave_ppm=500_000, p_join_ppm=400_000, peers={"credit0": 10 ** 5}))
    # exact queueing + in-block validation with a payer that runs out of covered credit
    cases.append(make_net(6, n_requests=300, seed=11, flags=3 | 16, p_duel_ppm=400_000, n_judges=2,
                          peers=requester_first(6, credit0=np.array([5_000, 10 ** 6, 10 ** 6, 10 ** 6, 10 ** 6, 10 ** 6]))))
    # the same with rewards far beyond 32 bits: payments and in-block spending stay 64-bit throughout
    cases.append(make_net(6, n_requests=300, seed=13, flags=3 | 16, p_duel_ppm=400_000, n_judges=2,
                          reward_R=2 ** 33 + 5, reward_add=2 ** 20 + 1, penalty_P=2 ** 21 + 7,
                          peers=requester_first(6, credit0=np.array([2 ** 39, 2 ** 36, 2 ** 36, 2 ** 35, 2 ** 40, 2 ** 34]))))
    for ci, (st, pa, rq) in enumerate(cases):
        g = Network(st, pa, 128); g.bind_requests(rq)
        o = Oracle(st, pa); o.bind_requests(rq)
        Q = rq["origin"].shape[1]
        first = 0
        step = 0
        while first < Q:
            cnt = min(100, Q - first)
            for sim in (g, o):
                sim.run_step(first, cnt, 700 * (step + 1), True, step % 2 == 0)
            assert_same_state(g, o, f"edge case {ci} step {step}", upto=first + cnt)
            first += cnt; step += 1
        g.close()
