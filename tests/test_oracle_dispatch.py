"""Pins for the oracle's dispatch stage.

Assumption 3 fixes the Proof-of-Stake selection probability p_i = s_i / sum_j s_j;
the policy ablation (Section "Impact of User-Level Policies") says delegated load
follows stake 1:2:3:4 and rises with the acceptance frequency.  Sampling without
replacement by successive proportional draws has the Plackett-Luce order law,
whose probabilities are enumerated exactly here.
"""
import itertools
import math

import numpy as np

from oracle import Oracle, binding
from tests.helpers import chi2_ok, entry_cap, entry_offline, entry_q, make_net, requester_first

ST_ORIGIN, ST_DRAW, ST_PROBE = 1, 2, 3


def _philox(seed, index, slot, replica, stage):
    return [int(x) for x in binding.philox4x32_10([index, slot, replica, stage], [seed & 0xFFFFFFFF, seed >> 32])]


def test_pos_share_follows_stake_1_2_3_4():
    Q = 40_000
    st, pa, rq = make_net(5, n_requests=Q, seed=4, flags=0, p_duel_ppm=0,
                          peers=requester_first(5, stake_pm=np.array([1000, 250, 500, 750, 1000])))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q)
    ex = o.results()["exec_a"][0]
    assert ex.min() >= 1
    cnt = np.bincount(ex, minlength=5)[1:]
    ok, stat, df = chi2_ok(cnt, Q * np.array([0.1, 0.2, 0.3, 0.4]))
    assert ok, (cnt, stat)


def _weights_second_routine(st, view_row, stake, wins, duels, o, blk):
    """The integer weights of one window, computed again with vectorised numpy fp32."""
    ids = 32 * blk + np.arange(32)
    W = np.zeros(32, np.uint64); sc = np.zeros(32, np.float32)
    inb = ids < st.n_peers
    idc = np.where(inb, ids, 0)
    e = view_row[idc]
    cap = entry_cap(e).astype(np.float32); q16 = (entry_q(e) * np.uint64(16)).astype(np.float32)
    elig = inb & (ids != o) & (e != 0) & (entry_offline(e) == 0) & (stake[idc] > 0) & (cap > 0)
    uwf = np.float32(st.util_window_ms) / np.float32(1000.0)
    with np.errstate(divide="ignore", invalid="ignore"):
        rep = (wins[idc] + 1).astype(np.float32) / (duels[idc] + 2).astype(np.float32) if st.flags & 1 else np.float32(1)
        spare = np.maximum(np.float32(0), np.float32(1) - q16 / (cap * uwf)) if st.flags & 2 else np.float32(1)
        score = (stake[idc].astype(np.float32) * rep).astype(np.float32) * spare
    scaled = (score.astype(np.float32) * np.float32(256)).astype(np.float32)
    W[elig] = np.minimum(np.floor(scaled[elig].astype(np.float64)), 2.0 ** 56).astype(np.uint64)
    sc[elig & (W > 0)] = score[elig & (W > 0)]
    return W, sc


def test_pick_is_the_lane_whose_integer_interval_holds_the_draw():
    """Run a mixed network for a few steps, then check every first pick of a big
    batch against weights recomputed by a second routine and big-integer prefix sums."""
    N, Q = 70, 3000          # three blocks, the last one ragged (6 peers)
    rng = np.random.default_rng(0)
    peers = {"cap_true_tok_s": rng.integers(500, 8000, N), "stake_pm": rng.integers(0, 1001, N),
             "quality_fx": rng.integers(0, 2 ** 32, N, dtype=np.uint64)}
    st, pa, rq = make_net(N, n_requests=Q, seed=21, p_duel_ppm=300_000, peers=peers,
                          origin=rng.integers(0, N, Q), max_probes=1)
    o = Oracle(st, pa); o.bind_requests(rq)
    for s in range(4):      # build up backlog, reputation and adverts
        o.run_step(s * 500, 500, 1000 * (s + 1), True)
    first, cnt = 2000, 1000
    o.advance_time(5000); o.gossip_round()
    view = o.view()[0]; stake = o.table("stake")[0]; wins = o.table("wins")[0]; duels = o.table("duels")[0]
    o.dispatch_batch(first, cnt)
    res = o.results()
    checked = near = 0
    for q in range(first, first + cnt):
        a = res["exec_a"][0, q]
        if a in (-1, -3, -4):
            continue
        orig = int(rq["origin"][0, q])
        W, sc, blk = o.window_weights(0, q)
        x = _philox(st.seed, q, 0, 0, ST_ORIGIN)
        assert blk == (orig // 32 + ((x[2] * 3) >> 32)) % 3
        W2, sc2 = _weights_second_routine(st, view[orig], stake, wins, duels, orig, blk)
        assert np.array_equal(W, W2) and np.array_equal(sc, sc2)
        S = int(W.astype(object).sum())
        if S == 0:
            assert a == -2
            continue
        y = _philox(st.seed, q, 0, 0, ST_DRAW)
        r64 = (((y[0] << 32) | y[1]) * S) >> 64
        incl = np.cumsum(W.astype(object))
        lane = int(np.searchsorted(np.array(incl, dtype=object) > r64, True))
        assert W[lane] > 0
        lo, hi = (int(incl[lane]) - int(W[lane])), int(incl[lane])
        assert lo <= r64 < hi
        is_near = min(r64 - lo, hi - 1 - r64) <= S // 100000
        near += is_near
        assert (res["flags"][0, q] & 1) == int(is_near)
        # max_probes = 1: the first pick is the executor iff its probe accepted
        if a >= 0:
            assert a == 32 * blk + lane
            assert res["score_a"][0, q] == sc[lane]
            f = np.float32(0)
            for v in sc:
                f = np.float32(f + v)
            assert res["score_sum"][0, q] == f
        checked += 1
    assert checked > 500


def test_plackett_luce_order_probabilities():
    """Executor, challenger and two judges of a duel are four successive draws
    without replacement from four candidates: all 24 orders, exact probabilities."""
    Q = 60_000
    w = np.array([0, 1, 2, 3, 4], float)
    st, pa, rq = make_net(5, n_requests=Q, seed=8, flags=0, p_duel_ppm=1_000_000, n_judges=2,
                          peers=requester_first(5, stake_pm=(w * 250).astype(int).clip(0) + np.array([1000, 0, 0, 0, 0])))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q); o.duel_judge()
    res = o.results()
    assert np.all(res["outcome"][0] != 4) and np.all(res["outcome"][0] != 0)
    order = np.stack([res["exec_a"][0], res["exec_b"][0], res["judges"][0, :, 0], res["judges"][0, :, 1]], 1)
    perms = list(itertools.permutations([1, 2, 3, 4]))
    obs, exp = [], []
    for p in perms:
        rest, pr = w[1:].sum(), 1.0
        for node in p:
            pr *= w[node] / rest
            rest -= w[node]
        exp.append(pr * Q)
        obs.append(int(np.all(order == np.array(p)[None, :], axis=1).sum()))
    assert sum(obs) == Q
    ok, stat, df = chi2_ok(obs, exp)
    assert ok, (stat, df)


def test_share_rises_with_acceptance_frequency_exact_law():
    """Equal stakes, acceptance frequencies .25/.5/.75/1, three probes at most:
    P(executor = i) by enumeration of draw orders and refusals."""
    Q = 60_000
    acc = np.array([0, 0.25, 0.5, 0.75, 1.0])
    st, pa, rq = make_net(5, n_requests=Q, seed=13, flags=0, p_duel_ppm=0, max_probes=3,
                          peers=requester_first(5, accept_ppm=(acc * 1e6).astype(int)))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q)
    ex = o.results()["exec_a"][0]
    p = np.zeros(6)   # index 1..4 executors, 5 = nobody willing
    for perm in itertools.permutations([1, 2, 3, 4], 3):
        pr = 1.0 / (4 * 3 * 2)
        refused = 1.0
        for node in perm:
            p[node] += pr * refused * acc[node]
            refused *= 1 - acc[node]
        p[5] += pr * refused
    obs = np.array([(ex == i).sum() for i in (1, 2, 3, 4)] + [(ex == -4).sum()])   # origin has no capacity
    assert obs.sum() == Q
    ok, stat, df = chi2_ok(obs, Q * p[1:])
    assert ok, (obs, Q * p[1:], stat)
    assert obs[0] < obs[1] < obs[2] < obs[3]
    assert o.stats_dict()["n_probes"] > Q


def test_origin_policy_cases():
    """Hand cases of the local-vs-delegate rule (Section "Request Routing and Node Design")."""
    N, Q = 4, 8
    origin = np.array([0, 1, 2, 3, 0, 1, 2, 3])
    peers = {"offload_util_pm": np.array([700, 700, 0, 0]), "credit0": np.array([10_000, 10_000, 50, 10_000]),
             "online0": np.array([1, 1, 1, 0])}
    st, pa, rq = make_net(N, n_requests=Q, peers=peers, origin=origin, p_duel_ppm=0, flags=0)
    o = Oracle(st, pa); o.bind_requests(rq)
    # util window = 10 s * 2000 tok/s = 20000 tokens; 700 per mille = 14000 tokens
    o.poke_peer(0, 0, backlog=14_000)     # exactly at the threshold: offloads
    o.poke_peer(0, 1, backlog=13_999)     # just below: stays local
    o.dispatch_batch(0, Q)
    ex = o.results()["exec_a"][0]
    assert ex[0] >= 0 and ex[4] >= 0 and ex[0] != 0
    assert ex[1] == -1 and ex[5] == -1
    assert ex[2] == -1 and ex[6] == -1      # cannot afford R = 100 with 50 credits
    assert ex[3] == -3 and ex[7] == -3      # origin offline: dropped
    assert not np.isin(ex[[0, 4]], [3]).any()   # offline peer is never an executor


def test_probe_uses_true_state_not_the_advert():
    """A candidate whose true utilisation is at its accept threshold refuses even
    though the origin's (stale) view shows it idle; fallback is local service."""
    N, Q = 3, 200
    st, pa, rq = make_net(N, n_requests=Q, p_duel_ppm=0, peers={"accept_util_pm": 700, "credit0": 10 ** 7})
    o = Oracle(st, pa); o.bind_requests(rq)
    o.poke_peer(0, 1, backlog=14_000)
    o.dispatch_batch(0, Q)
    ex = o.results()["exec_a"][0]
    assert set(np.unique(ex)) == {2}
    o.duel_judge(); o.settle_credits(True)
    o.poke_peer(0, 2, backlog=20_000)
    o.dispatch_batch(0, Q)
    assert np.all(o.results()["exec_a"][0] == -2)
    # offload frequency: Bernoulli(offload_ppm)
    st2, pa2, rq2 = make_net(3, n_requests=20_000, p_duel_ppm=0, peers={"offload_ppm": 800_000})
    o2 = Oracle(st2, pa2); o2.bind_requests(rq2)
    o2.dispatch_batch(0, 20_000)
    frac = (o2.results()["exec_a"][0] >= 0).mean()
    assert abs(frac - 0.8) < 5 * math.sqrt(0.8 * 0.2 / 20_000)


def test_load_and_reputation_factors_shift_the_share():
    """With the load factor on, a candidate advertising a half-full queue gets half the weight."""
    Q = 30_000
    st, pa, rq = make_net(3, n_requests=Q, p_duel_ppm=0, flags=2, seed=6, peers=requester_first(3))
    o = Oracle(st, pa); o.bind_requests(rq)
    # entry of peer 1 in the origin's row: version 5, capacity 2000, queue 10000 tokens = 625 units of 16
    o.poke_view(0, 0, 1, (5 << 40) | (2000 << 20) | 625)
    o.dispatch_batch(0, Q)
    ex = o.results()["exec_a"][0]
    n1 = (ex == 1).sum()
    assert abs(n1 - Q / 3) < 5 * math.sqrt(Q * (1 / 3) * (2 / 3))   # weights 0.5 : 1
    W, sc, _ = o.window_weights(0, 0)
    assert W[1] * 2 == W[2] and sc[1] * 2 == sc[2]


def test_tiny_weights_hit_interval_boundaries_exactly():
    """Stakes of a few credits give weights of a few hundred, so draws land on interval
    ends often; the pick must be the lane with prefix_excl <= r64 < prefix_incl."""
    N, Q = 6, 6000
    st, pa, rq = make_net(N, n_requests=Q, seed=77, flags=0, p_duel_ppm=0,
                          peers=requester_first(N, credit0=np.array([10 ** 6, 1, 2, 3, 1, 2])))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q)
    res = o.results()
    W, _, blk = o.window_weights(0, 0)
    assert list(W[:6]) == [0, 256, 512, 768, 256, 512] and blk == 0
    S = int(W.astype(object).sum()); incl = np.cumsum(W.astype(object))
    on_edge = 0
    for q in range(Q):
        y = _philox(st.seed, q, 0, 0, ST_DRAW)
        r64 = (((y[0] << 32) | y[1]) * S) >> 64
        lane = next(c for c in range(32) if incl[c] > r64)
        assert res["exec_a"][0, q] == lane
        lo, hi = int(incl[lane]) - int(W[lane]), int(incl[lane])
        assert (res["flags"][0, q] & 1) == int(r64 == lo or r64 == hi - 1)     # tolerance S // 100000 = 0
        on_edge += int(r64 in [int(v) for v in incl[:6]] or r64 + 1 in [int(v) for v in incl[:6]])
    assert on_edge > 20


def test_truly_offline_peers_never_serve_or_judge():
    """Peers that crashed but are still believed online get drawn, fail their probe,
    and are skipped as judges."""
    N, Q = 12, 5000
    st, pa, rq = make_net(N, n_requests=Q, seed=41, flags=0, p_duel_ppm=1_000_000, n_judges=3, max_probes=6,
                          peers=requester_first(N, credit0=10 ** 8))
    o = Oracle(st, pa); o.bind_requests(rq)
    dead = [2, 5, 6, 9]
    for j in dead:
        o.poke_peer(0, j, online=0)
    o.dispatch_batch(0, Q); o.duel_judge()
    res = o.results()
    assert not np.isin(res["exec_a"][0], dead).any() and not np.isin(res["exec_b"][0], dead).any()
    assert not np.isin(res["judges"][0], dead).any()
    decided = np.isin(res["outcome"][0], (1, 2, 3))
    assert decided.mean() > 0.9
    assert np.all((res["judges"][0][decided] >= 0).sum(-1) == 3)     # 7 live candidates: always a full panel
    assert o.stats_dict()["n_probes"] > 2 * Q                          # refused probes were spent on the dead


def test_greedy_rule_takes_the_best_weight_then_the_next():
    """Greedy dispatch (flag 4): executor = highest weight of the window recomputed by the
    second routine; a refusing best candidate hands over to the runner-up; ties go to the
    lowest id; the flag marks a runner-up within 1e-5."""
    N, Q = 70, 1500
    rng = np.random.default_rng(3)
    peers = {"cap_true_tok_s": rng.integers(500, 8000, N), "stake_pm": rng.integers(1, 1001, N)}
    st, pa, rq = make_net(N, n_requests=Q, seed=9, flags=3 | 4, p_duel_ppm=1_000_000, n_judges=2, peers=peers,
                          origin=rng.integers(0, N, Q), max_probes=2)
    o = Oracle(st, pa); o.bind_requests(rq)
    for s in range(2):
        o.run_step(s * 500, 500, 1000 * (s + 1), True)
    o.advance_time(3000); o.gossip_round()
    view = o.view()[0]; stake = o.table("stake")[0]; wins = o.table("wins")[0]; duels = o.table("duels")[0]
    o.dispatch_batch(1000, 500); o.duel_judge()
    res = o.results()
    n_chk = 0
    for q in range(1000, 1500):
        a = res["exec_a"][0, q]
        if a < 0:
            continue
        orig = int(rq["origin"][0, q])
        _, _, blk = o.window_weights(0, q)
        W, _ = _weights_second_routine(st, view[orig], stake, wins, duels, orig, blk)
        order = sorted(range(32), key=lambda c: (-int(W[c]), c))
        order = [c for c in order if W[c] > 0]
        got = [a, res["exec_b"][0, q]] + list(res["judges"][0, q, :2])
        got = [g - 32 * blk for g in got if g >= 0]
        assert got == order[:len(got)], (q, got, order[:6])     # all peers accept: strict weight order
        n_chk += 1
    assert n_chk > 300
    # refusal: the best candidate never accepts -> the runner-up serves; tie -> lowest id
    st2, pa2, rq2 = make_net(6, n_requests=50, flags=4, p_duel_ppm=0,
                             peers=requester_first(6, credit0=np.array([10 ** 6, 500, 900, 900, 100, 100]),
                                                   accept_ppm=np.array([0, 10 ** 6, 0, 10 ** 6, 10 ** 6, 10 ** 6])))
    o2 = Oracle(st2, pa2); o2.bind_requests(rq2)
    o2.dispatch_batch(0, 50)
    r2 = o2.results()
    assert np.all(r2["exec_a"][0] == 3)           # 2 and 3 tie at the top, 2 is asked first and refuses
    assert np.all(r2["flags"][0] & 1 == 1)        # a tie is as near as it gets
    assert o2.stats_dict()["n_probes"] == 100
    # near flag threshold: weights 256*100000 vs 256*99999 differ by 256 <= W/100000 = 256 -> flagged;
    # 256*100000 vs 256*99998 differ by 512 -> not flagged
    for other, flagged in ((99_999, 1), (99_998, 0)):
        st3, pa3, rq3 = make_net(3, n_requests=4, flags=4, p_duel_ppm=0,
                                 peers=requester_first(3, credit0=np.array([10 ** 6, 100_000, other])))
        o3 = Oracle(st3, pa3); o3.bind_requests(rq3)
        o3.dispatch_batch(0, 4)
        assert np.all(o3.results()["exec_a"][0] == 1) and np.all((o3.results()["flags"][0] & 1) == flagged)


def test_candidate_block_follows_the_rank_distribution():
    """D3: the candidate window is the block `rank` places after the origin's own block on the id
    ring; the rank is uniform, or drawn from a supplied distribution (Zipf(1.1) in config 3).
    Equal stakes, everybody accepts, so the executor is uniform inside the chosen block."""
    from paper_2603_20661_b200 import synth
    N, Q, origin = 160, 60_000, 70                                # five blocks of 32; the origin sits in block 2
    for cdf, law in ((None, np.full(5, 0.2)),
                     (synth.zipf_rank_cdf(5, 1.1), (1 / np.arange(1, 6) ** 1.1) / (1 / np.arange(1, 6) ** 1.1).sum()),
                     (synth.zipf_rank_cdf(3, 1.1), np.r_[(1 / np.arange(1, 4) ** 1.1) / (1 / np.arange(1, 4) ** 1.1).sum(), 0, 0])):
        kw = {} if cdf is None else {"rank_cdf": cdf}
        st, pa, rq = make_net(N, n_requests=Q, seed=21, flags=0, p_duel_ppm=0, origin=np.full(Q, origin, np.uint32),
                              peers={"cap_true_tok_s": np.where(np.arange(N) == origin, 0, 2000), "credit0": 10 ** 9}, **kw)
        o = Oracle(st, pa); o.bind_requests(rq)
        o.dispatch_batch(0, Q)
        ex = o.results()["exec_a"][0]
        assert ex.min() >= 0 and np.all(ex != origin)
        by_rank = np.bincount((ex // 32 - origin // 32) % 5, minlength=5)      # rank 0 = the origin's own block
        ok, stat, _ = chi2_ok(by_rank, Q * law)
        assert ok, (by_rank, Q * law, stat)
        # inside a block: uniform over its eligible peers (31 in the origin's block, 32 elsewhere)
        for blk in range(5):
            cnt = np.bincount(ex[ex // 32 == blk] - 32 * blk, minlength=32)
            if cnt.sum() == 0:
                continue
            elig = np.array([32 * blk + c != origin for c in range(32)])
            ok, stat, _ = chi2_ok(cnt, cnt.sum() * elig / elig.sum())
            assert ok, (blk, stat)
