"""Pins for the oracle's duel-and-judge and credit settlement stages.

Assumption 3: Q_i = (1 + q_i - Qbar)/2 with Qbar the stake-weighted mean quality.
Lemma 1: expected payoff per served delegated request R + p_d [Q R_add - (1-Q) P]
(cost c_i = 0: the ledger books no operating costs).
Section "Overhead of Duel-and-Judge Mechanism": N*alpha*p_d*(1+k) extra requests.
Theorem 1: the stake share of the better group grows.
"""
import math

import numpy as np

from oracle import Oracle
from paper_2603_20661_b200 import synth
from tests.helpers import make_net, requester_first, run_workload


def _fx(q):
    return np.minimum(np.floor(np.asarray(q) * 2.0 ** 32), 2.0 ** 32 - 1).astype(np.uint64)


def _duel_run(N, Q, quality, seed, **kw):
    st, pa, rq = make_net(N, n_requests=Q, seed=seed, flags=0, p_duel_ppm=1_000_000,
                          peers=requester_first(N, quality_fx=_fx(quality), credit0=10 ** 9), **kw)
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q); o.duel_judge()
    return o, o.results()


def test_single_judge_win_probability_with_noise():
    """k = 1: P(A wins) = (1-nu) p + nu (1-p), p = (1 + q_A - q_B)/2, per ordered pair."""
    q = np.array([0.0, 0.9, 0.2, 0.6, 0.5])
    nu = 0.1
    o, res = _duel_run(5, 80_000, q, seed=3, n_judges=1, p_noise_ppm=100_000)
    a, b, oc = res["exec_a"][0], res["exec_b"][0], res["outcome"][0]
    assert set(np.unique(oc)) <= {1, 2}
    for A in (1, 2, 3, 4):
        for B in (1, 2, 3, 4):
            if A == B:
                assert not np.any((a == A) & (b == B))
                continue
            m = (a == A) & (b == B)
            n = m.sum()
            p = 0.5 * (1 + q[A] - q[B])
            pw = (1 - nu) * p + nu * (1 - p)
            assert n > 1000
            assert abs((oc[m] == 1).mean() - pw) < 5 * math.sqrt(pw * (1 - pw) / n), (A, B)
    # judges are never one of the duelists nor the origin
    j = res["judges"][0, :, 0]
    assert np.all((j != a) & (j != b) & (j > 0))


def test_three_judges_majority_closed_form():
    q = np.array([0.0, 0.8, 0.3, 0.5, 0.5, 0.5, 0.5])
    o, res = _duel_run(7, 60_000, q, seed=5, n_judges=3)
    a, b, oc = res["exec_a"][0], res["exec_b"][0], res["outcome"][0]
    m = (a == 1) & (b == 2)
    p = 0.5 * (1 + 0.8 - 0.3)
    pm = p ** 3 + 3 * p ** 2 * (1 - p)
    assert abs((oc[m] == 1).mean() - pm) < 5 * math.sqrt(pm * (1 - pm) / m.sum())
    assert np.all(np.isin(oc, (1, 2)))                       # odd panel: no draws
    # two judges (the paper's ablation uses k = 2): ties happen and nothing is decided
    o2, res2 = _duel_run(7, 30_000, q, seed=6, n_judges=2)
    m2 = (res2["exec_a"][0] == 1) & (res2["exec_b"][0] == 2)
    assert abs((res2["outcome"][0][m2] == 3).mean() - 2 * p * (1 - p)) < 5 * math.sqrt(0.25 / m2.sum())


def test_win_rate_reproduces_assumption_3():
    """Averaged over a PoS-drawn opponent, node i wins with (1 + q_i - Qbar_{-i})/2, which
    is the paper's Q_i up to the 1/N effect of never duelling oneself."""
    N = 32
    rng = np.random.default_rng(12)
    q = np.concatenate([[0.0], rng.random(N - 1)])
    stake = np.concatenate([[1000], rng.integers(200, 1001, N - 1)])
    Q = 120_000
    st, pa, rq = make_net(N, n_requests=Q, seed=17, flags=0, p_duel_ppm=1_000_000, n_judges=1,
                          peers=requester_first(N, quality_fx=_fx(q), stake_pm=stake, credit0=10 ** 9))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q); o.duel_judge()
    res = o.results()
    a, oc = res["exec_a"][0], res["outcome"][0]
    s = stake[1:].astype(float); qq = q[1:]
    qbar = (s * qq).sum() / s.sum()
    worst = 0.0
    for i in range(1, N):
        m = a == i
        n = m.sum()
        qbar_wo = ((s * qq).sum() - s[i - 1] * qq[i - 1]) / (s.sum() - s[i - 1])
        exact = 0.5 * (1 + q[i] - qbar_wo)
        emp = (oc[m] == 1).mean()
        assert abs(emp - exact) < 5 * math.sqrt(0.25 / n), i
        worst = max(worst, abs(emp - 0.5 * (1 + q[i] - qbar)))
    assert worst < 5 * math.sqrt(0.25 / (Q / N / 4)) + 1.0 / (N - 2)


def test_extra_request_count_identity_and_expectation():
    wl = synth.make_workload("zipf1k", n_replicas=2, n_requests=4000)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    run_workload(o, wl)
    res = o.results(); sd = o.stats_dict()
    decided = np.isin(res["outcome"], (1, 2, 3))
    nj = (res["judges"] >= 0).sum(-1)
    extra = int((1 + nj[decided]).sum())
    assert extra == sd["n_judge_evals"] + sd["n_duel"] - sd["n_duel_cancelled"]
    assert np.all(nj[~decided] == 0) and np.all(res["exec_b"][~decided] == -1)
    k, pd = wl.settings.n_judges, wl.settings.p_duel_ppm / 1e6
    exp = sd["n_delegated"] * pd * (1 + k)
    assert abs(extra - exp) < 5 * (1 + k) * math.sqrt(sd["n_delegated"] * pd) + (1 + k) * sd["n_duel_cancelled"]
    assert sd["n_requests"] == 8000
    assert sd["n_requests"] == sd["n_local"] + sd["n_fallback_local"] + sd["n_dropped"] + sd["n_failed"] + sd["n_delegated"]


def _ledger_from_results(wl, res, R, R_add, P):
    """Recompute every peer's credit change from the result records alone (vectorised)."""
    Rp, N = wl.settings.n_replicas, wl.settings.n_peers
    d = np.zeros((Rp, N), np.int64)
    for r in range(Rp):
        a, b, oc, jd = res["exec_a"][r], res["exec_b"][r], res["outcome"][r], res["judges"][r]
        o = wl.requests["origin"][r].astype(np.int64)
        deleg = a >= 0
        np.add.at(d[r], o[deleg], -R); np.add.at(d[r], a[deleg], R)
        duel = np.isin(oc, (1, 2, 3))
        np.add.at(d[r], o[duel], -R); np.add.at(d[r], b[duel], R)
        dec = np.isin(oc, (1, 2))
        win = np.where(oc == 1, a, b); lose = np.where(oc == 1, b, a)
        nj = (jd >= 0).sum(-1)
        share = np.where(nj > 0, (P - R_add) // np.maximum(nj, 1), 0)
        np.add.at(d[r], lose[dec], -P)
        np.add.at(d[r], win[dec], (R_add + (P - R_add) - share * nj)[dec])
        for l in range(4):
            m = dec & (jd[:, l] >= 0)
            np.add.at(d[r], jd[m, l], share[m])
    return d


def test_credit_conserved_and_ledger_matches_results():
    for name, kw in (("tiny", {}), ("tiers64", dict(n_requests=5000)), ("zipf1k", dict(n_replicas=2, n_requests=3000)),
                     ("adversarial16k", dict(n_replicas=1, n_peers=1024, n_requests=4000))):
        wl = synth.make_workload(name, **kw)
        o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
        total0 = wl.peers["credit0"].sum(axis=1)

        def check(s, first, cnt):
            st = o.stats()
            assert np.array_equal(st[:-1, 17].astype(np.int64), total0)
        run_workload(o, wl, on_step=check)
        assert o.error() == 0
        st = wl.settings
        d = _ledger_from_results(wl, o.results(), st.reward_R, st.reward_add, st.penalty_P)
        assert np.array_equal(o.table("credit") - wl.peers["credit0"], d)
        assert np.array_equal(o.table("stake"), np.maximum(o.table("credit"), 0) * wl.peers["stake_pm"] // 1000)
        res = o.results()
        for r in range(st.n_replicas):
            dec = np.isin(res["outcome"][r], (1, 2))
            win = np.where(res["outcome"][r] == 1, res["exec_a"][r], res["exec_b"][r])[dec]
            assert np.array_equal(o.table("wins")[r], np.bincount(win, minlength=st.n_peers))
            dl = np.isin(res["outcome"][r], (1, 2, 3))
            both = np.concatenate([res["exec_a"][r][dl], res["exec_b"][r][dl]])
            assert np.array_equal(o.table("duels")[r], np.bincount(both, minlength=st.n_peers))


def test_pending_block_is_invisible_until_finalized():
    st, pa, rq = make_net(6, n_requests=400, seed=1, p_duel_ppm=500_000, peers=requester_first(6))
    o = Oracle(st, pa); o.bind_requests(rq)
    c0 = o.table("credit").copy(); s0 = o.table("stake").copy()
    o.dispatch_batch(0, 50); o.duel_judge(); o.settle_credits(False)
    assert np.array_equal(o.table("credit"), c0) and np.array_equal(o.table("stake"), s0)
    assert o.table("d_credit").sum() == 0 and np.any(o.table("d_credit") != 0)
    assert o.stats_dict()["credit_total"] == c0.sum() and o.stats_dict()["blocks"] == 0
    o.dispatch_batch(50, 50); o.duel_judge(); o.settle_credits(True)
    assert np.all(o.table("d_credit") == 0) and o.table("credit").sum() == c0.sum()
    assert o.stats_dict()["blocks"] == 1
    # uneven judge pot: P - R_add = 30 over 2 judges -> 15 each; over 4 judges -> 7 each, winner keeps 2
    st2, pa2, rq2 = make_net(8, n_requests=300, seed=2, p_duel_ppm=1_000_000, n_judges=4,
                             peers=requester_first(8, credit0=10 ** 6))
    o2 = Oracle(st2, pa2); o2.bind_requests(rq2)
    o2.dispatch_batch(0, 300); o2.duel_judge(); o2.settle_credits(True)
    res = o2.results()
    d = _ledger_from_results(synth.Workload("x", st2, pa2, rq2, 300, 1), res, 100, 40, 70)
    assert np.array_equal(o2.table("credit") - pa2["credit0"], d)
    q = int(np.flatnonzero(res["outcome"][0] == 1)[0])
    assert (res["judges"][0, q] >= 0).sum() == 4
    # queues: executors take the request's tokens, each judge reads both answers (len_in + 2 len_out)
    bl = np.zeros(8, np.int64)
    np.add.at(bl, res["exec_a"][0], 768); np.add.at(bl, res["exec_b"][0], 768)
    np.add.at(bl, res["judges"][0].ravel(), 512 + 2 * 256)
    assert np.array_equal(o2.table("backlog")[0], bl)
    assert np.array_equal(o2.table("served")[0], np.bincount(np.concatenate([res["exec_a"][0], res["exec_b"][0]]), minlength=8))


def test_lemma_1_mean_payoff_of_the_primary_executor():
    """Per delegated request served as primary executor: R, plus with probability p_d
    the duel term Q R_add - (1-Q) P (single judge, no noise, no draws)."""
    N, Q, pd = 12, 150_000, 0.3
    rng = np.random.default_rng(4)
    q = np.concatenate([[0.0], rng.random(N - 1)])
    st, pa, rq = make_net(N, n_requests=Q, seed=23, flags=0, p_duel_ppm=int(pd * 1e6), n_judges=1,
                          peers=requester_first(N, quality_fx=_fx(q), credit0=10 ** 9))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, Q); o.duel_judge(); o.settle_credits(True)
    res = o.results()
    a, b, oc = res["exec_a"][0], res["exec_b"][0], res["outcome"][0]
    R, Ra, P = st.reward_R, st.reward_add, st.penalty_P
    pay = R + np.where(oc == 1, Ra + (P - Ra) - (P - Ra) // 1 * 1, 0) - np.where(oc == 2, P, 0)
    for i in range(1, N):
        m = a == i
        qbar_wo = (q[1:].sum() - q[i]) / (N - 2)
        Qi = 0.5 * (1 + q[i] - qbar_wo)
        delta = R + pd * (Qi * Ra - (1 - Qi) * P)
        sd = pay[m].std() / math.sqrt(m.sum())
        assert abs(pay[m].mean() - delta) < 5 * sd + 1e-9, i
    # the ledger agrees with those per-request payoffs once challenger and judge income is added
    d = o.table("credit")[0] - pa["credit0"][0]
    as_b = oc != 0
    inc = np.bincount(a, weights=pay, minlength=N)
    inc += np.bincount(b[as_b], weights=(R + np.where(oc == 2, Ra, 0) - np.where(oc == 1, P, 0))[as_b], minlength=N)
    inc += np.bincount(res["judges"][0, as_b, 0], weights=np.full(as_b.sum(), P - Ra), minlength=N)
    inc[0] -= R * (len(a) + as_b.sum())
    assert np.array_equal(d, inc.astype(np.int64))


def test_theorem_1_better_group_gains_stake_share():
    N = 32
    q = np.concatenate([np.full(N // 2, 0.8), np.full(N // 2, 0.3)])
    Q = 40_000
    rng = np.random.default_rng(0)
    st, pa, rq = make_net(N, n_requests=Q, seed=31, flags=0, p_duel_ppm=500_000, n_judges=3,
                          peers={"quality_fx": _fx(q)}, origin=rng.integers(0, N, Q))
    o = Oracle(st, pa); o.bind_requests(rq)
    shares = []
    for s in range(Q // 400):
        o.run_step(s * 400, 400, 0, False)
        stake = o.table("stake")[0].astype(float)
        shares.append(stake[: N // 2].sum() / stake.sum())
    assert shares[0] >= 0.5 - 0.01
    assert shares[-1] > shares[0] + 0.03
    quarters = [np.mean(shares[i * 25:(i + 1) * 25]) for i in range(4)]
    assert quarters == sorted(quarters)
    wins = o.table("wins")[0] / np.maximum(o.table("duels")[0], 1)
    assert wins[: N // 2].min() > wins[N // 2:].max()


def test_advance_time_and_latency_hand_cases():
    """Hand cases of the queue model (a reading: the paper gives no formula)."""
    st, pa, rq = make_net(3, n_requests=4, origin=np.array([1, 1, 0, 0]), lens=(600, 400), p_duel_ppm=0,
                          peers={"offload_ppm": np.array([1_000_000, 0, 0]), "cap_true_tok_s": np.array([1000, 2000, 4000])})
    o = Oracle(st, pa); o.bind_requests(rq)
    o.poke_peer(0, 1, backlog=5000)
    o.advance_time(1500)                       # peer 1 drains 2000 * 1.5 = 3000 tokens
    assert o.table("backlog")[0, 1] == 2000
    o.advance_time(1501)                       # 2000 * 1 / 1000 = 2 tokens
    assert o.table("backlog")[0, 1] == 1998
    o.advance_time(60_000)
    assert o.table("backlog")[0, 1] == 0
    o.poke_peer(0, 1, backlog=3000)
    o.poke_peer(0, 2, backlog=1001)
    o.dispatch_batch(0, 4); o.duel_judge(); o.settle_credits(True)
    res = o.results()["exec_a"][0]
    assert list(res[:2]) == [-1, -1] and np.all(res[2:] >= 1)
    sd = o.stats_dict()
    # local at peer 1: ceil((3000 + 1000) * 1000 / 2000) = 2000 ms each (batch-start queue for both)
    lat = 2 * 2000
    for ex in res[2:]:
        lat += {1: 2000, 2: math.ceil((1001 + 1000) * 1000 / 4000)}[int(ex)]
    assert sd["sum_latency_ms"] == lat
    # deadline 2 * ceil(1000 * 1000 / 2000) = 1000 ms: only requests served by peer 2 (501 ms) meet it
    assert sd["slo_met"] == int((res[2:] == 2).sum())
    assert o.table("backlog")[0, 1] == 3000 + 1000 * (2 + int((res[2:] == 1).sum()))
    # the drain runs at the effective (halved) rate while a priority window is active
    st3, pa3, _ = make_net(2, peers={"prio_flag": 1}, p_prio_active_ppm=1_000_000)
    o3 = Oracle(st3, pa3)
    assert np.all(o3.table("cap_eff") == 1000)
    o3.poke_peer(0, 0, backlog=5000)
    o3.advance_time(1500)
    assert o3.table("backlog")[0, 0] == 3500
    # priority window halves capacity while active
    st2, pa2, _ = make_net(400, peers={"prio_flag": 1}, p_prio_active_ppm=500_000, seed=3)
    o2 = Oracle(st2, pa2)
    halves = []
    for w in range(4):
        o2.advance_time(w * 60_000 + 5)
        cap = o2.table("cap_eff")[0]
        assert set(np.unique(cap)) <= {1000, 2000}
        halves.append((cap == 1000).mean())
        o2.advance_time(w * 60_000 + 59_999)
        assert np.array_equal(o2.table("cap_eff")[0], cap)      # constant inside a window
    assert all(abs(h - 0.5) < 5 * math.sqrt(0.25 / 400) for h in halves) and len(set(halves)) > 1


def test_fifo_queueing_inside_a_batch_hand_cases():
    """Flag 16: requests of one batch queue behind each other at their executor (all roles
    count: executions, challenger runs, judge evaluations).  One executor, known sizes."""
    lens = (600, 400)                                       # 1000 tokens per request
    st, pa, rq = make_net(2, n_requests=6, lens=lens, p_duel_ppm=0, flags=16,
                          peers=requester_first(2, cap_true_tok_s=np.array([0, 1000]), credit0=10 ** 6))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.poke_peer(0, 1, backlog=500)
    o.dispatch_batch(0, 4); o.duel_judge(); o.settle_credits(True)
    assert np.all(o.results()["exec_a"][0, :4] == 1)
    # latencies: (500 + k*1000 + 1000) tokens at 1000 tok/s -> 1500, 2500, 3500, 4500 ms
    assert o.stats_dict()["sum_latency_ms"] == 1500 + 2500 + 3500 + 4500
    assert o.stats_dict()["slo_met"] == 0                   # deadline 2 * 500 ms
    assert o.table("backlog")[0, 1] == 4500
    # next batch starts from the folded queue
    o.dispatch_batch(4, 2); o.duel_judge(); o.settle_credits(True)
    assert o.stats_dict()["sum_latency_ms"] == 12000 + 5500 + 6500
    # without the flag every request of a batch sees only the batch-start queue
    st.flags = 0
    o2 = Oracle(st, pa); o2.bind_requests(rq)
    o2.poke_peer(0, 1, backlog=500)
    o2.dispatch_batch(0, 4); o2.duel_judge(); o2.settle_credits(True)
    assert o2.stats_dict()["sum_latency_ms"] == 4 * 1500
    # challenger and judge work queues too: N = 5, every request a duel with 2 judges
    st3, pa3, rq3 = make_net(5, n_requests=40, lens=lens, p_duel_ppm=1_000_000, n_judges=2, flags=16, seed=3,
                             peers=requester_first(5, credit0=10 ** 6))
    o3 = Oracle(st3, pa3); o3.bind_requests(rq3)
    o3.dispatch_batch(0, 40); o3.duel_judge(); o3.settle_credits(True)
    res = o3.results()
    queued = np.zeros(5, np.int64); total = 0
    for q in range(40):
        a, b = res["exec_a"][0, q], res["exec_b"][0, q]
        total += -(-(queued[a] + 1000) * 1000 // 2000)      # ceil((ahead + work) * 1000 / cap)
        queued[a] += 1000; queued[b] += 1000
        for j in res["judges"][0, q]:
            if j >= 0:
                queued[j] += 600 + 2 * 400
    assert o3.stats_dict()["sum_latency_ms"] == total
    assert np.array_equal(o3.table("backlog")[0], queued)


def test_in_block_validation_counts_uncovered_payments():
    """Flag 16: a payment is covered by the finalized balance minus what the payer already spent
    in the open block (this batch and earlier batches); earnings of the open block do not count."""
    # origin has 350 credits, R = 100: payments 1-3 are covered, 4-6 are not
    st, pa, rq = make_net(2, n_requests=12, p_duel_ppm=0, flags=16,
                          peers=requester_first(2, credit0=np.array([350, 10 ** 6])))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.dispatch_batch(0, 6); o.duel_judge(); o.settle_credits(False)
    assert o.stats_dict()["n_delegated"] == 6 and o.stats_dict()["n_uncovered"] == 3
    # same block, next batch: the finalized balance is still 350 and 600 are already spent
    o.dispatch_batch(6, 2); o.duel_judge(); o.settle_credits(True)
    assert o.stats_dict()["n_uncovered"] == 5
    # after the block is finalized the balance is 350 - 800 < R: the origin cannot delegate at all
    o.dispatch_batch(8, 2); o.duel_judge(); o.settle_credits(True)
    assert o.stats_dict()["n_delegated"] == 8 and o.stats_dict()["n_uncovered"] == 5
    # a duel costs the origin 2R; earnings inside the block are not spendable
    st2, pa2, rq2 = make_net(4, n_requests=4, p_duel_ppm=1_000_000, n_judges=1, flags=16,
                             peers=requester_first(4, credit0=np.array([350, 10 ** 6, 10 ** 6, 10 ** 6])))
    o2 = Oracle(st2, pa2); o2.bind_requests(rq2)
    o2.dispatch_batch(0, 4); o2.duel_judge(); o2.settle_credits(True)
    assert np.all(np.isin(o2.results()["outcome"][0], (1, 2)))
    assert o2.stats_dict()["n_uncovered"] == 3              # 200 covered, then 150 left < 200 three times
    # finalization closes the block: what was spent in it no longer counts against the new balance
    st4, pa4, rq4 = make_net(2, n_requests=9, p_duel_ppm=0, flags=16,
                             peers=requester_first(2, credit0=np.array([1000, 10 ** 6])))
    o4 = Oracle(st4, pa4); o4.bind_requests(rq4)
    o4.dispatch_batch(0, 6); o4.duel_judge(); o4.settle_credits(True)      # 600 spent, all covered, balance 400
    o4.dispatch_batch(6, 3); o4.duel_judge(); o4.settle_credits(True)      # 300 more: covered by the 400
    assert o4.stats_dict()["n_delegated"] == 9 and o4.stats_dict()["n_uncovered"] == 0
    # without the flag nothing is counted
    st.flags = 0
    o3 = Oracle(st, pa); o3.bind_requests(rq)
    o3.dispatch_batch(0, 6); o3.duel_judge(); o3.settle_credits(True)
    assert o3.stats_dict()["n_uncovered"] == 0


def test_judges_are_peers_that_are_truly_online():
    """J2: a drawn candidate serves as a judge only if it is online now, whatever the origin's view
    still believes; executor and challenger must be online too (the probe reaches the real peer)."""
    N = 10
    st, pa, rq = make_net(N, n_requests=600, seed=4, p_duel_ppm=1_000_000, n_judges=3, max_probes=8,
                          peers=requester_first(N, credit0=10 ** 7))
    o = Oracle(st, pa); o.bind_requests(rq)
    gone = (3, 6, 7)
    for j in gone:
        o.poke_peer(0, j, online=0)                      # crashed since the last gossip round: the views do not know yet
    assert np.all(np.array([(int(o.view()[0, 0, j]) >> 39) & 1 for j in gone]) == 0)
    o.dispatch_batch(0, 600); o.duel_judge(); o.settle_credits(True)
    res = o.results()
    decided = np.isin(res["outcome"][0], (1, 2, 3))
    assert decided.sum() > 300
    jd = res["judges"][0][decided]
    assert not np.isin(jd, gone).any() and not np.isin(res["exec_a"][0], gone).any() and not np.isin(res["exec_b"][0], gone).any()
    assert np.all((jd >= 0).sum(axis=1) == 3)            # six peers remain online besides A and B: always three judges
    # every online peer other than the requester does serve as a judge at some point
    assert set(np.unique(jd[jd >= 0])) == set(range(1, N)) - set(gone)


def test_hop_latency_is_added_to_delegated_requests_only():
    """S4: a delegated request pays the network hop once, a locally served one does not."""
    def total_latency(hop):
        st, pa, rq = make_net(3, n_requests=40, origin=np.array([1, 0] * 20), lens=(600, 400), p_duel_ppm=0, hop_ms=hop,
                              peers={"offload_ppm": np.array([1_000_000, 0, 0]), "cap_true_tok_s": np.array([1000, 2000, 4000])})
        o = Oracle(st, pa); o.bind_requests(rq)
        o.dispatch_batch(0, 40); o.duel_judge(); o.settle_credits(True)
        ex = o.results()["exec_a"][0]
        return o.stats_dict()["sum_latency_ms"], int((ex >= 0).sum()), int((ex == -1).sum()), o.stats_dict()["slo_met"]
    lat0, deleg0, local0, met0 = total_latency(0)
    lat7, deleg7, local7, met7 = total_latency(37)
    assert (deleg0, local0) == (deleg7, local7) == (20, 20)
    assert lat7 - lat0 == 37 * deleg0
    # with a hop longer than any deadline no delegated request meets it, the local ones are unaffected
    _, _, _, met_far = total_latency(10_000)
    assert met0 > met_far and met_far <= local0
