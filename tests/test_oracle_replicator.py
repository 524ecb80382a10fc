"""The oracle's long-run stake shares against the paper's replicator equations.

Section "Theoretical Analysis": with PoS selection p_i = s_i / S (Assumption 3), stakes that
move with realised payoff (Assumption 4) and a pairwise win probability 1/2 (1 + q_i - Qbar),
the share of a group H follows (Proposition 2)

    dp_H/dt = (eta lambda / S) p_H (1 - p_H) (Delta_H - Delta_notH),

and the better group takes over (Theorem 1).  Here time is counted in delegated requests
(eta lambda = 1) and the stake of a provider is its credit.  In the simulated mechanism both
contestants of a duel are PoS draws and each receives the base reward, so per request the
payoff of a node, conditional on being drawn, is

    Delta'_i = R + p_d [ R + 2 (Q_i W - (1 - Q_i) P) + share ],

W = the winner's prize, share = what the judge earns.  Only the Q_i term differs between nodes:
Delta'_H - Delta'_notH = p_d (W + P) (q_H - q_notH), twice the paper's primary-only coefficient.
With one judge and no vote noise the duel outcome has exactly the probability of Assumption 3.
"""
import numpy as np

from oracle import Oracle
from tests.helpers import make_net


def _fx(q):
    return np.minimum(np.round(np.asarray(q, float) * 2.0 ** 32), 2.0 ** 32 - 1).astype(np.uint64).astype(np.uint32)


def _simulate(q, p_duel, Q, B, Rp, R=100, R_add=40, P=70):
    """Mean over replicas of the stake share of the first half of the providers after every block."""
    N = len(q)
    cap = np.full(N, 2000); cap[0] = 0                       # peer 0 only issues requests
    credit = np.full(N, 10_000, np.int64); credit[0] = 10 ** 12
    st, pa, rq = make_net(N, n_replicas=Rp, n_requests=Q, seed=5, flags=0, p_duel_ppm=int(p_duel * 1e6), n_judges=1,
                          reward_R=R, reward_add=R_add, penalty_P=P,
                          peers={"quality_fx": _fx(q), "cap_true_tok_s": cap, "credit0": credit})
    o = Oracle(st, pa); o.bind_requests(rq)
    half = 1 + (N - 1) // 2
    shares, totals = [], []
    for s in range(Q // B):
        o.run_step(s * B, B, 0, False)
        stake = o.table("stake")[:, 1:].astype(float)
        shares.append((stake[:, : half - 1].sum(1) / stake.sum(1)).mean())
        totals.append(stake.sum(1).mean())
    sd = o.stats_dict()
    o.close()
    return np.array(shares), np.array(totals), sd


def _replicator(p0, S0, coeff, inflow, n_blocks, B):
    """Proposition 2 integrated block by block.  Stakes are constant inside a block, so the group's
    stake grows by its share of the inflow plus S dp_H/dt = p_H (1 - p_H) coeff per request."""
    sH, S, out = p0 * S0, S0, []
    for _ in range(n_blocks):
        p = sH / S
        sH += B * (p * inflow + p * (1.0 - p) * coeff)
        S += B * inflow
        out.append(sH / S)
    return np.array(out)


def test_group_share_follows_the_replicator_equation():
    N, B, Q, Rp = 32, 250, 60_000, 24
    q = np.concatenate([[0.5], np.full(15, 0.8), np.full(16, 0.3)])
    p_d, R, W, P = 0.5, 100, 40, 70
    shares, totals, sd = _simulate(q, p_d, Q, B, Rp, R, W, P)
    assert sd["n_delegated"] == Rp * Q and sd["n_duel_cancelled"] == 0
    # total provider stake grows by what the requester pays: R per execution, 1 + p_d executions per request
    inflow = R * (1 + p_d)
    assert abs(totals[-1] - (31 * 10_000 + Q * inflow)) < 0.01 * totals[-1]
    p0 = 15 / 31
    coeff = p_d * (W + P) * (0.8 - 0.3)                      # Delta'_H - Delta'_notH
    model = _replicator(p0, 31 * 10_000.0, coeff, inflow, Q // B, B)
    assert model[-1] - p0 > 0.04                             # the effect is far above the tolerance below
    assert np.max(np.abs(shares - model)) < 0.004
    # the paper's primary-only coefficient (one contestant per duel) predicts half the drift: rejected
    half = _replicator(p0, 31 * 10_000.0, coeff / 2, inflow, Q // B, B)
    assert abs(shares[-1] - half[-1]) > 0.015


def test_equal_quality_groups_keep_their_share():
    N, B, Q, Rp = 32, 250, 20_000, 24
    q = np.concatenate([[0.5], np.full(31, 0.6)])
    shares, _, _ = _simulate(q, 0.5, Q, B, Rp)
    assert np.max(np.abs(shares - 15 / 31)) < 0.004           # Delta_H = Delta_notH: no drift


def test_share_drift_scales_with_the_duel_probability():
    N, B, Q, Rp = 32, 250, 30_000, 24
    q = np.concatenate([[0.5], np.full(15, 0.9), np.full(16, 0.2)])
    gains = []
    for p_d in (0.0, 0.25, 0.5):
        shares, _, _ = _simulate(q, p_d, Q, B, Rp)
        model = _replicator(15 / 31, 31 * 10_000.0, p_d * 110 * 0.7, 100 * (1 + p_d), Q // B, B)
        assert np.max(np.abs(shares - model)) < 0.005
        gains.append(shares[-1] - 15 / 31)
    assert abs(gains[0]) < 0.003 and gains[1] > 0.02 and gains[2] > gains[1] + 0.01
