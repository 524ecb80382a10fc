"""Pins for the oracle's randomness and its gossip round.

Randomness: the published known-answer vectors of Philox4x32-10.
Gossip (Appendix "Gossip-Driven Peer Synchronization"): entries only get newer,
never run ahead of their owner, move one hop per round, converge without a
coordinator, departures are detected and joins are integrated.
"""
import math
import os

import numpy as np
import pytest

from oracle import Oracle, binding
from tests.helpers import OFFBIT, entry_offline, entry_ver, make_net

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        v = [int(x, 16) for x in row]
        out = binding.philox4x32_10(v[0:4], v[4:6])
        assert [int(x) for x in out] == v[6:10]


def test_range_reductions_exact_and_uniform():
    L = binding.lib()
    for x in (0, 1, 4294, 4295, 2 ** 31, 2 ** 32 - 1):
        assert L.orc_ppm(x) == (x * 1_000_000) >> 32
        for n in (1, 7, 32, 16384):
            assert L.orc_below(x, n) == (x * n) >> 32
    assert L.orc_ppm(2 ** 32 - 1) == 999_999
    for x, s in ((2 ** 64 - 1, 2 ** 61), (12345678901234567, 987654321987), (0, 5), (2 ** 63, 3)):
        assert L.orc_mulhi64(x, s) == (x * s) >> 64
    # uniformity of below(philox, 10) over 20000 counters
    cnt = np.zeros(10)
    for i in range(5000):
        for w in binding.philox4x32_10([i, 0, 0, 5], [7, 0]):
            cnt[L.orc_below(int(w), 10)] += 1
    chi = ((cnt - 2000.0) ** 2 / 2000.0).sum()
    assert chi < 9 + 5 * math.sqrt(18)


def test_merge_is_a_semilattice_join():
    L = binding.lib()
    rng = np.random.default_rng(1)
    v = [int(x) for x in rng.integers(0, 2 ** 63, 30, dtype=np.uint64)]
    for a in v[:10]:
        assert L.orc_merge(a, a) == a
        for b in v[10:20]:
            assert L.orc_merge(a, b) == L.orc_merge(b, a)
            for c in v[20:25]:
                assert L.orc_merge(L.orc_merge(a, b), c) == L.orc_merge(a, L.orc_merge(b, c))
    # newer version wins whatever the payload; at equal version the offline mark wins
    old = (5 << 40) | (1 << 39) | 12345
    new = (6 << 40) | 1
    assert L.orc_merge(old, new) == new
    assert L.orc_merge((6 << 40) | 77, (6 << 40) | 77 | OFFBIT) == (6 << 40) | 77 | OFFBIT


def _net(N, k, **kw):
    st, pa, _ = make_net(N, fanout_k=k, **kw)
    return Oracle(st, pa)


@pytest.mark.parametrize("N,k", [(16, 2), (64, 2), (100, 3)])
def test_gossip_monotone_bounded_staleness(N, k):
    o = _net(N, k, init_stale_max=5, seed=3)
    prev = o.view()
    bound = 2 * math.log2(N) + 8
    for t in range(int(bound) + 12):
        o.gossip_round()
        v = o.view()
        ver_true = o.table("ver")[0]
        assert np.all(v >= prev), "an entry went back in time"
        assert np.all(entry_ver(v[0]) <= ver_true[None, :].astype(np.uint64)), "entry newer than its owner"
        assert np.all(entry_ver(np.diagonal(v[0])) == ver_true.astype(np.uint64)), "own entry not current"
        prev = v
        if t >= bound:
            stale = ver_true[None, :].astype(np.int64) - entry_ver(v[0]).astype(np.int64)
            assert stale.max() <= bound, "updates did not diffuse in O(log N) rounds"
    assert o.error() == 0


def test_gossip_synchronous_one_hop_per_round():
    """Every new entry is an old entry of the same column (own or a partner's),
    a fresh self entry, or a hello; a fresh version is known to at most 1+k nodes
    after the round that issued it (partners read the OLD buffer)."""
    N, k = 48, 3
    o = _net(N, k, seed=11)
    for t in range(6):
        old = o.view()[0]
        o.gossip_round()
        new = o.view()[0]
        ver_true = o.table("ver")[0].astype(np.uint64)
        for c in range(N):
            fresh = entry_ver(new[:, c]) == ver_true[c]
            assert 1 <= fresh.sum() <= 1 + k
            ok = np.isin(new[~fresh, c], old[:, c])
            assert ok.all(), "entry that is neither old nor fresh"
        # a row gains at most what k partner rows and its own old row hold
        for i in range(0, N, 7):
            src = [p for p in range(N) if p != i and np.all(new[i][np.arange(N) != i] >= old[p][np.arange(N) != i])]
            assert len(src) >= 1  # at least one partner row is dominated (k>=1, all online, all known)


def test_gossip_detects_departure_and_stops_pulling_it():
    N, k = 64, 2
    o = _net(N, k, seed=5)
    for _ in range(3):
        o.gossip_round()
    dead = 17
    o.poke_peer(0, dead, online=0)
    ver_dead = int(o.table("ver")[0, dead])
    rounds = 0
    while True:
        o.gossip_round()
        rounds += 1
        v = o.view()[0]
        col = np.delete(v[:, dead], dead)
        if np.all(entry_offline(col) == 1):
            break
        assert rounds < 2 * math.log2(N) + 20, "departure not detected"
    assert int(o.table("ver")[0, dead]) == ver_dead, "an offline peer must not issue versions"
    marks = o.stats_dict()["n_offline_marks"]
    assert marks >= 1
    # once everybody believes it offline nobody pulls from it any more
    for _ in range(5):
        o.gossip_round()
    assert o.stats_dict()["n_offline_marks"] == marks
    # the dead peer's own row is frozen
    row = o.view()[0, dead].copy()
    o.gossip_round()
    assert np.array_equal(o.view()[0, dead], row)


def test_gossip_integrates_a_joining_peer():
    """A peer everybody believes offline can only be discovered through its own
    pulls (the hello entry); afterwards the news spreads by ordinary pulls."""
    N, k = 64, 2
    online0 = np.ones(N, np.uint8); online0[9] = 0
    st, pa, _ = make_net(N, fanout_k=k, seed=2, peers={"online0": online0}, p_join_ppm=1_000_000)
    o = Oracle(st, pa)
    v0 = o.view()[0]
    assert np.all(entry_offline(v0[:, 9]) == 1)
    rounds = 0
    while True:
        o.gossip_round()
        rounds += 1
        v = o.view()[0]
        if np.all(entry_offline(v[:, 9]) == 0):
            break
        assert rounds < 2 * math.log2(N) + 20, "join not integrated"
    assert o.table("online")[0, 9] == 1
    # after the first round exactly the joiner and its k partners know
    o2 = Oracle(st, pa)
    o2.gossip_round()
    knows = (entry_offline(o2.view()[0][:, 9]) == 0).sum()
    assert 2 <= knows <= 1 + k


def test_gossip_churn_statistics_and_queue_loss():
    N = 2000
    st, pa, _ = make_net(N, fanout_k=1, seed=9, p_leave_ppm=100_000, p_join_ppm=300_000)
    o = Oracle(st, pa)
    for j in range(N):
        o.poke_peer(0, j, backlog=1000)
    o.gossip_round()
    on = o.table("online")[0]
    left = (on == 0).sum()
    assert abs(left - 200) < 5 * math.sqrt(N * 0.1 * 0.9)
    assert np.all(o.table("backlog")[0][on == 0] == 0) and np.all(o.table("backlog")[0][on == 1] == 1000)
    o.gossip_round()
    on2 = o.table("online")[0]
    rejoined = ((on == 0) & (on2 == 1)).sum()
    assert abs(rejoined - left * 0.3) < 5 * math.sqrt(left * 0.3 * 0.7)


def test_gossip_version_overflow_is_reported():
    st, pa, _ = make_net(4, fanout_k=1, init_stale_max=0)
    st.init_stale_max = (1 << 24) - 3    # ver starts two below the limit
    o = Oracle(st, pa)
    o.gossip_round()
    assert o.error() == 0
    o.gossip_round()
    assert o.error() == 4


def test_push_pull_exchange_is_symmetric_and_faster():
    """Flag 8: both ends of an exchange reconcile (the appendix figure shows two nodes swapping
    views).  After a round each end dominates the other's old row; versions stay honest and
    monotone; updates spread in fewer rounds than with pulls alone."""
    N, k = 96, 1
    rounds = {}
    for flags in (0, 8):
        st, pa, _ = make_net(N, fanout_k=k, seed=4, flags=flags, init_stale_max=7)
        o = Oracle(st, pa)
        t_conv = None
        for t in range(40):
            old = o.view()[0]
            o.gossip_round()
            new = o.view()[0]
            ver_true = o.table("ver")[0].astype(np.uint64)
            assert np.all(new >= old) and np.all(entry_ver(new) <= ver_true[None, :])
            # one hop per round in both modes: the version a node issued this round is known to itself
            # and to the (at most k) partners it greeted; a pushed row is the OLD row of the pusher
            fresh = (entry_ver(new) == ver_true[None, :]).sum(axis=0)
            assert np.all(fresh >= 1) and np.all(fresh <= 1 + k)
            if flags == 8:
                # somebody's old row is dominated by row i: its partner's; and row i's old content
                # reached that partner: new[p] >= old[i] for at least one p != i
                off = ~np.eye(N, dtype=bool)
                for i in range(0, N, 11):
                    dom_pull = [p for p in range(N) if p != i and np.all((new[i] >= old[p])[off[i]])]
                    dom_push = [p for p in dom_pull if np.all((new[p] >= old[i])[off[p]])]
                    assert dom_pull and dom_push, i
            stale = (ver_true[None, :].astype(np.int64) - entry_ver(new).astype(np.int64)).max()
            if t_conv is None and t >= 8 and stale <= 2 * math.log2(N):
                t_conv = t
        rounds[flags] = (t_conv, stale)
    assert rounds[8][1] < rounds[0][1], rounds       # steady-state staleness is lower with push-pull


def test_partner_choice_is_uniform_and_slots_are_independent():
    """After the first round of a fresh network, node p knows the new version of node i exactly when
    i pulled p (the hello; pulled rows are old ones), so the view shows who pulled whom.  Every slot
    picks uniformly among the other N - 1 peers, independently of the other slots:
    P(i pulls p) = 1 - (1 - 1/(N-1))^k for every ordered pair, and the number of distinct partners
    of a node has the occupancy distribution of k balls in N - 1 boxes."""
    from tests.helpers import chi2_ok
    N, k, Rp = 9, 3, 600
    st, pa, _ = make_net(N, n_replicas=Rp, fanout_k=k, gossip_tries=8, seed=11)
    o = Oracle(st, pa)
    v0 = int(entry_ver(o.view()[0, 0, 0]))
    o.gossip_round()
    pulled = entry_ver(o.view()) == v0 + 1                       # [replica, p, i]: p knows i's new entry
    idx = np.arange(N)
    assert pulled[:, idx, idx].all()
    pulled[:, idx, idx] = False
    pairs = pulled.sum(0)[~np.eye(N, dtype=bool)]                # 72 ordered pairs, each Binomial(Rp, P)
    P = 1 - (1 - 1 / (N - 1)) ** k
    stat = float(((pairs - Rp * P) ** 2 / (Rp * P * (1 - P))).sum())
    assert stat < 72 + 5 * np.sqrt(2 * 72), stat
    # distinct partners per node: 1, 2 or 3 of 8 boxes
    distinct = pulled.sum(1).ravel()                             # per (replica, i): how many p it pulled
    m = N - 1
    exp = np.array([m * 1, m * (m - 1) * 3, m * (m - 1) * (m - 2)], float) / m ** 3
    ok, s2, _ = chi2_ok(np.bincount(distinct, minlength=4)[1:], distinct.size * exp)
    assert ok, s2


def test_own_entry_advertises_capacity_and_queue_in_16_token_units():
    """G1: an online peer's fresh entry carries its version, its advertised capacity (true rate x
    misreport factor, saturating at 2^19 - 1) and its queue in 16-token units (saturating at
    2^20 - 1); the views of the peers that pull it take the same entry."""
    from tests.helpers import entry_cap, entry_q
    N = 12
    cap = np.arange(N) * 700 + 100
    st, pa, _ = make_net(N, fanout_k=3, seed=2, peers={"cap_true_tok_s": cap, "misreport_mul": np.where(np.arange(N) % 4 == 0, 4, 1)})
    o = Oracle(st, pa)
    queues = {1: 15, 2: 16, 3: 1000, 4: 123_457, 5: (1 << 24) + 5, 6: 1 << 40}
    for j, b in queues.items():
        o.poke_peer(0, j, backlog=b)
    o.gossip_round()
    v = o.view()[0]
    ver = o.table("ver")[0]
    for j in range(N):
        own = v[j, j]
        assert int(entry_ver(own)) == ver[j] and int(entry_offline(own)) == 0
        assert int(entry_cap(own)) == min((1 << 19) - 1, int(cap[j]) * (4 if j % 4 == 0 else 1))
        assert int(entry_q(own)) == min((1 << 20) - 1, queues.get(j, 0) >> 4)
    # whoever holds the current version of j holds exactly that entry
    for i in range(N):
        for j in range(N):
            if int(entry_ver(v[i, j])) == ver[j]:
                assert (int(v[i, j]) | OFFBIT) == (int(v[j, j]) | OFFBIT)
