"""Pins for the oracle's initial state: what every node knows about every peer at time 0.

Reading taken (the paper describes no bootstrap; its networks are a handful of nodes that all
know each other): a node starts with an entry for every peer, its own entry current and the
others 0..init_stale_max versions old, uniformly ("stale gossip views up to 5 rounds old").
The checks below do not go through the oracle's own arithmetic: the staleness is recomputed from
a Philox4x32-10 written here (itself checked against the published known answers), the law is
tested by chi-square, and the entry fields are compared with the inputs.
"""
import os

import numpy as np
import pytest

from oracle import Oracle
from tests.helpers import chi2_ok, entry_cap, entry_offline, entry_q, entry_ver, make_net

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
M32 = 0xFFFFFFFF
ST_INIT = 8


def philox_py(ctr, key):
    """Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC'11), plain Python integers."""
    c0, c1, c2, c3 = ctr
    k0, k1 = key
    for _ in range(10):
        p0, p1 = 0xD2511F53 * c0, 0xCD9E8D57 * c2
        c0, c1, c2, c3 = ((p1 >> 32) ^ c1 ^ k0) & M32, p1 & M32, ((p0 >> 32) ^ c3 ^ k1) & M32, p0 & M32
        k0, k1 = (k0 + 0x9E3779B9) & M32, (k1 + 0xBB67AE85) & M32
    return c0, c1, c2, c3


def test_python_philox_matches_published_vectors():
    rows = [ln.split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    for row in rows:
        v = [int(x, 16) for x in row]
        assert list(philox_py(v[0:4], v[4:6])) == v[6:10]


def _network(N, Rp, stale_max, seed, offset=0):
    rng = np.random.default_rng(seed + 11)
    cap = rng.integers(1, 300_000, (Rp, N))
    cap[:, 3] = 0                                     # a requester-only node advertises no capacity
    mis = np.where(rng.random((Rp, N)) < 0.3, 4, 1)
    on = (rng.random((Rp, N)) < 0.8).astype(np.uint8)
    st, pa, _ = make_net(N, Rp, seed=seed, init_stale_max=stale_max, replica_offset=offset,
                         peers={"cap_true_tok_s": cap, "misreport_mul": mis, "online0": on})
    return st, pa, Oracle(st, pa)


def test_initial_staleness_is_the_init_draw_scaled_to_the_range():
    """V[i][j].version = ver[j] - ((w0 * (init_stale_max + 1)) >> 32), w0 the first word of the
    generator at counter (i, j, global replica, INIT); the diagonal is current."""
    N, Rp, smax, seed, off = 40, 3, 5, 0x1234567_89ABCDEF, 7
    st, pa, o = _network(N, Rp, smax, seed, off)
    v, ver = o.view(), o.table("ver")
    assert np.all(ver == smax + 1)
    key = (seed & M32, seed >> 32)
    rng = np.random.default_rng(5)
    triples = [(int(rng.integers(Rp)), int(rng.integers(N)), int(rng.integers(N))) for _ in range(200)]
    triples += [(0, 0, 1), (Rp - 1, N - 1, 0), (1, 17, 17)]
    for r, i, j in triples:
        w0 = philox_py((i, j, r + off, ST_INIT), key)[0]
        stale = 0 if i == j else (w0 * (smax + 1)) >> 32
        assert int(entry_ver(v[r, i, j])) == smax + 1 - stale, (r, i, j)
    o.close()


def test_initial_staleness_is_uniform_and_diagonal_current():
    N, smax = 200, 5
    st, pa, o = _network(N, 1, smax, 3)
    v = o.view()[0]
    stale = (smax + 1) - entry_ver(v).astype(np.int64)
    assert np.all(np.diagonal(stale) == 0)
    off_diag = stale[~np.eye(N, dtype=bool)]
    assert off_diag.min() == 0 and off_diag.max() == smax          # the whole range 0..init_stale_max, nothing beyond
    cnt = np.bincount(off_diag, minlength=smax + 1)
    ok, stat, df = chi2_ok(cnt, np.full(smax + 1, off_diag.size / (smax + 1)))
    assert ok, (stat, df, cnt)
    # rows are drawn independently: no two observers share the same pattern
    assert len({stale[i].tobytes() for i in range(N)}) == N
    # (i, j) and (j, i) use different counters
    assert np.mean(stale == stale.T) < 0.3
    o.close()


@pytest.mark.parametrize("smax", [0, 1, 7])
def test_staleness_range_follows_the_setting(smax):
    st, pa, o = _network(64, 1, smax, 9)
    stale = (smax + 1) - entry_ver(o.view()[0]).astype(np.int64)
    assert stale.min() == 0 and stale.max() == smax
    o.close()


def test_initial_entry_fields_come_from_the_peer_inputs():
    """offline bit = not online at time 0; advertised capacity = true capacity x misreport factor,
    saturating at 2^19 - 1; advertised queue 0; every column of a row carries its subject's data."""
    N, Rp = 48, 2
    st, pa, o = _network(N, Rp, 4, 21)
    v = o.view()
    for r in range(Rp):
        want_cap = np.minimum(pa["cap_true_tok_s"][r].astype(np.int64) * pa["misreport_mul"][r], (1 << 19) - 1)
        assert want_cap.max() == (1 << 19) - 1 and want_cap.min() == 0       # both ends of the field are exercised
        for i in (0, 5, N - 1):
            assert np.array_equal(entry_cap(v[r, i]).astype(np.int64), want_cap)
            assert np.array_equal(entry_offline(v[r, i]).astype(np.uint8), 1 - pa["online0"][r])
            assert np.all(entry_q(v[r, i]) == 0)
    assert np.all(v != 0)                                                     # nobody starts unknown
    o.close()


def test_initial_ledger_is_the_given_credit_with_its_stake():
    rng = np.random.default_rng(2)
    N = 30
    credit0 = rng.integers(-500, 20_000, (1, N))
    stake_pm = rng.integers(0, 1001, (1, N))
    st, pa, _ = make_net(N, 1, peers={"credit0": credit0, "stake_pm": stake_pm})
    o = Oracle(st, pa)
    assert np.array_equal(o.table("credit"), credit0)
    assert np.array_equal(o.table("stake"), np.maximum(credit0, 0) * stake_pm // 1000)
    for t in ("d_credit", "d_wins", "d_duels", "wins", "duels", "backlog", "served"):
        assert not o.table(t).any(), t
    sd = o.stats_dict()
    assert sd["blocks"] == 0 and sd["credit_total"] == int(credit0.sum())
    o.close()


def test_priority_window_is_the_prio_draw_of_peer_and_window():
    """A peer with its own prioritized load serves at half rate in the windows where
    ppm(w0) < p_prio_active, w0 the first word of the generator at counter
    (peer, window number, global replica, PRIO); windows are prio_window_ms long."""
    ST_PRIO = 7
    N, seed, off, p = 60, 77, 3, 400_000
    prio = (np.arange(N) % 3 != 0).astype(np.uint8)                 # every third peer has no such load
    st, pa, _ = make_net(N, 2, seed=seed, replica_offset=off, p_prio_active_ppm=p, prio_window_ms=7000,
                         peers={"prio_flag": prio, "cap_true_tok_s": 2001})
    o = Oracle(st, pa)
    for now in (0, 6999, 7000, 20_999, 21_000, 1_000_000):
        o.advance_time(now)
        cap = o.table("cap_eff")
        w = now // 7000
        for r in range(2):
            for j in range(N):
                w0 = philox_py((j, w, r + off, ST_PRIO), (seed & M32, seed >> 32))[0]
                active = bool(prio[j]) and ((w0 * 1_000_000) >> 32) < p
                assert cap[r, j] == (2001 // 2 if active else 2001), (now, r, j)
    o.close()
