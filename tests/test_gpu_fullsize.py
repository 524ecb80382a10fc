"""Full-size parity in the benchmark's launch configuration.

All five configurations are run at their full sizes through `wwws_step` (the call the
benchmark times).  Replicas are independent and keyed by their global index, so one replica
of the full run can be checked completely against the oracle run on that replica alone:
every result record, every per-peer table, the counters, and sampled rows of its view matrix.
"""
import os

import numpy as np
import pytest

from oracle import Oracle
from paper_2603_20661_b200 import synth
from tests.helpers import TABLE_NAMES

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,replica,steps", [("tiny", 0, 20), ("tiers64", 0, 200), ("zipf1k", 200, 8), ("churn4k", 37, 12),
                                                ("adversarial16k", 5, 12)])
def test_one_replica_of_the_full_run_matches_the_oracle(name, replica, steps):
    from paper_2603_20661_b200.binding import Network
    wl = synth.make_workload(name)
    st = wl.settings
    g = Network(st, wl.peers, wl.batch)
    g.bind_requests(wl.requests, scores=False)
    one = synth.slice_replicas(wl, replica, replica + 1)
    o = Oracle(one.settings, one.peers)
    o.bind_requests(one.requests)
    for s in range(steps):
        args = (s * wl.batch, wl.batch, wl.step_now_ms(s), s % wl.gossip_every == 0)
        g.step(*args)
        o.run_step(*args)
    upto = steps * wl.batch
    rg, ro = g.results(), o.results()
    for k in ("exec_a", "exec_b", "judges", "outcome", "flags"):
        assert np.array_equal(rg[k][replica, :upto], ro[k][0, :upto]), f"{name}: {k} differs"
    for t in TABLE_NAMES:
        assert np.array_equal(g.table(t)[replica].astype(np.int64), o.table(t)[0]), f"{name}: table {t} differs"
    assert np.array_equal(g.stats()[replica], o.stats()[0]), f"{name}: counters differ"
    ov = o.view()[0]
    N = st.n_peers
    rows = sorted(set([0, 1, min(31, N - 1), min(32, N - 1), N // 2, max(N - 33, 0), N - 1]
                      + list(np.random.default_rng(1).integers(0, N, 40))))
    for i in rows:
        assert np.array_equal(g.view_rows(replica, int(i), 1)[0], ov[i]), f"{name}: view row {i} differs"
    # properties that hold at any size, over all replicas
    sd = g.stats()
    assert np.all(sd[:-1, 0] == upto)
    assert np.array_equal(sd[:-1, 17].astype(np.int64), wl.peers["credit0"].sum(axis=1))
    ex = rg["exec_a"][:, :upto]
    assert ex.max() < N and ex.min() >= -4
    assert np.all(ex != wl.requests["origin"][:, :upto].astype(np.int64))          # never delegated to oneself
    dec = np.isin(rg["outcome"][:, :upto], (1, 2, 3))
    assert np.all(rg["exec_b"][:, :upto][dec] >= 0) and np.all(rg["exec_b"][:, :upto][~dec] == -1)
    assert o.error() == 0
    g.close()


@pytest.mark.parametrize("name,batch,replica", [("zipf1k", 10000, 131), ("adversarial16k", 100000, 9)])
def test_one_replica_of_the_saturated_launch_matches_the_oracle(name, batch, replica):
    """The benchmark's saturated leg: a replica's whole request stream in one step (2.56 M and 1.6 M
    requests per launch; every warp of the streaming kernel runs through hundreds of requests).
    One replica is checked completely against the oracle run on that replica alone."""
    from paper_2603_20661_b200.binding import Network
    wl = synth.make_workload(name)
    wl.batch = batch
    g = Network(wl.settings, wl.peers, wl.batch)
    g.bind_requests(wl.requests, scores=False)
    one = synth.slice_replicas(wl, replica, replica + 1)
    one.batch = batch
    o = Oracle(one.settings, one.peers)
    o.bind_requests(one.requests)
    steps = min(2, wl.n_steps)
    for s in range(steps):
        args = (s * batch, batch, wl.step_now_ms(s), s == 0)
        g.step(*args)
        o.run_step(*args)
    upto = steps * batch
    rg, ro = g.results(), o.results()
    for k in ("exec_a", "exec_b", "judges", "outcome", "flags"):
        assert np.array_equal(rg[k][replica, :upto], ro[k][0, :upto]), f"{name}: {k} differs"
    for t in TABLE_NAMES:
        assert np.array_equal(g.table(t)[replica].astype(np.int64), o.table(t)[0]), f"{name}: table {t} differs"
    assert np.array_equal(g.stats()[replica], o.stats()[0]), f"{name}: counters differ"
    sd = g.stats()
    assert np.all(sd[:-1, 0] == upto)
    assert np.array_equal(sd[:-1, 17].astype(np.int64), wl.peers["credit0"].sum(axis=1))
    g.close()


@pytest.mark.skipif(os.environ.get("WWWS_MAX_SIZE") != "1",
                    reason="the oracle needs over a minute and about 100 GB of host memory at 65,535 peers: set WWWS_MAX_SIZE=1")
@pytest.mark.parametrize("n_peers", [32768, 65535])
def test_largest_networks_match_the_oracle(n_peers):
    """The maximum peer count (65,535: the narrowest view panels, a ragged last candidate block,
    34 GB per view buffer) and half of it, one replica, two gossip rounds with churn and three
    batches: tables, results, counters and the whole view matrix."""
    from paper_2603_20661_b200.binding import Network
    from tests.helpers import assert_same_state
    wl = synth.make_workload("adversarial16k", n_replicas=1, n_requests=3000, n_peers=n_peers)
    wl.settings.p_leave_ppm = wl.settings.p_join_ppm = 50_000
    g = Network(wl.settings, wl.peers, wl.batch); g.bind_requests(wl.requests)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    for s in range(3):
        g.step(s * wl.batch, wl.batch, wl.step_now_ms(s), s < 2)
        o.run_step(s * wl.batch, wl.batch, wl.step_now_ms(s), s < 2)
    assert_same_state(g, o, f"{n_peers} peers", upto=3 * wl.batch, views=False)
    ov = o.view()[0]
    for r0 in range(0, n_peers, 4096):                        # block by block: never two full copies at once
        a = g.view_rows(0, r0, min(4096, n_peers - r0))
        assert np.array_equal(a, ov[r0:r0 + a.shape[0]]), f"view rows from {r0} differ"
    g.close()
