"""Full-size parity in the benchmark's launch configuration.

All five configurations are run at their full sizes through `wwws_step` (the call the
benchmark times).  Replicas are independent and keyed by their global index, so one replica
of the full run can be checked completely against the oracle run on that replica alone:
every result record, every per-peer table, the counters, and sampled rows of its view matrix.
"""
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
