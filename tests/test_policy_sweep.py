"""User-level policies as a batched sweep (Section "Impact of User-Level Policies": stakes 1:2:3:4,
acceptance and offloading frequencies 0.25 .. 1.0 for nodes 1-4, requests from a requester-only node).

The paper reports that nodes with a higher stake or acceptance frequency take a larger share of the
delegated requests.  In the simulated mechanism those shares have closed forms, which both the oracle
and the CUDA path must reproduce: stake share = stake / total stake when everybody accepts;
with refusals, the probability of each draw order times the refusals before the acceptance."""
import itertools

import numpy as np
import pytest

from oracle import Oracle
from paper_2603_20661_b200 import synth
from tests.helpers import assert_same_state, chi2_ok, run_workload


def _accept_law(acc, probes=3):
    p = np.zeros(6)                                   # 1..4 executors, 5 = nobody willing
    for perm in itertools.permutations([1, 2, 3, 4], probes):
        refused = 1.0
        for node in perm:
            p[node] += refused * acc[node] / 24.0
            refused *= 1 - acc[node]
        p[5] += refused / 24.0
    return p[1:]


def _check_laws(wl, res):
    ex, origin = res["exec_a"], wl.requests["origin"]
    ax = wl.axis
    # stake axis: first draw always accepted, share = stake share
    e = ex[ax == 0].ravel()
    assert e.min() >= 1
    ok, stat, _ = chi2_ok(np.bincount(e, minlength=5)[1:], e.size * np.array([0.1, 0.2, 0.3, 0.4]))
    assert ok, ("stake", stat)
    # acceptance axis: enumeration of draw orders and refusals; the requester has no capacity, so "nobody willing" = -4
    e = ex[ax == 1].ravel()
    obs = np.array([(e == i).sum() for i in (1, 2, 3, 4)] + [(e == -4).sum()])
    assert obs.sum() == e.size
    ok, stat, _ = chi2_ok(obs, e.size * _accept_law(np.array([0, 0.25, 0.5, 0.75, 1.0])))
    assert ok, ("accept", obs, stat)
    assert obs[0] < obs[1] < obs[2] < obs[3]
    # offloading axis: a provider delegates its own users' requests with its offloading frequency
    e, o = ex[ax == 2].ravel(), origin[ax == 2].ravel()
    for node, f in zip((1, 2, 3, 4), (0.25, 0.5, 0.75, 1.0)):
        m = o == node
        n, k = int(m.sum()), int((e[m] >= 0).sum())
        assert abs(k - n * f) <= 5 * np.sqrt(max(n * f * (1 - f), 1.0)), ("offload", node, k, n)
        assert np.all((e[m] >= 0) | (e[m] == -1))     # otherwise served locally by policy


def test_policy_sweep_laws_in_the_oracle():
    wl = synth.make_policy_sweep(replicas_per_axis=6, n_requests=3000)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    run_workload(o, wl)
    _check_laws(wl, o.results())
    assert o.stats_dict()["n_duel"] > 0


@pytest.mark.gpu
def test_policy_sweep_on_the_gpu_matches_oracle_and_laws():
    from paper_2603_20661_b200.binding import Network
    wl = synth.make_policy_sweep(replicas_per_axis=32, n_requests=4000)
    g = Network(wl.settings, wl.peers, wl.batch); g.bind_requests(wl.requests)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    for s in range(wl.n_steps):
        first = s * wl.batch
        g.step(first, wl.batch, wl.step_now_ms(s), s % wl.gossip_every == 0)
        o.run_step(first, wl.batch, wl.step_now_ms(s), s % wl.gossip_every == 0)
    assert_same_state(g, o, "policy sweep", upto=wl.n_requests)
    _check_laws(wl, g.results())
