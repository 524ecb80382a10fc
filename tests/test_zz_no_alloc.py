"""The gossip round that allocates nothing, against the ordinary one.

Some programs embed the library where device memory cannot be obtained (the GPU's memory is
all in another allocator's pool, or allocation is not allowed or too disruptive at that
point).  For them `wwws_gossip_round_static` keeps the round's scratch in a fixed array
inside the library.  This file is collected last on purpose: the entry point shares one
array per GPU, and a failure here must not hide results of the other tests.
"""
import numpy as np
import pytest

from oracle import Oracle
from paper_2603_20661_b200 import synth
from tests.helpers import assert_same_state

pytestmark = pytest.mark.gpu


def _evolved_network(wl):
    """A network a few steps into its life: queues, adverts and churn are non-trivial."""
    from paper_2603_20661_b200.binding import Network
    net = Network(wl.settings, wl.peers, wl.batch)
    net.bind_requests(wl.requests)
    for s in range(3):
        net.step(s * wl.batch, wl.batch, wl.step_now_ms(s), s == 0)
    return net


def _evolved_oracle(wl):
    o = Oracle(wl.settings, wl.peers)
    o.bind_requests(wl.requests)
    for s in range(3):
        o.run_step(s * wl.batch, wl.batch, wl.step_now_ms(s), s == 0)
    return o


@pytest.mark.parametrize("push_pull", [False, True], ids=["pull", "pairwise_exchange"])
def test_static_round_equals_ordinary_round_twice_in_a_row(push_pull):
    wl = synth.make_workload("churn4k", n_replicas=3, n_requests=4000, n_peers=1100)
    if push_pull:
        wl.settings.flags |= 8                # the partner lists in the built-in array also feed the reverse lists
    a, b, o = _evolved_network(wl), _evolved_network(wl), _evolved_oracle(wl)
    assert np.array_equal(a.view(), b.view())
    for rnd in range(2):                      # second call reuses the array with the first call's contents in it
        a.gossip_round()
        b.gossip_round_static()
        o.gossip_round()
        assert np.array_equal(a.view(), b.view()), f"round {rnd}: views differ"
        for t in ("online", "backlog", "ver"):
            assert np.array_equal(a.table(t), b.table(t)), f"round {rnd}: {t} differs"
        assert np.array_equal(a.stats(), b.stats()), f"round {rnd}: counters differ"
        # and against the CPU oracle: every table, the whole view matrix, the counters
        assert_same_state(b, o, f"static round {rnd}", upto=3 * wl.batch)
    # the networks stay interchangeable afterwards
    a.step(3 * wl.batch, wl.batch, wl.step_now_ms(3), True)
    b.step(3 * wl.batch, wl.batch, wl.step_now_ms(3), True)
    ra, rb = a.results(), b.results()
    for k in ra:
        assert np.array_equal(ra[k], rb[k]), k
    assert np.array_equal(a.view(), b.view())


def test_static_round_rejects_networks_beyond_its_array():
    from paper_2603_20661_b200.binding import Network, WwwsError
    wl = synth.make_workload("zipf1k", n_replicas=65, n_requests=500, n_peers=1024)     # 66,560 peers > 65,536
    net = Network(wl.settings, wl.peers, wl.batch)
    before = net.view_rows(0, 0, 4)
    with pytest.raises(WwwsError) as e:
        net.gossip_round_static()
    assert e.value.status == 1 and "65536" in str(e.value)
    assert np.array_equal(net.view_rows(0, 0, 4), before)       # nothing ran
    net.gossip_round()                                           # the ordinary round still works
