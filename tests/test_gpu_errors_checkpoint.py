"""GPU-side error reporting (no fault is ever provoked: every case is bounds-checked by the
library and surfaces as a status) and checkpoint / resume."""
import numpy as np
import pytest

from paper_2603_20661_b200 import synth
from tests.helpers import make_net

pytestmark = pytest.mark.gpu


def test_call_order_and_range_errors_are_statuses():
    from paper_2603_20661_b200.binding import Network, WwwsError
    st, pa, rq = make_net(40, n_requests=300, seed=1)
    g = Network(st, pa, 100)
    with pytest.raises(WwwsError) as e:
        g.dispatch_batch(0, 10)                   # nothing bound
    assert e.value.status == 3
    g.bind_requests(rq)
    for call, status in ((lambda: g.duel_judge(), 3), (lambda: g.settle_credits(), 3),
                         (lambda: g.dispatch_batch(0, 101), 1), (lambda: g.dispatch_batch(250, 100), 1),
                         (lambda: g.dispatch_batch(0, 0), 1)):
        with pytest.raises(WwwsError) as e:
            call()
        assert e.value.status == status
    g.dispatch_batch(0, 100)
    for call in (lambda: g.dispatch_batch(100, 100), lambda: g.gossip_round(), lambda: g.advance_time(5),
                 lambda: g.settle_credits(), lambda: g.import_table("backlog", np.zeros((1, 40), np.int64))):
        with pytest.raises(WwwsError) as e:
            call()
        assert e.value.status == 3
    g.duel_judge(); g.settle_credits()
    g.advance_time(100)
    with pytest.raises(WwwsError) as e:
        g.advance_time(99)                        # time must not go back
    assert e.value.status == 1
    assert g.stats_dict()["n_requests"] == 100    # the handle is still usable


def test_bad_origin_index_is_dropped_and_reported():
    from paper_2603_20661_b200.binding import Network, WwwsError
    origin = np.arange(64) % 40
    origin[7] = 40; origin[20] = 2 ** 31
    st, pa, rq = make_net(40, n_requests=64, seed=2, origin=origin)
    g = Network(st, pa, 64); g.bind_requests(rq)
    g.step(0, 64, 10, True)
    with pytest.raises(WwwsError) as e:
        g.stats()
    assert e.value.status == 1 and "origin" in str(e.value)
    ex = g.results()["exec_a"][0]
    assert ex[7] == -3 and ex[20] == -3 and np.all(ex[np.r_[0:7, 8:20, 21:64]] != -3)
    sd = g.stats_dict()                           # the error word was cleared by the report
    assert sd["n_dropped"] == 2 and sd["n_requests"] == 64


def test_version_overflow_is_reported():
    from paper_2603_20661_b200.binding import Network, WwwsError
    st, pa, _ = make_net(8, fanout_k=1)
    st.init_stale_max = (1 << 24) - 3
    g = Network(st, pa, 1)
    g.gossip_round()
    g.stats()
    g.gossip_round()
    with pytest.raises(WwwsError) as e:
        g.stats()
    assert e.value.status == 4


@pytest.mark.parametrize("flags,cut", [(0, 3), (16, 2)], ids=["block_closed_at_the_cut", "exact_queueing_block_open_at_the_cut"])
def test_checkpoint_resume_continues_bit_for_bit(flags, cut):
    """Steps 0 and 2 finalize, step 1 does not: a cut after two steps leaves a block open, and with
    exact queueing the credits spent inside it (table blk_spent) decide which later payments are covered."""
    from paper_2603_20661_b200.binding import Network
    wl = synth.make_workload("churn4k", n_replicas=2, n_requests=6000, n_peers=300)
    wl.settings.p_duel_ppm = 300_000
    wl.settings.flags |= flags
    if flags & 16:
        wl.peers["credit0"][:] = 900              # a few payments per peer are covered, the rest are not

    def run(net, s0, s1):
        for s in range(s0, s1):
            net.step(s * wl.batch, wl.batch, wl.step_now_ms(s), s % 2 == 0, s % 3 != 1)

    a = Network(wl.settings, wl.peers, wl.batch); a.bind_requests(wl.requests)
    run(a, 0, cut)
    ck = a.checkpoint()
    if flags & 16:
        assert ck["tables"]["blk_spent"].any() and ck["tables"]["d_credit"].any()       # the cut is inside a block
    b = Network(wl.settings, wl.peers, wl.batch); b.bind_requests(wl.requests)
    b.restore(ck)
    run(a, cut, 6); run(b, cut, 6)
    ra, rb = a.results(), b.results()
    lo, hi = cut * wl.batch, 6 * wl.batch
    for k in ("exec_a", "exec_b", "judges", "outcome", "flags"):
        assert np.array_equal(ra[k][:, lo:hi], rb[k][:, lo:hi]), k
    assert np.array_equal(a.view(), b.view()) and np.array_equal(a.stats(), b.stats())
    ca, cb = a.checkpoint(), b.checkpoint()
    for k in ca["tables"]:
        assert np.array_equal(ca["tables"][k], cb["tables"][k]), k
    assert ca["clock"] == cb["clock"]
    if flags & 16:
        assert a.stats_dict()["n_uncovered"] > 0
