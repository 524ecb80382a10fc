"""The queue model of the oracle against the textbook recursion for the unfinished work of a
single first-come-first-served server with batch arrivals (Lindley's recursion):

    U <- max(0, U - drained since the last batch);   wait of a job = U / rate;   U <- U + job size.

The paper gives no queue formula (it measures latency on real backends), so the model is a
reading; these tests pin its arithmetic, with the stated integer roundings (tokens drained =
floor(rate * dt / 1000), latency = ceil(tokens * 1000 / rate) ms), to that recursion computed with
numpy prefix sums, on random job sizes and random gaps between batches."""
import numpy as np

from oracle import Oracle
from tests.helpers import make_net


def _lindley(cap, cap_ref, batches, times, slo=(2, 1), u0=0):
    """Sum of latencies, number of deadlines met and final unfinished work."""
    u, t_prev, lat_sum, met = u0, 0, 0, 0
    for work, t in zip(batches, times):
        u = max(0, u - cap * (t - t_prev) // 1000)
        t_prev = t
        ahead = u + np.cumsum(work)                                   # tokens to finish before each job is done
        lat = -(-ahead * 1000 // cap)
        deadline = slo[0] * (-(-work * 1000 // cap_ref)) // slo[1]
        lat_sum += int(lat.sum()); met += int((lat <= deadline).sum())
        u = int(ahead[-1])
    return lat_sum, met, u


def _run(cap, gaps_ms, sizes, B, flags, rng):
    Q = len(sizes)
    st, pa, rq = make_net(2, n_requests=Q, flags=flags, p_duel_ppm=0, origin=np.ones(Q, np.uint32),
                          peers={"cap_true_tok_s": np.array([1000, cap]), "offload_ppm": 0})
    rq["len_in"] = (sizes // 2).astype(np.uint16); rq["len_out"] = (sizes - sizes // 2).astype(np.uint16)
    o = Oracle(st, pa); o.bind_requests(rq)
    times = np.cumsum(gaps_ms)
    for b, t in enumerate(times):
        o.run_step(b * B, B, int(t), False)
    assert np.all(o.results()["exec_a"][0] == -1)                     # all served at the node itself
    return o, times


def test_fifo_latencies_follow_lindleys_recursion():
    rng = np.random.default_rng(7)
    met_all = 0
    for cap in (700, 2000, 5003):
        B, nb = 8, 60
        sizes = rng.integers(2, 3000, B * nb)
        gaps = rng.integers(1, 90_000, nb)                            # some gaps empty the queue, some do not
        o, times = _run(cap, gaps, sizes, B, 16, rng)
        lat, met, u = _lindley(cap, 2000, sizes.reshape(nb, B), times)
        sd = o.stats_dict()
        assert sd["sum_latency_ms"] == lat and sd["slo_met"] == met
        assert o.table("backlog")[0, 1] == u
        met_all += met
    assert 0.2 * 3 * 480 < met_all < 0.8 * 3 * 480                    # the cases separate met from missed deadlines


def test_without_exact_queueing_a_batch_sees_the_queue_at_its_start():
    """Flag 16 off: every job of a batch waits behind the unfinished work at the batch's arrival
    only (the stated simplification); the work still accumulates as in the recursion."""
    rng = np.random.default_rng(8)
    cap, B, nb = 1500, 30, 20
    sizes = rng.integers(2, 3000, B * nb)
    gaps = rng.integers(1, 60_000, nb)
    o, times = _run(cap, gaps, sizes, B, 0, rng)
    u, t_prev, lat_sum = 0, 0, 0
    for work, t in zip(sizes.reshape(nb, B), times):
        u = max(0, u - cap * (int(t) - t_prev) // 1000); t_prev = int(t)
        lat_sum += int((-(-(u + work) * 1000 // cap)).sum())
        u += int(work.sum())
    assert o.stats_dict()["sum_latency_ms"] == lat_sum
    assert o.table("backlog")[0, 1] == u
