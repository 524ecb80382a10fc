"""Pins for the oracle's credit block chain (Table "Structure of a Credit Block").

The mixer is pinned to the published SplitMix64 outputs; block ids are recomputed from the
result records by a vectorised routine that sums record hashes in a different order (the
digest is order-independent); a changed record, a changed parent or a changed height each
give a different id.
"""
import os

import numpy as np

from oracle import Oracle, binding
from paper_2603_20661_b200 import synth

GAMMA = np.uint64(0x9E3779B97F4A7C15)
M64 = (1 << 64) - 1


def mix64(z):
    z = np.asarray(z, np.uint64).copy()
    z ^= z >> np.uint64(30); z *= np.uint64(0xBF58476D1CE4E5B9)
    z ^= z >> np.uint64(27); z *= np.uint64(0x94D049BB133111EB)
    z ^= z >> np.uint64(31)
    return z


def test_mixer_matches_published_splitmix64_outputs():
    want = [int(ln, 16) for ln in open(os.path.join(os.path.dirname(__file__), "golden", "splitmix64_kat.txt"))
            if ln.strip() and not ln.startswith("#")]
    L = binding.lib()
    got = [L.orc_mix64(((i + 1) * int(GAMMA)) & M64) for i in range(3)]
    assert got == want
    with np.errstate(over="ignore"):
        assert [int(v) for v in mix64(np.arange(1, 4, dtype=np.uint64) * GAMMA)] == want


def _records(wl, res, lo, hi, r):
    """(q, kind, peer, amount) of every ledger record of requests [lo, hi) of replica r."""
    st = wl.settings
    R, Ra, P = st.reward_R, st.reward_add, st.penalty_P
    q = np.arange(lo, hi)
    a, b, oc, jd = res["exec_a"][r, lo:hi], res["exec_b"][r, lo:hi], res["outcome"][r, lo:hi], res["judges"][r, lo:hi]
    o = wl.requests["origin"][r, lo:hi].astype(np.int64)
    out = []
    m = a >= 0
    out += [(q[m], 1, o[m], np.full(m.sum(), -R)), (q[m], 2, a[m], np.full(m.sum(), R))]
    d = np.isin(oc, (1, 2, 3))
    out += [(q[d], 3, o[d], np.full(d.sum(), -R)), (q[d], 4, b[d], np.full(d.sum(), R))]
    dec = np.isin(oc, (1, 2))
    win = np.where(oc == 1, a, b); lose = np.where(oc == 1, b, a)
    nj = (jd >= 0).sum(-1)
    share = (P - Ra) // np.maximum(nj, 1)
    out += [(q[dec], 5, lose[dec], np.full(dec.sum(), -P)), (q[dec], 6, win[dec], (Ra + (P - Ra) - share * nj)[dec])]
    for l in range(4):
        mj = dec & (jd[:, l] >= 0)
        out.append((q[mj], 7 + l, jd[mj, l], share[mj]))
    return out


def _digest(wl, res, lo, hi, r):
    key = np.uint64(wl.settings.seed) ^ (np.uint64(r + wl.settings.replica_offset) * GAMMA)
    total = np.uint64(0)
    with np.errstate(over="ignore"):
        for q, kind, peer, amount in reversed(_records(wl, res, lo, hi, r)):
            word = (q.astype(np.uint64) << np.uint64(32)) | np.uint64(kind << 24) | peer.astype(np.uint64)
            h = mix64(mix64(key ^ word) + amount.astype(np.int64).view(np.uint64))
            total += h[::-1].sum(dtype=np.uint64)
    return total, key


def test_block_ids_recomputed_from_results():
    wl = synth.make_workload("zipf1k", n_replicas=2, n_requests=3000, n_peers=96, replica_offset=7)
    wl.settings.p_duel_ppm = 300_000
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    heads = np.stack([mix64(np.uint64(wl.settings.seed) ^ (np.uint64(r + 7) * GAMMA)) for r in range(2)])
    assert np.array_equal(o.stats()[:2, 18], heads)
    block_lo, height = 0, 0
    for s in range(wl.n_steps):
        fin = s % 3 == 2 or s == wl.n_steps - 1            # blocks of up to three batches
        o.run_step(s * wl.batch, wl.batch, wl.step_now_ms(s), s % 2 == 0, fin)
        res = o.results()
        hi = (s + 1) * wl.batch
        stats = o.stats()
        for r in range(2):
            dig, key = _digest(wl, res, block_lo, hi, r)
            if fin:
                with np.errstate(over="ignore"):
                    want = mix64(mix64(heads[r] ^ key) + dig + GAMMA * np.uint64(height + 1))
                assert stats[r, 18] == want and stats[r, 19] == 0
                heads[r] = want
            else:
                assert stats[r, 19] == dig and stats[r, 18] == heads[r]
        if fin:
            block_lo, height = hi, height + 1
    assert o.stats_dict()["blocks"] == 2 * height
    assert heads[0] != heads[1]


def test_chain_detects_changed_record_parent_and_height():
    st, pa, rq = None, None, None
    from tests.helpers import make_net, requester_first
    outs = {}
    for tag, kw in (("base", {}), ("other_reward", {"reward_add": 41})):
        st, pa, rq = make_net(6, n_requests=200, seed=5, p_duel_ppm=500_000, peers=requester_first(6, credit0=10 ** 6), **kw)
        o = Oracle(st, pa); o.bind_requests(rq)
        o.run_step(0, 100, 0, False, True)
        h1 = o.stats_dict()["chain_head"]
        o.run_step(100, 100, 0, False, True)
        outs[tag] = (h1, o.stats_dict()["chain_head"])
    assert outs["base"][0] != outs["other_reward"][0]         # one changed amount changes the block id
    assert outs["base"][0] != outs["base"][1]
    # empty blocks still chain: same (empty) content at heights 1 and 2 gives different ids
    st, pa, rq = make_net(4, n_requests=10, p_duel_ppm=0, peers={"offload_ppm": 0})
    o = Oracle(st, pa); o.bind_requests(rq)
    ids = [o.stats_dict()["chain_head"]]
    for s in range(2):
        o.run_step(5 * s, 5, 0, False, True)
        assert o.stats_dict()["pending_digest"] == 0
        ids.append(o.stats_dict()["chain_head"])
    assert len(set(ids)) == 3


def test_majority_validation_keeps_a_block_open_without_a_majority():
    """Flag 32: a proposed block is final only if more than half of the peers are online to
    confirm it; otherwise ledger, stakes and chain head stay as they were and the operations
    are committed with the next block that finds a majority."""
    from tests.helpers import make_net, requester_first
    st, pa, rq = make_net(5, n_requests=30, seed=2, p_duel_ppm=500_000, n_judges=1, flags=32,
                          peers=requester_first(5, credit0=10 ** 6))
    o = Oracle(st, pa); o.bind_requests(rq)
    o.run_step(0, 10, 0, False, True)
    d1 = o.stats_dict(); c1 = o.table("credit").copy()
    assert d1["blocks"] == 1 and d1["blocks_rejected"] == 0
    for j in (2, 3, 4):                                   # three of five crash: two online, no majority
        o.poke_peer(0, j, online=0)
    o.run_step(10, 10, 0, False, True)
    d2 = o.stats_dict()
    assert d2["blocks"] == 1 and d2["blocks_rejected"] == 1 and d2["chain_head"] == d1["chain_head"]
    assert np.array_equal(o.table("credit"), c1) and d2["pending_digest"] != 0
    assert np.any(o.table("d_credit") != 0) and d2["credit_total"] == d1["credit_total"]
    o.poke_peer(0, 2, online=1)                           # three online again: majority
    o.run_step(20, 10, 0, False, True)
    d3 = o.stats_dict()
    assert d3["blocks"] == 2 and d3["blocks_rejected"] == 1 and d3["pending_digest"] == 0
    assert np.all(o.table("d_credit") == 0) and o.table("credit").sum() == c1.sum()
    # the delayed block holds the operations of both batches: same ledger as one block over both
    st2, pa2, rq2 = make_net(5, n_requests=30, seed=2, p_duel_ppm=500_000, n_judges=1, flags=0,
                             peers=requester_first(5, credit0=10 ** 6))
    o2 = Oracle(st2, pa2); o2.bind_requests(rq2)
    o2.run_step(0, 10, 0, False, True)
    for j in (2, 3, 4):
        o2.poke_peer(0, j, online=0)
    o2.run_step(10, 10, 0, False, False)
    o2.poke_peer(0, 2, online=1)
    o2.run_step(20, 10, 0, False, True)
    assert np.array_equal(o2.table("credit"), o.table("credit"))
    assert o2.stats_dict()["chain_head"] == d3["chain_head"]
    # exactly half is not a majority
    st3, pa3, rq3 = make_net(4, n_requests=5, flags=32, p_duel_ppm=0, peers={"online0": np.array([1, 1, 0, 0])})
    o3 = Oracle(st3, pa3); o3.bind_requests(rq3)
    o3.run_step(0, 5, 0, False, True)
    assert o3.stats_dict()["blocks"] == 0 and o3.stats_dict()["blocks_rejected"] == 1
