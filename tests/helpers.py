"""Shared test helpers: small hand-built networks and the step driver."""
import numpy as np

from paper_2603_20661_b200 import synth

VER_SHIFT = 40
OFFBIT = 1 << 39


def entry_ver(e):
    return np.asarray(e, np.uint64) >> np.uint64(VER_SHIFT)


def entry_offline(e):
    return (np.asarray(e, np.uint64) >> np.uint64(39)) & np.uint64(1)


def entry_cap(e):
    return (np.asarray(e, np.uint64) >> np.uint64(20)) & np.uint64((1 << 19) - 1)


def entry_q(e):
    return np.asarray(e, np.uint64) & np.uint64((1 << 20) - 1)


def make_net(n_peers, n_replicas=1, n_requests=0, seed=0, peers=None, origin=None, lens=(512, 256), **settings):
    """A hand-built network: every peer identical unless `peers` overrides a field
    (scalar or array broadcastable to [n_replicas, n_peers])."""
    st = synth.Settings(n_peers, n_replicas, seed=seed, **settings)
    shape = (n_replicas, n_peers)
    base = {"cap_true_tok_s": 2000, "quality_fx": 1 << 31, "credit0": 10_000, "stake_pm": 1000,
            "offload_util_pm": 0, "accept_util_pm": 1001, "offload_ppm": 1_000_000, "accept_ppm": 1_000_000,
            "misreport_mul": 1, "prio_flag": 0, "online0": 1}
    base.update(peers or {})
    pa = {k: np.ascontiguousarray(np.broadcast_to(np.asarray(base[k]), shape).astype(dt))
          for k, dt in synth.PEER_FIELDS.items()}
    rq = None
    if n_requests:
        rs = (n_replicas, n_requests)
        org = np.zeros(rs, np.uint32) if origin is None else np.broadcast_to(np.asarray(origin), rs)
        rq = {"origin": np.ascontiguousarray(org, dtype=np.uint32),
              "t_ms": np.zeros(rs, np.uint32),
              "len_in": np.full(rs, lens[0], np.uint16), "len_out": np.full(rs, lens[1], np.uint16)}
    return st, pa, rq


def requester_first(n_peers, **over):
    """Per-peer overrides that make peer 0 a requester-only node (no capacity,
    always offloads); the paper's ablations use such a node to issue all requests."""
    cap = np.full(n_peers, 2000); cap[0] = 0
    d = {"cap_true_tok_s": cap}
    d.update(over)
    return d


def run_workload(sim, wl, steps=None, on_step=None):
    n = wl.n_steps if steps is None else min(steps, wl.n_steps)
    for s in range(n):
        first = s * wl.batch
        cnt = min(wl.batch, wl.n_requests - first)
        fin = (s + 1) % wl.finalize_every == 0
        sim.run_step(first, cnt, wl.step_now_ms(s), s % wl.gossip_every == 0, fin)
        if on_step:
            on_step(s, first, cnt)


def chi2_ok(obs, exp, z=5.0):
    """Chi-square statistic within z standard deviations of its mean (df, var 2 df)."""
    obs = np.asarray(obs, float); exp = np.asarray(exp, float)
    m = exp > 0
    assert np.all(obs[~m] == 0)
    stat = float(((obs[m] - exp[m]) ** 2 / exp[m]).sum())
    df = int(m.sum()) - 1
    return stat <= df + z * np.sqrt(2.0 * df), stat, df


# ---- GPU-vs-oracle comparison -----------------------------------------------------------------

TABLE_NAMES = ("online", "cap_eff", "backlog", "ver", "credit", "stake", "wins", "duels", "served", "served_local",
               "d_credit", "d_wins", "d_duels", "blk_spent")


def assert_same_state(gpu, orc, where, upto=None, views=True, scores=True, stats=True):
    """Bit-exact agreement of every table, the views, the result records of requests
    [0, upto) and the counters; fp32 scores within 1e-5 relative (they are expected to be
    bit-equal: both sides use the same IEEE operations)."""
    for name in TABLE_NAMES:
        a, b = gpu.table(name).astype(np.int64), orc.table(name)
        assert np.array_equal(a, b), f"{where}: table {name} differs at {np.argwhere(a != b)[:5].tolist()}"
    if views:
        a, b = gpu.view(), orc.view()
        assert np.array_equal(a, b), f"{where}: views differ at {np.argwhere(a != b)[:5].tolist()}"
    if upto:
        rg, ro = gpu.results(), orc.results()
        mism = 0
        for k in ("exec_a", "exec_b", "judges", "outcome", "flags"):
            a, b = rg[k][:, :upto], ro[k][:, :upto]
            if not np.array_equal(a, b):
                bad = np.argwhere(a != b)
                # a differing choice is tolerable only where the oracle flagged a near-boundary draw
                near = ro["flags"][bad[:, 0], bad[:, 1]] & 1
                assert near.all(), f"{where}: {k} differs at {bad[:5].tolist()} away from any interval end"
                mism += len(bad)
        assert mism == 0, f"{where}: {mism} near-boundary choice mismatches (expected none: scores are bit-equal)"
        if scores and "score_a" in rg:
            for k in ("score_a", "score_sum"):
                a, b = rg[k][:, :upto].astype(np.float64), ro[k][:, :upto].astype(np.float64)
                rel = np.abs(a - b) / np.maximum(np.abs(b), 1e-30)
                assert np.all((rel <= 1e-5) | (a == b)), f"{where}: {k} off by {rel.max()}"
    if stats:
        a, b = gpu.stats(), orc.stats()
        assert np.array_equal(a, b), f"{where}: stats differ: {dict(zip(range(18), (a - b).sum(0).tolist()))}"
