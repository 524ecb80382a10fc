"""ctypes binding of the C oracle (test infrastructure only).

`build()` compiles `wwws_oracle.c` with gcc into `libwwws_oracle.so` beside it
(no fused multiply-add, no fast-math) and `Oracle` wraps one simulated network.
The settings object it takes is duck-typed (attributes named like the fields of
the configuration record); per-peer and request inputs are numpy arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wwws_oracle.c")
_SO = os.path.join(_HERE, "libwwws_oracle.so")

STAT_NAMES = ("n_requests", "n_local", "n_fallback_local", "n_dropped", "n_failed", "n_delegated", "n_duel",
              "n_duel_cancelled", "n_draw", "n_judge_evals", "n_probes", "n_near_boundary", "slo_met",
              "sum_latency_ms", "n_offline_marks", "rounds", "blocks", "credit_total", "chain_head", "pending_digest", "n_uncovered", "blocks_rejected")
TABLES = ("online", "cap_eff", "backlog", "ver", "credit", "stake", "wins", "duels", "served", "served_local",
          "d_credit", "d_wins", "d_duels", "blk_spent")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-Wall",
                               "-shared", "-fPIC", "-o", _SO, _SRC])
    return _SO


class _Config(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in ("n_peers", "n_replicas", "replica_offset", "pad0")] + \
               [("seed", C.c_uint64)] + \
               [(n, C.c_uint32) for n in ("fanout_k", "gossip_tries", "max_probes", "n_judges", "p_duel_ppm",
                                          "p_noise_ppm", "p_leave_ppm", "p_join_ppm", "p_prio_active_ppm",
                                          "prio_window_ms", "util_window_ms", "cap_ref_tok_s", "slo_num", "slo_den",
                                          "hop_ms", "init_stale_max", "flags", "n_rank")] + \
               [(n, C.c_int64) for n in ("reward_R", "reward_add", "penalty_P")] + \
               [("rank_cdf", C.c_void_p)]


_PEER_ORDER = (("cap_true_tok_s", np.uint32), ("quality_fx", np.uint32), ("credit0", np.int64),
               ("stake_pm", np.uint16), ("offload_util_pm", np.uint16), ("accept_util_pm", np.uint16),
               ("offload_ppm", np.uint32), ("accept_ppm", np.uint32),
               ("misreport_mul", np.uint8), ("prio_flag", np.uint8), ("online0", np.uint8))


class _PeerInit(C.Structure):
    _fields_ = [(n, C.c_void_p) for n, _ in _PEER_ORDER]


_lib = None


def lib():
    global _lib
    if _lib is None:
        # WWWS_ORACLE_LIBRARY: another build of the oracle (the pin tests load deliberately broken copies
        # through it to show that each planted mistake is caught)
        L = C.CDLL(os.environ.get("WWWS_ORACLE_LIBRARY") or build())
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(_Config), C.POINTER(_PeerInit)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_bind_requests.argtypes = [C.c_void_p] + [C.c_void_p] * 4 + [C.c_uint64]
        L.orc_advance_time.argtypes = [C.c_void_p, C.c_uint32]
        L.orc_gossip_round.argtypes = [C.c_void_p]
        L.orc_dispatch_batch.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64]
        L.orc_duel_judge.argtypes = [C.c_void_p]
        L.orc_settle_credits.argtypes = [C.c_void_p, C.c_int]
        L.orc_stats.argtypes = [C.c_void_p, C.c_void_p]
        L.orc_error.argtypes = [C.c_void_p]
        L.orc_table.argtypes = [C.c_void_p, C.c_int, C.c_void_p]
        L.orc_window_weights.argtypes = [C.c_void_p, C.c_uint32, C.c_uint64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_poke_peer.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_int, C.c_int64, C.c_int64]
        L.orc_poke_view.argtypes = [C.c_void_p, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint64]
        L.orc_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_ppm.restype = C.c_uint32; L.orc_ppm.argtypes = [C.c_uint32]
        L.orc_below.restype = C.c_uint32; L.orc_below.argtypes = [C.c_uint32, C.c_uint32]
        L.orc_mulhi64.restype = C.c_uint64; L.orc_mulhi64.argtypes = [C.c_uint64, C.c_uint64]
        L.orc_merge.restype = C.c_uint64; L.orc_merge.argtypes = [C.c_uint64, C.c_uint64]
        L.orc_mix64.restype = C.c_uint64; L.orc_mix64.argtypes = [C.c_uint64]
        for name, ct in (("orc_view", C.c_uint64), ("orc_exec_a", C.c_int32), ("orc_exec_b", C.c_int32),
                         ("orc_judges", C.c_int32), ("orc_outcome", C.c_uint8), ("orc_flags", C.c_uint8),
                         ("orc_score_a", C.c_float), ("orc_score_sum", C.c_float)):
            getattr(L, name).restype = C.POINTER(ct)
            getattr(L, name).argtypes = [C.c_void_p]
        L.orc_stats_width.restype = C.c_uint32
        _lib = L
    return _lib


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, np.uint32); k = np.asarray(key, np.uint32); out = np.zeros(4, np.uint32)
    lib().orc_philox4x32_10(c.ctypes.data, k.ctypes.data, out.ctypes.data)
    return out


class Oracle:
    """One simulated network on the CPU.  Calls mirror the library's call sequence."""

    def __init__(self, settings, peers):
        L = lib()
        cfg = _Config()
        for name, _ in _Config._fields_:
            if name in ("pad0", "rank_cdf", "n_rank"):
                continue
            setattr(cfg, name, int(getattr(settings, name)))
        self._cdf = None
        if getattr(settings, "rank_cdf", None) is not None:
            self._cdf = np.ascontiguousarray(settings.rank_cdf, np.uint32)
            cfg.rank_cdf = self._cdf.ctypes.data
            cfg.n_rank = self._cdf.size
        self.Rp, self.N = int(settings.n_replicas), int(settings.n_peers)
        self._peers = {}
        init = _PeerInit()
        for name, dt in _PEER_ORDER:
            a = np.ascontiguousarray(peers[name], dt)
            assert a.shape == (self.Rp, self.N), (name, a.shape)
            self._peers[name] = a
            setattr(init, name, a.ctypes.data)
        self._h = L.orc_create(C.byref(cfg), C.byref(init))
        self.Q = 0
        self._req = None

    def close(self):
        if self._h:
            lib().orc_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    def bind_requests(self, requests):
        self._req = {k: np.ascontiguousarray(requests[k], dt) for k, dt in
                     (("origin", np.uint32), ("t_ms", np.uint32), ("len_in", np.uint16), ("len_out", np.uint16))}
        self.Q = int(self._req["origin"].shape[1])
        assert self._req["origin"].shape[0] == self.Rp
        lib().orc_bind_requests(self._h, *(self._req[k].ctypes.data for k in ("origin", "t_ms", "len_in", "len_out")),
                                self.Q)

    def advance_time(self, now_ms):
        lib().orc_advance_time(self._h, int(now_ms))

    def gossip_round(self):
        lib().orc_gossip_round(self._h)

    def dispatch_batch(self, first, count):
        rc = lib().orc_dispatch_batch(self._h, int(first), int(count))
        if rc:
            raise RuntimeError(f"oracle dispatch status {rc}")

    def duel_judge(self):
        rc = lib().orc_duel_judge(self._h)
        if rc:
            raise RuntimeError(f"oracle duel status {rc}")

    def settle_credits(self, finalize=True):
        rc = lib().orc_settle_credits(self._h, 1 if finalize else 0)
        if rc:
            raise RuntimeError(f"oracle settle status {rc}")

    def error(self):
        return int(lib().orc_error(self._h))

    def stats(self):
        w = int(lib().orc_stats_width())
        out = np.zeros((self.Rp + 1, w), np.uint64)
        lib().orc_stats(self._h, out.ctypes.data)
        return out

    def stats_dict(self, row=-1):
        s = self.stats()[row]
        d = {k: int(v) for k, v in zip(STAT_NAMES, s)}
        d["credit_total"] = int(np.int64(s[STAT_NAMES.index("credit_total")]))
        return d

    def table(self, name):
        out = np.zeros((self.Rp, self.N), np.int64)
        rc = lib().orc_table(self._h, TABLES.index(name), out.ctypes.data)
        assert rc == 0
        return out

    def view(self):
        p = lib().orc_view(self._h)
        return np.ctypeslib.as_array(p, shape=(self.Rp, self.N, self.N)).copy()

    def _res(self, fn, shape):
        return np.ctypeslib.as_array(getattr(lib(), fn)(self._h), shape=shape).copy()

    def results(self):
        s = (self.Rp, self.Q)
        return {"exec_a": self._res("orc_exec_a", s), "exec_b": self._res("orc_exec_b", s),
                "judges": self._res("orc_judges", s + (4,)), "outcome": self._res("orc_outcome", s),
                "flags": self._res("orc_flags", s), "score_a": self._res("orc_score_a", s),
                "score_sum": self._res("orc_score_sum", s)}

    def window_weights(self, r, q):
        W = np.zeros(32, np.uint64); sc = np.zeros(32, np.float32); blk = np.zeros(1, np.uint32)
        lib().orc_window_weights(self._h, r, q, W.ctypes.data, sc.ctypes.data, blk.ctypes.data)
        return W, sc, int(blk[0])

    def poke_peer(self, r, j, online=-1, backlog=-1, cap_eff=-1):
        lib().orc_poke_peer(self._h, r, j, online, backlog, cap_eff)

    def poke_view(self, r, i, j, entry):
        lib().orc_poke_view(self._h, r, i, j, int(entry))

    def run_step(self, first, count, now_ms, gossip, finalize=True):
        """advance -> [gossip] -> dispatch -> duel -> settle, the call sequence of one step."""
        self.advance_time(now_ms)
        if gossip:
            self.gossip_round()
        self.dispatch_batch(first, count)
        self.duel_judge()
        self.settle_credits(finalize)
