"""Thin Python binding of the wwws C-ABI: argument marshalling only.

Module-level functions carry the C names (`wwws_create_network`, ...) and return
the C status; `Network` is a convenience wrapper that owns the device workspace
(a torch tensor: PyTorch is used for device memory and streams, nothing else)
and raises `WwwsError` on a non-zero status.  Every step of the simulation runs
in the library's CUDA kernels; there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.environ.get("WWWS_LIBRARY") or os.path.join(_HERE, "libwwws.so")     # e.g. the index-checked build

STATUS = {0: "OK", 1: "ERR_ARG", 2: "ERR_ALLOC", 3: "ERR_STATE", 4: "ERR_RANGE", 5: "ERR_CUDA", 6: "ERR_INVARIANT",
          7: "ERR_TIMEOUT", 8: "ERR_INDEX"}
STAT_NAMES = ("n_requests", "n_local", "n_fallback_local", "n_dropped", "n_failed", "n_delegated", "n_duel",
              "n_duel_cancelled", "n_draw", "n_judge_evals", "n_probes", "n_near_boundary", "slo_met",
              "sum_latency_ms", "n_offline_marks", "rounds", "blocks", "credit_total", "chain_head", "pending_digest", "n_uncovered", "blocks_rejected")
TABLES = {"online": (0, np.uint8), "cap_eff": (1, np.uint32), "backlog": (2, np.int64), "ver": (3, np.uint32),
          "credit": (4, np.int64), "stake": (5, np.int64), "wins": (6, np.uint32), "duels": (7, np.uint32),
          "served": (8, np.uint64), "served_local": (9, np.uint64), "d_credit": (10, np.int64),
          "d_wins": (11, np.uint32), "d_duels": (12, np.uint32), "blk_spent": (13, np.int64)}
EXPORTS = ("wwws_workspace_bytes", "wwws_create_network", "wwws_destroy_network", "wwws_bind_requests",
           "wwws_advance_time", "wwws_gossip_round", "wwws_dispatch_batch", "wwws_duel_judge", "wwws_settle_credits",
           "wwws_step", "wwws_step_host", "wwws_stats", "wwws_export_table", "wwws_import_table",
           "wwws_export_view_rows", "wwws_kernel_launches", "wwws_last_error", "wwws_profile", "wwws_profile_read",
           "wwws_profile_kernels", "wwws_profile_kernel_name", "wwws_gossip_round_static", "wwws_import_view_rows",
           "wwws_export_clock", "wwws_import_clock", "wwws_import_stats", "wwws_set_option")


class WwwsError(RuntimeError):
    def __init__(self, status, text):
        super().__init__(f"wwws {STATUS.get(status, status)}: {text}")
        self.status = status


class Config(C.Structure):
    _fields_ = [("n_peers", C.c_uint32), ("n_replicas", C.c_uint32), ("replica_offset", C.c_uint32),
                ("max_batch", C.c_uint32), ("seed", C.c_uint64)] + \
               [(k, C.c_uint32) for k in ("fanout_k", "gossip_tries", "max_probes", "n_judges", "p_duel_ppm",
                                          "p_noise_ppm", "p_leave_ppm", "p_join_ppm", "p_prio_active_ppm",
                                          "prio_window_ms", "util_window_ms", "cap_ref_tok_s", "slo_num", "slo_den",
                                          "hop_ms", "init_stale_max", "flags", "n_rank")] + \
               [(k, C.c_int64) for k in ("reward_R", "reward_add", "penalty_P")] + [("rank_cdf", C.c_void_p)]


PEER_ORDER = (("cap_true_tok_s", np.uint32), ("quality_fx", np.uint32), ("credit0", np.int64), ("stake_pm", np.uint16),
              ("offload_util_pm", np.uint16), ("accept_util_pm", np.uint16), ("offload_ppm", np.uint32),
              ("accept_ppm", np.uint32), ("misreport_mul", np.uint8), ("prio_flag", np.uint8), ("online0", np.uint8))


class PeerInit(C.Structure):
    _fields_ = [(k, C.c_void_p) for k, _ in PEER_ORDER]


class Requests(C.Structure):
    _fields_ = [("origin", C.c_void_p), ("len_in", C.c_void_p), ("len_out", C.c_void_p), ("n_requests", C.c_uint64)]


class Results(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("exec_a", "exec_b", "judges", "outcome", "flags", "score_a", "score_sum")]


class HostIO(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("origin", "len_in", "len_out", "exec_a", "exec_b", "judges", "outcome", "flags")]


_lib = None


def load():
    """Load libwwws.so (raises if it has not been built: there is no other implementation)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise ImportError(f"{_SO} is missing: build it with `python -m paper_2603_20661_b200.build` "
                              "(needs nvcc); the package has no CPU path")
        L = C.CDLL(_SO)
        vp, u64, u32, i32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int
        sig = {
            "wwws_workspace_bytes": [C.POINTER(Config), C.POINTER(u64)],
            "wwws_create_network": [C.POINTER(Config), C.POINTER(PeerInit), vp, u64, vp, C.POINTER(vp)],
            "wwws_destroy_network": [vp],
            "wwws_bind_requests": [vp, C.POINTER(Requests), C.POINTER(Results)],
            "wwws_advance_time": [vp, u32], "wwws_gossip_round": [vp], "wwws_gossip_round_static": [vp],
            "wwws_dispatch_batch": [vp, u64, u64], "wwws_duel_judge": [vp], "wwws_settle_credits": [vp, i32],
            "wwws_step": [vp, u64, u64, u32, i32, i32],
            "wwws_step_host": [vp, C.POINTER(HostIO), u64, u64, u32, i32, i32, vp],
            "wwws_stats": [vp, vp], "wwws_export_table": [vp, i32, vp, u64], "wwws_import_table": [vp, i32, vp, u64],
            "wwws_export_view_rows": [vp, u32, u32, u32, vp],
            "wwws_profile": [vp, i32], "wwws_profile_read": [vp, vp, vp],
            "wwws_import_view_rows": [vp, u32, u32, u32, vp], "wwws_export_clock": [vp, C.POINTER(u32), C.POINTER(u32)],
            "wwws_import_clock": [vp, u32, u32], "wwws_import_stats": [vp, vp], "wwws_set_option": [vp, i32, C.c_int64],
        }
        for name, args in sig.items():
            f = getattr(L, name); f.argtypes = args; f.restype = C.c_int
        L.wwws_kernel_launches.argtypes = [vp]; L.wwws_kernel_launches.restype = u64
        L.wwws_last_error.argtypes = [vp]; L.wwws_last_error.restype = C.c_char_p
        L.wwws_profile_kernels.argtypes = []; L.wwws_profile_kernels.restype = u32
        L.wwws_profile_kernel_name.argtypes = [u32]; L.wwws_profile_kernel_name.restype = C.c_char_p
        _lib = L
    return _lib


def _export(name):
    def call(*a):
        return getattr(load(), name)(*a)
    call.__name__ = name
    call.__doc__ = f"C function {name}; see include/wwws.h."
    return call


for _n in EXPORTS:
    globals()[_n] = _export(_n)


def make_config(settings, max_batch):
    """Fill the C configuration record from a settings object (attribute names = field names)."""
    cfg = Config()
    for name, _ in Config._fields_:
        if name in ("rank_cdf", "n_rank", "max_batch"):
            continue
        setattr(cfg, name, int(getattr(settings, name)))
    cfg.max_batch = int(max_batch)
    keep = None
    if getattr(settings, "rank_cdf", None) is not None:
        keep = np.ascontiguousarray(settings.rank_cdf, np.uint32)
        cfg.rank_cdf = keep.ctypes.data
        cfg.n_rank = keep.size
    return cfg, keep


class Network:
    """One simulated network on one GPU.  Methods are the C calls with the status checked."""

    def __init__(self, settings, peers, max_batch, device="cuda:0", stream=None):
        import torch
        self._torch = torch
        L = load()
        self.device = torch.device(device)
        self.Rp, self.N = int(settings.n_replicas), int(settings.n_peers)
        cfg, self._cdf = make_config(settings, max_batch)
        nbytes = C.c_uint64()
        self._check(L.wwws_workspace_bytes(C.byref(cfg), C.byref(nbytes)), None)
        self.workspace_bytes = nbytes.value
        with torch.cuda.device(self.device):
            self._ws = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
            self._stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        init = PeerInit()
        self._peer_arrays = []
        for name, dt in PEER_ORDER:
            a = np.ascontiguousarray(peers[name], dt)
            if a.shape != (self.Rp, self.N):
                raise ValueError(f"{name}: expected shape {(self.Rp, self.N)}, got {a.shape}")
            self._peer_arrays.append(a)
            setattr(init, name, a.ctypes.data)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            self._check(L.wwws_create_network(C.byref(cfg), C.byref(init), self._ws.data_ptr(), self.workspace_bytes,
                                              self._stream.cuda_stream, C.byref(h)), None)
        self._h = h
        self.Q = 0
        self.req = self.res = None

    def _check(self, status, handle):
        if status != 0:
            raise WwwsError(status, load().wwws_last_error(handle).decode())

    def close(self):
        if getattr(self, "_h", None):
            load().wwws_destroy_network(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- requests -------------------------------------------------------------------------
    def bind_requests(self, requests, scores=True):
        """Upload request arrays (numpy, [Rp, Q]) and allocate result arrays on the device."""
        torch = self._torch
        t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a, dt).view(dt)).to(self.device)
        origin = np.ascontiguousarray(requests["origin"], np.uint32)
        self.Q = int(origin.shape[1])
        dev = self.device
        self.req = {"origin": t(origin.view(np.int32), np.int32), "len_in": t(np.ascontiguousarray(requests["len_in"], np.uint16).view(np.int16), np.int16),
                    "len_out": t(np.ascontiguousarray(requests["len_out"], np.uint16).view(np.int16), np.int16)}
        s = (self.Rp, self.Q)
        self.res = {"exec_a": torch.full(s, -9, dtype=torch.int32, device=dev),
                    "exec_b": torch.full(s, -9, dtype=torch.int32, device=dev),
                    "judges": torch.full(s + (4,), -9, dtype=torch.int32, device=dev),
                    "outcome": torch.zeros(s, dtype=torch.uint8, device=dev),
                    "flags": torch.zeros(s, dtype=torch.uint8, device=dev)}
        if scores:
            self.res["score_a"] = torch.zeros(s, dtype=torch.float32, device=dev)
            self.res["score_sum"] = torch.zeros(s, dtype=torch.float32, device=dev)
        self.bind_device(self.req, self.res)

    def bind_device(self, req, res):
        """Bind caller-owned device tensors (kept alive by this object)."""
        self.req, self.res = req, res
        self.Q = int(req["origin"].shape[1])
        rq = Requests(req["origin"].data_ptr(), req["len_in"].data_ptr(), req["len_out"].data_ptr(), self.Q)
        rs = Results(*(res[k].data_ptr() if k in res else None
                       for k in ("exec_a", "exec_b", "judges", "outcome", "flags", "score_a", "score_sum")))
        self._check(load().wwws_bind_requests(self._h, C.byref(rq), C.byref(rs)), self._h)

    # ---- the step ---------------------------------------------------------------------------
    def advance_time(self, now_ms):
        self._check(load().wwws_advance_time(self._h, int(now_ms)), self._h)

    def gossip_round(self):
        self._check(load().wwws_gossip_round(self._h), self._h)

    def gossip_round_static(self):
        """A gossip round whose scratch is the library's built-in array (see include/wwws.h)."""
        self._check(load().wwws_gossip_round_static(self._h), self._h)

    def dispatch_batch(self, first, count):
        self._check(load().wwws_dispatch_batch(self._h, int(first), int(count)), self._h)

    def duel_judge(self):
        self._check(load().wwws_duel_judge(self._h), self._h)

    def settle_credits(self, finalize=True):
        self._check(load().wwws_settle_credits(self._h, 1 if finalize else 0), self._h)

    def run_step(self, first, count, now_ms, gossip, finalize=True):
        """The six-call sequence of one step."""
        self.advance_time(now_ms)
        if gossip:
            self.gossip_round()
        self.dispatch_batch(first, count)
        self.duel_judge()
        self.settle_credits(finalize)

    def step(self, first, count, now_ms, gossip, finalize=True):
        """One step through the fused entry point."""
        self._check(load().wwws_step(self._h, int(first), int(count), int(now_ms), int(bool(gossip)),
                                     int(bool(finalize))), self._h)

    def step_host(self, io, first, count, now_ms, gossip, finalize=True, totals=True):
        """One step with host buffers (`io`: dict of pinned torch CPU tensors or numpy arrays)."""
        ptr = lambda a: a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
        h = HostIO(*(ptr(io[k]) for k in ("origin", "len_in", "len_out", "exec_a", "exec_b", "judges", "outcome", "flags")))
        out = np.zeros(len(STAT_NAMES), np.uint64) if totals else None
        self._check(load().wwws_step_host(self._h, C.byref(h), int(first), int(count), int(now_ms), int(bool(gossip)),
                                          int(bool(finalize)), out.ctypes.data if totals else None), self._h)
        return out

    # ---- reading state ------------------------------------------------------------------------
    def stats(self):
        out = np.zeros((self.Rp + 1, len(STAT_NAMES)), np.uint64)
        self._check(load().wwws_stats(self._h, out.ctypes.data), self._h)
        return out

    def stats_dict(self, row=-1):
        s = self.stats()[row]
        d = {k: int(v) for k, v in zip(STAT_NAMES, s)}
        d["credit_total"] = int(np.int64(s[STAT_NAMES.index("credit_total")]))
        return d

    def table(self, name):
        tid, dt = TABLES[name]
        out = np.zeros((self.Rp, self.N), dt)
        self._check(load().wwws_export_table(self._h, tid, out.ctypes.data, out.nbytes), self._h)
        return out

    def import_table(self, name, values):
        tid, dt = TABLES[name]
        a = np.ascontiguousarray(values, dt)
        assert a.shape == (self.Rp, self.N)
        self._check(load().wwws_import_table(self._h, tid, a.ctypes.data, a.nbytes), self._h)

    def view_rows(self, replica, row_first=0, n_rows=None):
        n_rows = self.N - row_first if n_rows is None else n_rows
        out = np.zeros((n_rows, self.N), np.uint64)
        self._check(load().wwws_export_view_rows(self._h, replica, row_first, n_rows, out.ctypes.data), self._h)
        return out

    def view(self):
        return np.stack([self.view_rows(r) for r in range(self.Rp)])

    def checkpoint(self):
        """Everything needed to resume: tables, views, counters, clock (host copies)."""
        now, rnd = C.c_uint32(), C.c_uint32()
        self._check(load().wwws_export_clock(self._h, C.byref(now), C.byref(rnd)), self._h)
        return {"tables": {k: self.table(k) for k in TABLES}, "view": self.view(), "stats": self.stats()[:-1].copy(),
                "clock": (now.value, rnd.value)}

    def restore(self, ck):
        """Load a checkpoint taken from a network of the same configuration."""
        for k, v in ck["tables"].items():
            self.import_table(k, v)
        for r in range(self.Rp):
            rows = np.ascontiguousarray(ck["view"][r], np.uint64)
            self._check(load().wwws_import_view_rows(self._h, r, 0, self.N, rows.ctypes.data), self._h)
        st = np.ascontiguousarray(ck["stats"], np.uint64)
        self._check(load().wwws_import_stats(self._h, st.ctypes.data), self._h)
        self._check(load().wwws_import_clock(self._h, *ck["clock"]), self._h)

    def results(self):
        self._torch.cuda.synchronize(self.device)
        return {k: v.cpu().numpy() for k, v in self.res.items()}

    def set_option(self, option, value):
        """Tuning option (see wwws_option in include/wwws.h); 0 = WWWS_OPT_REQUEST_KERNEL."""
        self._check(load().wwws_set_option(self._h, int(option), int(value)), self._h)

    def profile(self, enable):
        """Switch per-kernel event timing on or off (clears the sums)."""
        self._check(load().wwws_profile(self._h, int(bool(enable))), self._h)

    def profile_read(self):
        """{kernel name: (summed device ms, launches)} since profiling was switched on."""
        L = load()
        k = int(L.wwws_profile_kernels())
        ms = np.zeros(k, np.float64); cnt = np.zeros(k, np.uint64)
        self._check(L.wwws_profile_read(self._h, ms.ctypes.data, cnt.ctypes.data), self._h)
        return {L.wwws_profile_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(k) if cnt[i]}

    def kernel_launches(self):
        return int(load().wwws_kernel_launches(self._h))
