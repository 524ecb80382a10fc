"""The C-ABI library loads without a GPU, exports every function the header declares, and
rejects bad arguments on the host (no compute call is made here)."""
import ctypes as C
import os
import re

import numpy as np

from paper_2603_20661_b200 import binding, synth
from paper_2603_20661_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "wwws.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wwws_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_function_is_exported_and_bound():
    cuda_build.build()
    lib = binding.load()
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/wwws.h but not exported"
    assert set(binding.EXPORTS) == set(names), set(binding.EXPORTS) ^ set(names)
    for n in names:
        assert callable(getattr(binding, n))


def test_struct_layouts_match_the_header():
    assert C.sizeof(binding.Config) == 16 + 8 + 18 * 4 + 3 * 8 + 8
    assert C.sizeof(binding.PeerInit) == 11 * 8 and C.sizeof(binding.Requests) == 32
    assert C.sizeof(binding.Results) == 7 * 8 and C.sizeof(binding.HostIO) == 8 * 8
    assert len(binding.STAT_NAMES) == 22


def test_host_side_argument_checks():
    lib = binding.load()
    st = synth.Settings(64, 2)
    cfg, _ = binding.make_config(st, 100)
    n = C.c_uint64()
    assert lib.wwws_workspace_bytes(C.byref(cfg), C.byref(n)) == 0
    ld = 64
    assert n.value >= 2 * 2 * 64 * ld * 8 and n.value % 256 == 0
    assert lib.wwws_workspace_bytes(C.byref(cfg), None) == 1
    assert lib.wwws_workspace_bytes(None, C.byref(n)) == 1
    bad = [("n_peers", 1), ("n_peers", 70000), ("n_replicas", 0), ("fanout_k", 5), ("fanout_k", 0), ("max_probes", 16),
           ("n_judges", 5), ("p_duel_ppm", 1_000_001), ("util_window_ms", 0), ("slo_den", 0), ("reward_R", 0),
           ("reward_add", 71), ("max_batch", 0), ("init_stale_max", (1 << 24) - 2)]
    for field, val in bad:
        cfg2, _ = binding.make_config(st, 100)
        setattr(cfg2, field, val)
        assert lib.wwws_workspace_bytes(C.byref(cfg2), C.byref(n)) == 1, field
        assert len(lib.wwws_last_error(None)) > 0
    # a rank CDF must be nondecreasing and come with its length
    st.rank_cdf = np.array([10, 5, 20], np.uint32)
    cfg3, keep = binding.make_config(st, 100)
    assert lib.wwws_workspace_bytes(C.byref(cfg3), C.byref(n)) == 1
    # create: null workspace / misaligned workspace / null arrays are refused before any CUDA call
    st.rank_cdf = None
    cfg4, _ = binding.make_config(st, 100)
    h = C.c_void_p()
    init = binding.PeerInit()
    assert lib.wwws_create_network(C.byref(cfg4), C.byref(init), None, 0, None, C.byref(h)) == 1
    assert h.value is None
    assert lib.wwws_create_network(C.byref(cfg4), None, None, 0, None, C.byref(h)) == 1
    # a workspace that is not device memory is refused before anything is built on it: the GPU that
    # holds the workspace is the network's GPU, and every later call runs there whatever device is current
    pa = {k: np.ascontiguousarray(np.broadcast_to(np.asarray(v), (2, 64)).astype(dt)) for (k, dt), v in
          zip(binding.PEER_ORDER, (2000, 1 << 31, 10_000, 1000, 0, 1001, 10 ** 6, 10 ** 6, 1, 0, 1))}
    for k, _ in binding.PEER_ORDER:
        setattr(init, k, pa[k].ctypes.data)
    host_ws = np.zeros(n.value + 256, np.uint8)
    addr = (host_ws.ctypes.data + 255) & ~255
    assert lib.wwws_create_network(C.byref(cfg4), C.byref(init), addr, n.value, None, C.byref(h)) in (1, 5)
    assert h.value is None and len(lib.wwws_last_error(None)) > 0
    # null handles
    assert lib.wwws_gossip_round(None) == 1 and lib.wwws_dispatch_batch(None, 0, 1) == 1
    assert lib.wwws_gossip_round_static(None) == 1
    assert lib.wwws_destroy_network(None) == 0 and lib.wwws_kernel_launches(None) == 0
    assert lib.wwws_profile_kernels() == 16
    assert lib.wwws_profile_kernel_name(7) == b"k_gossip_merge"
