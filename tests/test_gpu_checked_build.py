"""The index-checked build of the library (-DWWWS_CHECK_INDICES) on a workload that reaches every
kernel family: every index a kernel takes from device data is range-checked there, a bad one would
surface as status WWWS_ERR_INDEX at the next synchronising call, and results must still match the
oracle.  Runs in a child process because the library to load is chosen when the binding is imported."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu

CHILD = r"""
import numpy as np
from oracle import Oracle
from paper_2603_20661_b200 import binding, synth
from paper_2603_20661_b200.binding import Network
from tests.helpers import assert_same_state
assert binding._SO.endswith("libwwws_checked.so")
for flags, kernel, churn in ((3, 0, 60_000), (3 | 8 | 16, 4, 0), (3 | 4 | 32, 3, 150_000), (3, 2, 0)):
    wl = synth.make_workload("churn4k", n_replicas=3, n_requests=3000, n_peers=700)
    wl.settings.flags = flags
    wl.settings.p_duel_ppm = 200_000
    wl.settings.p_leave_ppm = wl.settings.p_join_ppm = churn
    g = Network(wl.settings, wl.peers, wl.batch); g.bind_requests(wl.requests)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    g.set_option(1, kernel)
    for s in range(wl.n_steps):
        args = (s * wl.batch, wl.batch, wl.step_now_ms(s), True, s % 2 == 0)
        (g.step if s % 2 == 0 else g.run_step)(*args)
        o.run_step(*args)
    assert_same_state(g, o, f"checked build, flags {flags}", upto=wl.n_requests)      # stats() would raise on an index error
    g.close()
print("checked build ok")
"""


def test_checked_build_runs_clean_and_matches_the_oracle():
    from paper_2603_20661_b200 import build as cuda_build
    so = cuda_build.SO_CHECKED
    if not os.path.exists(so) or os.path.getmtime(so) < max(os.path.getmtime(p) for p in cuda_build.sources()):
        cuda_build.build(checked=True)
    env = dict(os.environ, WWWS_LIBRARY=so, PYTHONPATH=ROOT)
    out = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stdout[-1500:] + out.stderr[-3000:]
    assert "checked build ok" in out.stdout
