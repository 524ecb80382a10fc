"""The benchmark's reference arm (the CPU oracle timed on the host) runs without a GPU and
prints the contract's JSON line; its helpers agree with the workload's step structure."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiers64",
                          "--steps", "6", "--warmup", "3"], capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "requests/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["steps"] == 6 and d["warmup"] == 3 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] == 1
    assert d["e2e"] == {"value": d["value"], "unit": "requests/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "tiers64"


def test_reference_arm_other_ranks_exit_quietly():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--gpus", "2"], capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_step_schedule_and_byte_model():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2603_20661_b200 import synth
    wl = synth.make_workload("tiny")
    n = wl.n_steps
    first, cnt, now, gossip = bench.step_args(wl, 0)
    assert (first, cnt, gossip) == (0, wl.batch, True) and now == wl.step_now_ms(0)
    f2, c2, now2, _ = bench.step_args(wl, n)             # second pass over the stream: time keeps growing
    assert (f2, c2) == (0, wl.batch) and now2 > bench.step_args(wl, n - 1)[2]
    g, r = bench.algorithmic_bytes(wl, {"n_requests": 10, "n_delegated": 4, "n_fallback_local": 1, "n_failed": 0})
    assert g == 2 * 8 * 8 * 8 and r == 10 * 34 + 5 * 256


def test_gpus_2_starts_two_ranks_and_rank_0_prints_the_line():
    """`--gpus 2` outside a launcher starts two processes itself (one per GPU for the GPU arm); with
    the reference arm only rank 0 works and prints."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload", "tiny",
                          "--steps", "4", "--warmup", "3"], capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip().startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0


def test_launcher_command_and_missing_devices():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.launcher_command(["--gpus", "4", "--steps", "2"], 4, port=29555)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29555"
    assert cmd[-5] == os.path.join(ROOT, "bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "2"]
    import torch
    if torch.cuda.device_count() < 2:
        # fewer devices than ranks: a clear refusal, not a silent single-GPU timing
        env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
        out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--workload", "tiny"],
                             capture_output=True, text=True, timeout=120, cwd=ROOT, env=env)
        assert out.returncode != 0 and "--gpus 2" in out.stderr and out.stdout.strip() == ""


def test_counter_files_on_record_are_found_and_tied_to_their_source():
    """The ncu counters bench.py quotes (DRAM traffic of the merge, warp instructions per request of
    the request kernels) come from small text files written when a capture is taken; each names the
    kernel's source file and its digest, and a figure is withheld once the source has changed."""
    sys.path.insert(0, ROOT)
    import bench
    recs = bench.read_counter_files()
    assert len(recs) >= 4 and all({"kernel", "commit", "source", "source_sha256", "command"} <= set(r) for r in recs)
    merge = bench.find_counters("k_gossip_merge", n_peers=16384, fanout_k=4, flags=3)
    assert merge and 4.29e9 < float(merge["dram_bytes_per_replica_round"]) < 4.5e9       # compulsory 2 * 8 * N^2 = 4.295e9
    for wl in ("adversarial16k", "zipf1k", "zipf1k_saturated", "adversarial16k_saturated"):
        rec = bench.find_counters("k_step_fused", workload=wl)
        assert rec and 50 < float(rec["warp_instructions_per_request"]) < 1000, wl
        assert 1 <= float(rec["active_lanes_per_instruction"]) <= 32
    assert bench.find_counters("k_step_fused", workload="no_such_workload") is None
    assert bench.source_unchanged(merge) in (True, False)
    assert bench.source_unchanged({"source": "bench.py", "source_sha256": "0" * 64}) is False
