"""Host logic of bench.py that needs no GPU: how `--gpus N` starts its own ranks, and how the DRAM-traffic
figure of the roofline is tied to the kernels it was captured on."""
import os
import subprocess
import sys

import bench


def test_launcher_command_starts_one_rank_per_gpu_on_this_node():
    cmd = bench.launcher_command(["--gpus", "4", "--steps", "7", "--warmup", "3"], 4, 29511)
    assert cmd[0] == sys.executable and cmd[1:3] == ["-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29511"
    i = cmd.index(os.path.abspath(bench.__file__))
    assert cmd[i + 1:] == ["--gpus", "4", "--steps", "7", "--warmup", "3"]     # the ranks get the caller's arguments


def test_only_rank_zero_prints_the_reference_line():
    """Under a multi-rank launch the reference arm runs on rank 0 alone: the other ranks exit 0 without work."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, bench.__file__, "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                        "--config", "cfg1"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_traffic_figure_is_dropped_when_the_kernels_change(tmp_path, monkeypatch):
    h = bench.kernel_source_hash()
    prof = tmp_path / "profiles"
    prof.mkdir()
    (prof / "dram_traffic.txt").write_text(f"# path cfg extra read write hash\nsample cfg5 - 100 50 {h}\nsample cfg3 - 7 3 deadbeef\n")
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    monkeypatch.setattr(bench, "kernel_source_hash", lambda: h)
    assert bench.captured_traffic("sample", "cfg5")[0] == 150
    assert bench.captured_traffic("sample", "cfg3")[0] is None      # captured on other kernels
    assert bench.captured_traffic("greedy", "cfg5")[0] is None      # never captured
