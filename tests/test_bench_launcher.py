"""Host logic of bench.py that needs no GPU: `--gpus N` without a launcher starts N ranks on 127.0.0.1."""
import sys
import types

import pytest

import bench


def test_spawn_ranks_composes_a_torchrun_command_on_localhost(monkeypatch):
    seen = {}

    def fake_run(cmd, **kw):
        seen["cmd"] = cmd
        return types.SimpleNamespace(returncode=0)

    monkeypatch.setattr(bench.subprocess, "run", fake_run)
    monkeypatch.setattr(bench.torch.cuda, "device_count", lambda: 8)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "7", "--warmup", "3"])
    args = types.SimpleNamespace(gpus=4, same_device=False)
    assert bench.spawn_ranks(args) == 0
    cmd = seen["cmd"]
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert int(cmd[cmd.index("--master-port") + 1]) > 0
    assert cmd[-6:] == ["--gpus", "4", "--steps", "7", "--warmup", "3"] and cmd[-7].endswith("bench.py")


def test_spawn_ranks_refuses_more_ranks_than_gpus(monkeypatch, capsys):
    monkeypatch.setattr(bench.torch.cuda, "device_count", lambda: 1)
    monkeypatch.setattr(bench.subprocess, "run", lambda *a, **k: pytest.fail("must not launch"))
    assert bench.spawn_ranks(types.SimpleNamespace(gpus=8, same_device=False)) == 2
    assert "needs 8 GPUs" in capsys.readouterr().err


def test_roofline_arithmetic():
    """851 GB/s = 148 SMs x 64 lanes x 1.965 GHz / 21.875 ops per byte; the chain-count bound of the 16 GB file."""
    assert abs(bench.PEAK_GBS - 850.9) < 0.1
    r = bench.roofline_of("hash_chunks_split_kernel", 16_060_553_136, 65.65, 3830)
    assert abs(r["achieved"] - 244.6) < 0.2 and abs(r["frac"] - 0.2875) < 0.001
    assert abs(r["chain_count_bound_gbs"] - 258.9) < 0.2 and abs(r["chain_count_bound_at_issue_floor_gbs"] - 376.3) < 0.2
    assert bench.split_cycles_per_block(148 * 32) == 1860.0 and bench.split_cycles_per_block(148 * 32 + 1) == 1916.0
    assert r["traffic"] == int(bench.TRAFFIC_FACTOR["hash_chunks_split_kernel"] * 16_060_553_136) > 16_060_553_136
