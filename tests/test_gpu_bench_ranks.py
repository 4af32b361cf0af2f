"""`bench.py --gpus N` starts its own ranks and runs the whole multi-GPU step: every rank verifies its shard,
the global root comes from the all-gather of a few tree nodes, the mismatch counts are all-reduced.

Run here as two ranks on ONE GPU over gloo (`--same-device`): the ranks' kernels never wait on one another
(the exchange is a host-side collective between launches), so sharing a GPU is safe.  The global root the
ranks agree on must be the oracle's root over the two ranks' blobs laid end to end."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2510_23938_b200 import inputs

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_ranks_started_by_bench_agree_on_the_oracle_root_of_the_whole_blob():
    assert torch.cuda.is_available(), "the gpu-marked tests need a CUDA device"
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--same-device", "--dist-backend", "gloo",
           "--config", "1", "--steps", "3", "--warmup", "3", "--no-e2e", "--no-cpu"]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env, cwd=ROOT)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]          # rank 0 alone prints
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["verified_ok"] is True and out["value"] > 0
    assert "global root" in out["config"]["parallelism"] and "all-reduced" in out["config"]["parallelism"]
    chunk, nbytes = 64 << 10, 64 << 20
    whole = np.concatenate([inputs.uniform_bytes(nbytes, seed=1000 + r).numpy() for r in range(2)])
    want = oracle.merkle_root(oracle.hash_chunks(whole, chunk, nthreads=oracle.host_threads()))
    assert out["config"]["global_root"] == want.hex()


def test_gpus_flag_must_match_the_launcher():
    env = dict(os.environ, WORLD_SIZE="1", RANK="0", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--config", "1"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=ROOT)
    assert res.returncode != 0 and "--gpus 2" in res.stderr
