"""The multi-GPU path on CPU ranks: plan, exchange (gloo all-gather) and combination of the sharded root.

The ranks here have no GPU; the two tree operations the sharded code asks of a context are supplied by
the CPU oracle (an aligned run of 2^k leaves reduced with the oracle's root function is the level-k
node -- the property pinned in test_oracle_pins).  What is under test is the host logic: alignment of
the cut, which rank owns what, the gather order, ragged and empty shards."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2510_23938_b200 import sharded


class OracleTreeOps:
    def merkle_levels(self, nodes: torch.Tensor, levels: int) -> torch.Tensor:
        flat = nodes.numpy().reshape(-1, 32)
        run = 1 << levels
        out = [np.frombuffer(oracle.merkle_root(flat[s:s + run]), dtype=np.uint8) for s in range(0, len(flat), run)]
        return torch.from_numpy(np.stack(out).copy()) if out else torch.empty((0, 32), dtype=torch.uint8)

    def merkle_root(self, nodes: torch.Tensor) -> torch.Tensor:
        return torch.from_numpy(np.frombuffer(oracle.merkle_root(nodes.numpy()), dtype=np.uint8).copy())


def _leaves(n, seed=3):
    return np.random.default_rng(seed).integers(0, 256, size=(n, 32), dtype=np.uint8)


@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_plan_is_aligned_contiguous_and_complete(world):
    for n in list(range(0, 70)) + [1000, 1024, 1025, 2510, 3830, 28_672, 10_000]:
        p = sharded.plan_shards(n, world)
        run = 1 << p.level
        assert p.n_nodes == -(-n // run)
        assert p.leaf_ranges[0][0] == 0 and p.leaf_ranges[-1][1] == n
        for r in range(world):
            lo, hi = p.leaf_ranges[r]
            assert lo % run == 0 and lo <= hi
            if r + 1 < world:
                assert hi == p.leaf_ranges[r + 1][0]
                assert hi % run == 0 or hi == n
        if n >= world:
            assert all(hi > lo for lo, hi in p.node_ranges), (n, world)     # every rank has work


def test_balanced_plan_for_equal_shards():
    """With at least 64 nodes per rank the benchmark's shards (28,672 chunks per GPU) come out exactly equal."""
    for world in (2, 4, 8):
        p = sharded.plan_shards(world * 28_672, world, min_nodes_per_rank=64)
        assert all(hi - lo == 28_672 for lo, hi in p.leaf_ranges)
        assert p.level == 8 and p.n_nodes == world * 112
    p = sharded.plan_shards(1000, 3, min_nodes_per_rank=64)
    sizes = [hi - lo for lo, hi in p.leaf_ranges]
    assert sum(sizes) == 1000 and max(sizes) - min(sizes) <= 2 * (1 << p.level)


def test_single_process_emulation_of_ranks_gives_the_full_root():
    """All ranks' node lists concatenated in rank order reduce to the root of the whole tree."""
    ops = OracleTreeOps()
    for world in (2, 3, 5):
        for n in (1, 2, 3, 7, 8, 9, 31, 64, 65, 100, 1000, 2510):
            leaves = _leaves(n, seed=n)
            p = sharded.plan_shards(n, world)
            nodes = [ops.merkle_levels(torch.from_numpy(leaves[lo:hi]), p.level) for lo, hi in p.leaf_ranges if hi > lo]
            got = ops.merkle_root(torch.cat(nodes)).numpy().tobytes()
            assert got == oracle.merkle_root(leaves), (world, n)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, sizes, results):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ops = OracleTreeOps()
        ok = True
        for n in sizes:
            leaves = _leaves(n, seed=n)
            p = sharded.plan_shards(n, world)
            lo, hi = p.leaf_ranges[rank]
            root = sharded.sharded_root(ops, torch.from_numpy(leaves[lo:hi].copy()), p, rank)
            ok &= root.numpy().tobytes() == oracle.merkle_root(leaves)
            total = sharded.count_mismatches(rank + 1, "cpu")
            ok &= total == world * (world + 1) // 2
        results[rank] = bool(ok)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_root_over_gloo_ranks(world):
    sizes = [1, 2, 3, 5, 8, 17, 64, 100, 1023, 1024, 1025, 2510, 3830]
    with mp.Manager() as manager:
        results = manager.dict()
        mp.spawn(_rank_main, args=(world, _free_port(), sizes, results), nprocs=world, join=True)
        assert dict(results) == {r: True for r in range(world)}
