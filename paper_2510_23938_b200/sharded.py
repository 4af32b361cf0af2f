"""Global Merkle root of a blob whose chunks are spread over several GPUs.

The paper's multi-GPU scheme ("Multi-GPU Deployment Architectures": every GPU hashes its shard,
a global Merkle tree is built from the distributed hashes by hierarchical reduction) for the tree
rule of this library.  Pairing in the tree is index-aligned, so an aligned run of 2^k leaves is a
node of the global tree whoever computes it.  The plan therefore cuts the leaves at multiples of
2^k; every rank reduces its own leaves k levels (`iv_merkle_levels`), the few resulting nodes are
all-gathered (32 bytes each -- the only exchange on the path), and every rank finishes with
`iv_merkle_root` over the gathered nodes.  One process per GPU, `torch.distributed` for the
exchange (NCCL on GPUs; the tests run the same code over gloo).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch
import torch.distributed as dist


@dataclass(frozen=True)
class ShardPlan:
    n_leaves: int
    world: int
    level: int                      # k: every rank reduces its leaves k levels before the exchange
    n_nodes: int                    # level-k nodes of the whole tree
    node_ranges: tuple              # per rank (lo, hi) in level-k nodes
    leaf_ranges: tuple              # per rank (lo, hi) in leaves / chunks

    @property
    def max_nodes_per_rank(self) -> int:
        return max((hi - lo for lo, hi in self.node_ranges), default=0)


def plan_shards(n_leaves: int, world: int, min_nodes_per_rank: int = 1) -> ShardPlan:
    """Contiguous, 2^k-aligned leaf ranges, as even as the alignment allows (some may be empty).

    A rank's share is a whole number of 2^k-leaf runs, so a large k makes the shares uneven;
    `min_nodes_per_rank` trades a few more gathered nodes (32 bytes each) for balance: with 64 the
    shares differ by at most one part in 64."""
    assert n_leaves >= 0 and world >= 1 and min_nodes_per_rank >= 1
    level = 0
    while (2 << level) * world * min_nodes_per_rank <= n_leaves:   # largest k with 2^k * world * m <= n_leaves
        level += 1
    run = 1 << level
    n_nodes = -(-n_leaves // run)
    node_ranges = tuple((r * n_nodes // world, (r + 1) * n_nodes // world) for r in range(world))
    leaf_ranges = tuple((lo * run, min(hi * run, n_leaves)) for lo, hi in node_ranges)
    return ShardPlan(n_leaves, world, level, n_nodes, node_ranges, leaf_ranges)


def sharded_root(ctx, local_leaves: torch.Tensor, plan: ShardPlan, rank: int, group=None) -> torch.Tensor:
    """Root of the whole tree (32 uint8 on this rank's device) from this rank's leaf digests.

    `ctx` supplies merkle_levels(nodes, levels) and merkle_root(nodes); `local_leaves` holds the
    digests of leaf_ranges[rank] in order.  Collective: every rank of `group` must call it."""
    lo, hi = plan.leaf_ranges[rank]
    assert local_leaves.numel() == 32 * (hi - lo), "local digests do not match the plan"
    device = local_leaves.device
    cap = max(plan.max_nodes_per_rank, 1)
    mine = torch.zeros((cap, 32), dtype=torch.uint8, device=device)
    n_mine = plan.node_ranges[rank][1] - plan.node_ranges[rank][0]
    if n_mine:
        nodes = ctx.merkle_levels(local_leaves.view(-1, 32), plan.level)
        assert nodes.shape[0] == n_mine
        mine[:n_mine] = nodes
    if plan.world == 1:
        gathered = [mine]
    elif mine.is_cuda and dist.get_backend(group) == "gloo":
        # gloo gathers host tensors only (checking the multi-rank logic without NCCL): stage through the host
        host = mine.cpu()
        gathered = [torch.empty_like(host) for _ in range(plan.world)]
        dist.all_gather(gathered, host, group=group)
        gathered = [g.to(device) for g in gathered]
    else:
        gathered = [torch.empty_like(mine) for _ in range(plan.world)]
        dist.all_gather(gathered, mine, group=group)          # the one exchange step: <= cap * 32 bytes per rank
    parts = [gathered[r][:plan.node_ranges[r][1] - plan.node_ranges[r][0]] for r in range(plan.world)]
    all_nodes = torch.cat(parts) if parts else mine[:0]
    return ctx.merkle_root(all_nodes.contiguous())


def count_mismatches(local_count, device, group=None):
    """Total number of mismatching chunks over all ranks (an 8-byte all-reduce).

    `local_count` is an int (the total comes back as an int) or a one-element int64 tensor, e.g. the
    n_mismatch field of a verification result still on the device; then the total comes back as a
    tensor on `device` and nothing waits for the GPU."""
    as_tensor = isinstance(local_count, torch.Tensor)
    t = local_count.clone().reshape(1) if as_tensor else torch.tensor([local_count], dtype=torch.int64, device=device)
    if dist.is_initialized() and dist.get_world_size(group) > 1:
        if t.is_cuda and dist.get_backend(group) == "gloo":
            host = t.cpu()
            dist.all_reduce(host, group=group)
            t = host.to(t.device)
        else:
            dist.all_reduce(t, group=group)
    return t if as_tensor else int(t.item())
