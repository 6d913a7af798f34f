"""Host-side logic of the multi-GPU mode: data-parallel replicas, no data-path collective.

Sequences are independent, so N GPUs run N replicas of the step on disjoint batches.  The only communication is outside
the step: the policy weights reach every replica by one broadcast (at start and at every weight refresh of the RL loop,
Section 2.3), and the benchmark adds a barrier on both sides of the timed region, the max over ranks of the device time
and the sum over ranks of the emitted tokens.  Works on any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import torch

BASE_SEED = 2604026779


def replica_seed(rank: int, config_index: int = 3) -> int:
    """Seed of a rank's synthetic batch: rank 0 is the single-GPU workload, the others draw independent batches."""
    return BASE_SEED + 1000 * config_index + 17 * rank


def shard_by_tokens(lens, world: int):
    """Splits sequence indices into `world` groups of nearly equal total cached tokens (longest first, greedy), the
    balance that matters when lengths are long-tailed.  Returns a list of index lists."""
    order = sorted(range(len(lens)), key=lambda i: (-int(lens[i]), i))
    groups, loads = [[] for _ in range(world)], [0] * world
    for i in order:
        g = min(range(world), key=lambda r: (loads[r], r))
        groups[g].append(i)
        loads[g] += int(lens[i])
    return [sorted(g) for g in groups]


def reduce_job(ms_local: float, tokens_local: float, dist=None, device="cpu"):
    """(max over ranks of the time, sum over ranks of the tokens); identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms_local), float(tokens_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([tokens_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t[0]), float(n[0])


def broadcast_weights(arenas, dist=None, src: int = 0, chunk_bytes: int = 1 << 30):
    """Overwrites every rank's weight arenas (flat uint8 tensors, same sizes on all ranks) with rank `src`'s, in place and
    in chunks so that no second copy of the weights is held: how refreshed policy weights reach the replicas.  Identity
    without a process group.  Returns the bytes broadcast."""
    total = 0
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return total
    for a in arenas:
        flat = a.view(-1)
        for off in range(0, flat.numel(), chunk_bytes):
            piece = flat[off : off + chunk_bytes]
            dist.broadcast(piece, src=src)
            total += piece.numel() * piece.element_size()
    return total
