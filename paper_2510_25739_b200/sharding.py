"""Data-parallel sharding of a verify step: sequences are the independent unit.

Both guidance streams of a sequence stay on one rank (the accept stage needs the conditional and the
unconditional logit row together), every rank holds its own KV shard and a replica of the head weight,
and nothing is exchanged on the data path.  Only the two int32 results per sequence are gathered when
one rank wants them all.  Index arithmetic only: no step of the method is computed here.
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np


def sequence_range(B: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced split of B sequences: the first B % world ranks hold one more."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside world of {world}")
    base, extra = divmod(B, world)
    b0 = rank * base + min(rank, extra)
    return b0, b0 + base + (1 if rank < extra else 0)


def stream_rows(B: int, b0: int, b1: int) -> np.ndarray:
    """Global stream ids of a shard, conditional streams first then unconditional (local order)."""
    seq = np.arange(b0, b1)
    return np.concatenate([seq, B + seq])


_PER_STREAM = ("q", "k_cache", "v_cache", "prefix_len", "logits")
_PER_SEQUENCE = ("q_probs", "draft", "u_accept", "u_resample")


def shard_step_inputs(inputs: Dict[str, np.ndarray], B: int, world: int, rank: int) -> Dict[str, np.ndarray]:
    """Slices a dict of whole-batch step inputs down to this rank's sequences.

    Tensors indexed by stream ([2B, ...]) keep the conditional-then-unconditional order locally;
    tensors indexed by sequence ([B, ...]) are sliced; "x" ([2B*K, hidden]) is sliced by stream;
    anything else (the head weight, scalars) is shared.
    """
    b0, b1 = sequence_range(B, world, rank)
    rows = stream_rows(B, b0, b1)
    out = {}
    for name, a in inputs.items():
        if name in _PER_STREAM:
            out[name] = np.ascontiguousarray(a[rows])
        elif name in _PER_SEQUENCE:
            out[name] = np.ascontiguousarray(a[b0:b1])
        elif name == "x":
            K = a.shape[0] // (2 * B)
            out[name] = np.ascontiguousarray(a.reshape(2 * B, K, -1)[rows].reshape(len(rows) * K, -1))
        else:
            out[name] = a
    return out


def gather_results(accept_len, out_token, B: int, group=None):
    """all_gather of the per-sequence results of every rank into whole-batch tensors (torch.distributed)."""
    import torch
    import torch.distributed as dist
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    sizes = [sequence_range(B, world, r) for r in range(world)]
    width = max(b1 - b0 for b0, b1 in sizes)
    mine = torch.full((2, width), -2, dtype=torch.int32, device=accept_len.device)
    n = sizes[rank][1] - sizes[rank][0]
    mine[0, :n] = accept_len
    mine[1, :n] = out_token
    parts = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(parts, mine, group=group)
    lens = torch.cat([p[0, : b1 - b0] for p, (b0, b1) in zip(parts, sizes)])
    toks = torch.cat([p[1, : b1 - b0] for p, (b0, b1) in zip(parts, sizes)])
    return lens, toks
