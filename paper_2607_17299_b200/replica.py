"""Replica-side plumbing for more than one GPU.

The step itself needs no exchange: every rank (one process per GPU = one rollout replica) holds the whole
trajectory index and its own requests and KV cache.  The one exchange the method has is at the end of an RL step,
when every replica must add the trajectories that ALL replicas finished in that step to its own index (the paper's
cross-worker suffix-cache synchronisation, Section 3.3).  `gather_trajectories` does that with plain
`torch.distributed` collectives into each rank's own memory, in rank order, so that every rank appends the same
trajectories in the same order; `append_step_trajectories` then calls the library's `war_index_append`.
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np
import torch
import torch.distributed as dist


def shard_requests(n_requests: int, rank: int, world: int) -> slice:
    """Contiguous, balanced split of a global request list (used when one global batch is dealt to replicas)."""
    base, extra = divmod(n_requests, world)
    start = rank * base + min(rank, extra)
    return slice(start, start + base + (1 if rank < extra else 0))


def gather_trajectories(tokens: np.ndarray, offsets: np.ndarray, device: torch.device | str = "cpu",
                        group: Optional[dist.ProcessGroup] = None) -> Tuple[np.ndarray, np.ndarray]:
    """All-gathers this rank's finished trajectories (flat int32 tokens + int64 offsets[T+1]) from every rank.
    Returns the concatenation in rank order, identical on every rank.  Tensors travel on `device`
    ("cpu" with gloo, the rank's GPU with NCCL)."""
    world = dist.get_world_size(group)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    lens = np.diff(np.asarray(offsets, dtype=np.int64))
    meta = torch.tensor([len(lens), int(lens.sum())], dtype=torch.int64, device=device)
    metas = [torch.zeros_like(meta) for _ in range(world)]
    dist.all_gather(metas, meta, group=group)
    counts = [int(m[0]) for m in metas]
    totals = [int(m[1]) for m in metas]
    max_t, max_n = max(counts + [1]), max(totals + [1])
    pad_len = torch.zeros(max_t, dtype=torch.int64, device=device)
    pad_len[:len(lens)] = torch.from_numpy(lens).to(device)
    pad_tok = torch.zeros(max_n, dtype=torch.int32, device=device)
    pad_tok[:len(tokens)] = torch.from_numpy(tokens).to(device)
    all_len = [torch.zeros_like(pad_len) for _ in range(world)]
    all_tok = [torch.zeros_like(pad_tok) for _ in range(world)]
    dist.all_gather(all_len, pad_len, group=group)
    dist.all_gather(all_tok, pad_tok, group=group)
    out_tok = np.concatenate([all_tok[r][:totals[r]].cpu().numpy() for r in range(world)]).astype(np.int32)
    out_len = np.concatenate([all_len[r][:counts[r]].cpu().numpy() for r in range(world)]).astype(np.int64)
    out_off = np.zeros(len(out_len) + 1, dtype=np.int64)
    out_off[1:] = np.cumsum(out_len)
    return out_tok, out_off


def window_eviction(stored: int, incoming: int, window: int) -> int:
    """How many of the oldest stored trajectories must go so that stored + incoming <= window (a sliding window
    over the trajectory stream; every rank computes the same number because it appends the same trajectories)."""
    if window <= 0:
        return 0
    return max(0, min(stored, stored + incoming - window))


def append_step_trajectories(ix, tokens: np.ndarray, offsets: np.ndarray, device: torch.device,
                             group: Optional[dist.ProcessGroup] = None, window: int = 0) -> Tuple[np.ndarray, np.ndarray]:
    """End-of-step synchronisation on a GPU rank: gather everybody's new trajectories and append them to this rank's
    index; with `window` > 0 the oldest trajectories are evicted first so that at most `window` stay stored."""
    from . import binding as war
    all_tok, all_off = gather_trajectories(tokens, offsets, device, group)
    n_new = len(all_off) - 1
    if n_new > 0:
        if window > 0:
            n_new_kept = min(n_new, window)                       # more new ones than the window holds: keep the latest
            all_tok, all_off = all_tok[all_off[n_new - n_new_kept]:], all_off[n_new - n_new_kept:] - all_off[n_new - n_new_kept]
            n_evict = window_eviction(int(war.war_index_info(ix).T), n_new_kept, window)
            if n_evict:
                war.war_index_evict(ix, n_evict)
        war.war_index_append(ix, torch.from_numpy(np.ascontiguousarray(all_tok)).to(device), all_off)
    return all_tok, all_off
