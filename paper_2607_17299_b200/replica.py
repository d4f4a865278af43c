"""Replica-side plumbing for more than one GPU.

The step itself needs no exchange: every rank (one process per GPU = one rollout replica) holds the whole
trajectory index and its own requests and KV cache.  The one exchange the method has is at the end of an RL step,
when every replica must add the trajectories that ALL replicas finished in that step to its own index (the paper's
cross-worker suffix-cache synchronisation, Section 3.3: the finished prompt-response sequences go to every rollout
worker, off the critical path of training).  `gather_trajectories` does that with plain `torch.distributed`
collectives into each rank's OWN memory (NCCL all-gather on the GPU, gloo on the CPU), in rank order, so that every
rank appends the same trajectories in the same order; `append_step_trajectories` then calls the library's
`war_index_append` on the gathered tokens, which never leave the device.

Inside one replica, tensor-parallel ranks need no exchange for the verification either: kv heads are independent
problems, so rank r calls `war_verify_attn` on its own slice of the q heads and of the KV pools (`kv_head_shard`).
"""
from __future__ import annotations

from typing import Optional, Tuple

import numpy as np
import torch
import torch.distributed as dist


def _world(group) -> int:
    return dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1


def shard_requests(n_requests: int, rank: int, world: int) -> slice:
    """Contiguous, balanced split of a global request list (used when one global batch is dealt to replicas)."""
    base, extra = divmod(n_requests, world)
    start = rank * base + min(rank, extra)
    return slice(start, start + base + (1 if rank < extra else 0))


def kv_head_shard(n_kv_heads: int, rank: int, world: int) -> slice:
    """The kv heads a tensor-parallel rank verifies (its q heads are the groups of exactly these kv heads)."""
    if n_kv_heads % world:
        raise ValueError("the kv heads must divide evenly among the tensor-parallel ranks")
    per = n_kv_heads // world
    return slice(rank * per, (rank + 1) * per)


def gather_trajectories(tokens, offsets: np.ndarray, device: torch.device | str = "cpu",
                        group: Optional[dist.ProcessGroup] = None) -> Tuple[torch.Tensor, np.ndarray]:
    """All-gathers this rank's finished trajectories (flat int32 tokens, a numpy array or a tensor on `device`, and
    int64 offsets[T+1] on the host) from every rank.  Returns (tokens, offsets) of the concatenation in rank order,
    identical on every rank: the tokens as an int32 tensor on `device` ("cpu" with gloo, the rank's GPU with NCCL;
    they are gathered there and stay there), the offsets as a host array (the library wants them on the host).
    Without an initialised process group the world is this rank alone."""
    world = _world(group)
    tok = tokens if isinstance(tokens, torch.Tensor) else torch.from_numpy(np.ascontiguousarray(tokens, dtype=np.int32))
    tok = tok.to(device=device, dtype=torch.int32)
    lens = np.diff(np.asarray(offsets, dtype=np.int64))
    if int(lens.sum()) != tok.numel():
        raise ValueError("offsets do not describe the token array")
    if world == 1:
        off = np.zeros(len(lens) + 1, dtype=np.int64)
        off[1:] = np.cumsum(lens)
        return tok.contiguous(), off
    # 1. how much everybody brings (two numbers per rank)
    meta = torch.tensor([len(lens), int(lens.sum())], dtype=torch.int64, device=device)
    metas = torch.zeros(world * 2, dtype=torch.int64, device=device)
    dist.all_gather_into_tensor(metas, meta, group=group)
    metas = metas.cpu().numpy().reshape(world, 2)
    counts, totals = metas[:, 0], metas[:, 1]
    max_t, max_n = int(max(counts.max(), 1)), int(max(totals.max(), 1))
    # 2. lengths and tokens, padded to the largest contribution so that one all-gather moves each
    pad_len = torch.zeros(max_t, dtype=torch.int64, device=device)
    pad_len[:len(lens)] = torch.from_numpy(lens).to(device)
    pad_tok = torch.zeros(max_n, dtype=torch.int32, device=device)
    pad_tok[:tok.numel()] = tok
    all_len = torch.zeros(world * max_t, dtype=torch.int64, device=device)
    all_tok = torch.zeros(world * max_n, dtype=torch.int32, device=device)
    dist.all_gather_into_tensor(all_len, pad_len, group=group)
    dist.all_gather_into_tensor(all_tok, pad_tok, group=group)
    # 3. drop the padding: tokens on the device, lengths on the host
    out_tok = torch.cat([all_tok[r * max_n:r * max_n + int(totals[r])] for r in range(world)])
    h_len = all_len.cpu().numpy().reshape(world, max_t)
    out_len = np.concatenate([h_len[r, :int(counts[r])] for r in range(world)]).astype(np.int64)
    out_off = np.zeros(len(out_len) + 1, dtype=np.int64)
    out_off[1:] = np.cumsum(out_len)
    return out_tok, out_off


def window_eviction(stored: int, incoming: int, window: int) -> int:
    """How many of the oldest stored trajectories must go so that stored + incoming <= window (a sliding window
    over the trajectory stream; every rank computes the same number because it appends the same trajectories)."""
    if window <= 0:
        return 0
    return max(0, min(stored, stored + incoming - window))


def append_step_trajectories(ix, tokens, offsets: np.ndarray, device: torch.device,
                             group: Optional[dist.ProcessGroup] = None, window: int = 0) -> Tuple[torch.Tensor, np.ndarray]:
    """End-of-step synchronisation on a GPU rank: gather everybody's new trajectories (on the device) and append them
    to this rank's index; with `window` > 0 the oldest trajectories are evicted first so that at most `window` stay
    stored.  Returns what was gathered (device tokens, host offsets)."""
    from . import binding as war
    all_tok, all_off = gather_trajectories(tokens, offsets, device, group)
    n_new = len(all_off) - 1
    if n_new > 0:
        if window > 0:
            n_new_kept = min(n_new, window)                       # more new ones than the window holds: keep the latest
            first = int(all_off[n_new - n_new_kept])
            all_tok, all_off = all_tok[first:].contiguous(), all_off[n_new - n_new_kept:] - first
            n_evict = window_eviction(int(war.war_index_info(ix).T), n_new_kept, window)
            if n_evict:
                war.war_index_evict(ix, n_evict)
        war.war_index_append(ix, all_tok.contiguous(), all_off)
    return all_tok, all_off
