"""Advancing a request by its accepted tokens, written out plainly (test infrastructure).

A speculate-and-verify step ends by making the accepted tokens part of the request (paper, Section 3.3: with accepted
drafts a request moves ahead by several tokens in one forward pass; Section 2.3: the rejected drafts leave no trace,
the output is the target model's own).  The paper does not spell the
bookkeeping out; this is the reading used here, in the slot convention of the draft tree (slot 0 = the
request's last context token, whose K/V sits at logical position prefix_len, slot j at prefix_len + j):

  * context:   context' = context ++ ids[path[0]] ++ ... ++ ids[path[k-1]] (++ bonus, when the target supplied one)
  * KV cache:  the K/V rows of the accepted slots become positions prefix_len + 1 .. prefix_len + k, in path
               order; rows of rejected slots are dead (whatever is beyond the new end is unspecified)
  * root:      the last token of context' is the next step's root.  With a bonus token its K/V does not exist
               yet: prefix_len' = prefix_len + k + 1.  Without one (per-node targets) the last accepted token, or
               the old root when k = 0, stays the root: prefix_len' = prefix_len + k.
  * tail:      the last P tokens of context', right-aligned; tail_len' = min(P, tail_len + tokens added).

Only tests/, the smoke check and the timed CPU baseline may import this module.
"""
from __future__ import annotations

import numpy as np


def commit_request(kv_k: np.ndarray, kv_v: np.ndarray, prefix_len: int, ids, accept_len: int, accept_path, bonus: int,
                   tail: np.ndarray, tail_len: int):
    """kv_k / kv_v: dense [positions, Hkv, D] arrays of one request, positions >= prefix_len + N.
    Returns (kv_k', kv_v', prefix_len', tail', tail_len'); rows from prefix_len' + (0 if bonus given else 1) on are
    whatever they were (callers compare only the live part)."""
    k = int(accept_len)
    P = len(tail)
    new_k, new_v = kv_k.copy(), kv_v.copy()
    for d in range(k):                                   # path order; sources are read from the untouched copy
        src = prefix_len + int(accept_path[d])
        new_k[prefix_len + 1 + d] = kv_k[src]
        new_v[prefix_len + 1 + d] = kv_v[src]
    added = [int(ids[int(accept_path[d])]) for d in range(k)]
    if bonus >= 0:
        added.append(int(bonus))
    context_tail = [int(x) for x in tail[P - tail_len:]] + added
    new_len = min(P, len(context_tail))
    new_tail = np.zeros(P, dtype=np.int32)
    if new_len:
        new_tail[P - new_len:] = context_tail[-new_len:]
    new_prefix = prefix_len + k + (1 if bonus >= 0 else 0)
    return new_k, new_v, new_prefix, new_tail, new_len


def live_positions(prefix_len_after: int, has_bonus: bool) -> int:
    """Number of leading positions of the cache that hold defined K/V after a commit."""
    return prefix_len_after if has_bonus else prefix_len_after + 1
