"""Longest accepted root path by enumeration (test infrastructure).

Verification is lossless (paper, Section 2.3: checking the drafts leaves the target model's output distribution
as it is; Section 3.3: a request moves ahead by several tokens per forward pass whenever drafts are accepted): the
step may only emit tokens the target model itself chose.  With the target's
choices supplied as ids, a draft slot is accepted exactly when every slot on its root path equals the
target's choice at that point.

  mode 0 (per slot): target[p] is the token the target emits AFTER slot p; slot j matches when
                     ids[j] == target[parent[j]].  bonus = target[result slot] (the next real token).
  mode 1 (per node): slot j matches when ids[j] == target[j].  bonus = -1.

Result slot = the deepest slot whose whole root path matches (ties: the lowest slot index); accept_len is its
depth (root = 0) and accept_path the slots from the root's child down to it.
"""
from __future__ import annotations

import numpy as np


def accept_request(ids, parent, n: int, target, mode: int):
    """Enumerates every root-to-slot path.  Returns (accept_len, path list, bonus)."""
    best_depth, best_slot, best_path = -1, -1, []
    for r in range(n):
        path = []
        a = r
        while a > 0:
            path.append(a)
            a = int(parent[a])
        path.reverse()                                     # slots below the root, top-down
        ok = True
        for j in path:
            want = int(target[parent[j]]) if mode == 0 else int(target[j])
            if int(ids[j]) != want:
                ok = False
                break
        if ok and len(path) > best_depth:
            best_depth, best_slot, best_path = len(path), r, path
    if n == 0:
        return 0, [], -1
    bonus = int(target[best_slot]) if mode == 0 else -1
    return best_depth, best_path, bonus


def accept_batch(ids, parent, num_nodes, target, mode: int = 0):
    """Library convention: accept_path rows are filled with -1 beyond accept_len."""
    B, N = ids.shape
    alen = np.zeros(B, np.int32)
    path = np.full((B, N), -1, np.int32)
    bonus = np.full(B, -1, np.int32)
    for i in range(B):
        l, p, b = accept_request(ids[i], parent[i], int(num_nodes[i]), target[i], mode)
        alen[i], bonus[i] = l, b
        path[i, :l] = p
    return alen, path, bonus
