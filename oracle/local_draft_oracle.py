"""Drafting from the request's own context, and the choice between two draft trees (test infrastructure).

The SuffixDecoding method that the paper adopts (Section 3.3: a cache of the token patterns of earlier
trajectories) keeps, besides the cache of finished trajectories, the tokens of the running request itself:
text that a rollout has produced or read once (a file, a tool result) tends to come back inside the same trajectory.
The paper does not spell this part out; the rules below are this build's reading and are listed in the design notes.

  match   the largest l <= min(P, tail_len, L - 1) such that the last l tokens of the context c[0..L) also occur
          ending at an earlier position e <= L - 2 (so the occurrence has at least one token after it inside the
          context); occurrences may overlap each other and the tail itself.  Tokens < 0 never match.
  window  of all occurrences of that longest suffix only the `max_occ` most recent ones (largest e) are used.
  tree    exactly the rules of the cross-trajectory draft (`draft_oracle.build_draft_tree`), with the context as the
          only trajectory and the window as the occurrence list: count = number of window occurrences followed by
          the slot's root path inside the context; k most frequent continuations per node (count desc, token asc);
          slots best-first (count desc, parent slot asc, token asc); node budget and probability threshold alike.

  pick    between two trees of one request (e.g. cross-trajectory and own-context): score = (sum of count[1:]) /
          count[0], the expected number of accepted draft tokens under the tree's own statistics; the second tree
          wins only with a strictly larger score (exact fractions).

Two implementations of the draft live here: a definitional one (nested Python loops, explicit re-scan per path) for
tiny inputs, and the one used at realistic sizes, which reuses the cross-trajectory tree builder on a one-trajectory
corpus.  The tests hold them against each other and against a hand-worked example.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np

from . import draft_oracle as D

MAX_OCC = 32


def local_occurrences(ctx: np.ndarray, l: int) -> np.ndarray:
    """End positions e <= L - 2 of the occurrences of the last l tokens of ctx (plain scan, ascending)."""
    L = len(ctx)
    if l <= 0 or l > L - 1:
        return np.zeros(0, np.int64)
    pat = ctx[L - l:]
    if (pat < 0).any():
        return np.zeros(0, np.int64)
    ends = np.arange(l - 1, L - 1, dtype=np.int64)
    for i in range(l):                                     # token i counted from the end of the pattern
        ends = ends[ctx[ends - i] == pat[l - 1 - i]]
    return ends


def local_match(ctx: np.ndarray, P: int, tail_len: int) -> Tuple[int, np.ndarray]:
    """(match_len, window): the longest suffix that occurs earlier, and the ends of its MAX_OCC most recent occurrences."""
    L = len(ctx)
    best, ends = 0, np.zeros(0, np.int64)
    for l in range(1, min(P, tail_len, L - 1) + 1):        # occurrence is monotone in l: stop at the first miss
        e = local_occurrences(ctx, l)
        if len(e) == 0:
            break
        best, ends = l, e
    return best, ends[-MAX_OCC:]


def draft_local(ctx: np.ndarray, P: int, tail_len: int, N: int, k: int, min_match: int = 1, spec_factor=(0, 1),
                min_prob=(0, 1)):
    """Returns (match_len, ids, parent, count) of the own-context draft; root id = last context token."""
    ctx = np.ascontiguousarray(ctx, dtype=np.int32)
    L = len(ctx)
    ml, window = local_match(ctx, P, tail_len)
    # a token < 0 is a trajectory of its own: nothing matches it and no continuation runs into it
    cuts = sorted({0, L} | {int(p) for p in np.flatnonzero(ctx < 0)} | {int(p) + 1 for p in np.flatnonzero(ctx < 0)})
    one = D.Corpus(ctx, np.array(cuts, dtype=np.int64))
    tail = ctx[-1:] if L else np.zeros(1, np.int32)
    ids, parent, count = D.build_draft_tree(one, tail, ml, window, N, k, min_match, spec_factor, min_prob)
    return ml, ids, parent, count


def draft_local_definitional(ctx: Sequence[int], P: int, tail_len: int, N: int, k: int, min_match: int = 1):
    """The same by nested loops over plain lists (tiny inputs; no thresholds)."""
    c = [int(x) for x in ctx]
    L = len(c)
    ml, occ = 0, []
    for l in range(1, min(P, tail_len, L - 1) + 1):
        pat = c[L - l:]
        found = [e for e in range(l - 1, L - 1) if c[e - l + 1:e + 1] == pat and min(pat) >= 0]
        if found:
            ml, occ = l, found
    occ = sorted(occ)[-MAX_OCC:]
    ids, parent, count, paths = [c[-1] if L else 0], [-1], [len(occ) if ml > 0 else 0], [[]]
    if ml < max(1, min_match) or N <= 1:
        return ml, ids, parent, count

    def cnt_of(path):                                       # a path never holds a token < 0, so it never crosses one
        return sum(1 for e in occ if e + len(path) <= L - 1 and c[e + 1:e + 1 + len(path)] == path)

    def offers(slot):
        cand = []
        for x in sorted({t for t in c if t >= 0}):
            n = cnt_of(paths[slot] + [x])
            if n > 0:
                cand.append((-n, x))
        cand.sort()
        return [(-a, slot, x) for a, x in cand[:k]]

    frontier = offers(0)
    while len(ids) < N and frontier:
        frontier.sort(key=lambda e: (-e[0], e[1], e[2]))
        n, p, x = frontier.pop(0)
        ids.append(x); parent.append(p); count.append(n)
        paths.append(paths[p] + [x])
        frontier.extend(offers(len(ids) - 1))
    return ml, ids, parent, count


def draft_local_batch(ctx: np.ndarray, ctx_off: np.ndarray, tail_len: np.ndarray, P: int, N: int, k: int, min_match: int = 1,
                      spec_batch_limit: int = 0, spec_factor=(0, 1), min_prob=(0, 1)):
    """Batched form with the library's output convention and the workload-aware switch of `draft_oracle.draft_batch`."""
    B = len(ctx_off) - 1
    match_len = np.zeros(B, np.int32)
    num_nodes = np.zeros(B, np.int32)
    ids = np.full((B, N), -1, np.int32)
    parent = np.full((B, N), -1, np.int32)
    count = np.zeros((B, N), np.int32)
    running = [i for i in range(B) if int(tail_len[i]) >= 0]
    plain = spec_batch_limit > 0 and len(running) > spec_batch_limit
    for i in running:
        c = ctx[ctx_off[i]:ctx_off[i + 1]]
        if plain or len(c) == 0:
            num_nodes[i] = 1
            ids[i, 0] = c[-1] if len(c) else -1
            continue
        ml, a, b, n = draft_local(c, P, int(tail_len[i]), N, k, min_match, spec_factor, min_prob)
        match_len[i], num_nodes[i] = ml, len(a)
        ids[i, :len(a)], parent[i, :len(a)], count[i, :len(a)] = a, b, n
    return match_len, num_nodes, ids, parent, count


def pick_by_score(a, b):
    """a, b: (match_len, num_nodes, ids, parent, count) batches of the same shape.  Per request the second tree is
    taken only if its score is strictly larger.  Returns (source [B] 0/1, match_len, num_nodes, ids, parent, count)."""
    B = len(a[0])
    src = np.zeros(B, np.int32)
    out = [x.copy() for x in a]
    for i in range(B):
        na, nb = int(a[1][i]), int(b[1][i])
        sa = (int(a[4][i, 1:na].sum()), int(a[4][i, 0])) if na > 0 else (0, 0)
        sb = (int(b[4][i, 1:nb].sum()), int(b[4][i, 0])) if nb > 0 else (0, 0)
        # num_b / den_b > num_a / den_a, a zero denominator scoring 0
        lhs = sb[0] * max(sa[1], 1) if sb[1] > 0 else 0
        rhs = sa[0] * max(sb[1], 1) if sa[1] > 0 else 0
        if lhs > rhs:
            src[i] = 1
            for o, x in zip(out, b):
                o[i] = x[i]
    return (src, *out)
