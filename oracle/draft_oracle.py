"""Longest-suffix match and draft-tree construction by brute force (test infrastructure).

What is computed (paper, Section 3: SuffixDecoding keeps the trajectories generated so far and drafts by
matching the request's current tokens against them; Section 3.3: the cache holds the token patterns of earlier
trajectories, and likely next tokens are predicted from them):

  match   the largest l <= min(P, tail_len) such that the last l context tokens occur contiguously inside
          ONE stored trajectory (occurrences never straddle two trajectories);
  tree    slot 0 is the root (the last context token).  Every other slot is one continuation token of the
          matched string; count = number of occurrences (with multiplicity, overlaps included, over all
          trajectories) of matched string + root path.  Each node offers its k most frequent continuations
          (count descending, then token id ascending); slots are created best-first from the pool of
          offered continuations (count descending, then parent slot ascending, then token id ascending)
          until N slots exist or nothing is offered.

The paper fixes none of the tie rules or the node budget convention; the rules above are this build's
reading and are listed in the design notes.  No suffix tree or suffix array appears here on purpose.

Two implementations live side by side:
  * `*_definitional`: nested pure-Python loops straight from the definition, for tiny inputs;
  * the numpy versions used at realistic sizes, which filter explicit occurrence lists.
They are written differently (re-scan per candidate string vs. filtering), and the tests hold them against
each other, against hand-worked examples and against invariants.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


# ----------------------------------------------------------------------------------------------
# definitional versions (tiny inputs only)
# ----------------------------------------------------------------------------------------------

def occurrences_definitional(trajs: Sequence[Sequence[int]], s: Sequence[int]) -> List[Tuple[int, int]]:
    """All (t, p) with trajs[t][p : p+len(s)] == s."""
    s = [int(x) for x in s]
    out = []
    for t, tr in enumerate(trajs):
        tr = [int(x) for x in tr]
        for p in range(0, len(tr) - len(s) + 1):
            if tr[p:p + len(s)] == s:
                out.append((t, p))
    return out


def match_definitional(trajs, tail: Sequence[int], tail_len: int) -> int:
    """Largest l <= tail_len whose suffix of the tail occurs; every l is tested, nothing is assumed monotone."""
    P = len(tail)
    best = 0
    for l in range(1, tail_len + 1):
        if occurrences_definitional(trajs, tail[P - l:]):
            best = l
    return best


def draft_definitional(trajs, tail: Sequence[int], tail_len: int, N: int, k: int, min_match: int = 1):
    """Returns (match_len, ids, parent, count) as Python lists of length num_nodes."""
    P = len(tail)
    tail = [int(x) for x in tail]
    ml = match_definitional(trajs, tail, tail_len)
    s = tail[P - ml:] if ml > 0 else []
    ids, parent, count = [tail[P - 1]], [-1], [len(occurrences_definitional(trajs, s)) if ml > 0 else 0]
    if ml < max(1, min_match) or N <= 1:
        return ml, ids, parent, count
    alphabet = sorted({int(x) for tr in trajs for x in tr})
    paths = [[]]

    def offers(slot):
        cand = []
        for x in alphabet:
            c = len(occurrences_definitional(trajs, s + paths[slot] + [x]))
            if c > 0:
                cand.append((-c, x))
        cand.sort()
        return [(-negc, slot, x) for negc, x in cand[:k]]

    frontier = offers(0)
    while len(ids) < N and frontier:
        frontier.sort(key=lambda e: (-e[0], e[1], e[2]))
        c, p, x = frontier.pop(0)
        ids.append(x); parent.append(p); count.append(c)
        paths.append(paths[p] + [x])
        frontier.extend(offers(len(ids) - 1))
    return ml, ids, parent, count


# ----------------------------------------------------------------------------------------------
# numpy versions
# ----------------------------------------------------------------------------------------------

class Corpus:
    """The stored trajectories, kept as one flat array plus, for every flat position, the flat bounds of the
    trajectory that position belongs to.  This is bookkeeping, not an index: every query scans all tokens."""

    def __init__(self, tokens: np.ndarray, offsets: np.ndarray):
        self.tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        self.offsets = np.asarray(offsets, dtype=np.int64)
        lens = np.diff(self.offsets)
        self.start_of = np.repeat(self.offsets[:-1], lens)
        self.end_of = np.repeat(self.offsets[1:], lens)

    @classmethod
    def from_lists(cls, trajs):
        lens = [len(t) for t in trajs]
        off = np.zeros(len(trajs) + 1, dtype=np.int64)
        off[1:] = np.cumsum(lens)
        tok = np.concatenate([np.asarray(t, dtype=np.int32) for t in trajs]) if trajs else np.zeros(0, np.int32)
        return cls(tok, off)


def longest_suffix_match(corpus: Corpus, tail: np.ndarray, tail_len: int) -> Tuple[int, np.ndarray]:
    """Returns (match_len, ends): `ends` are the flat positions of the LAST token of every occurrence of the
    longest occurring suffix.  Occurrence is monotone in the suffix length (dropping the first token of an
    occurring string leaves an occurring string), so the scan grows l until no occurrence survives."""
    P = len(tail)
    tok = corpus.tokens
    if tail_len <= 0 or len(tok) == 0:
        return 0, np.zeros(0, dtype=np.int64)
    ends = np.flatnonzero(tok == tail[P - 1]).astype(np.int64)
    if len(ends) == 0:
        return 0, ends
    l = 1
    while l < tail_len:
        first = ends - l                                  # where the (l+1)-token suffix would start
        inside = first >= corpus.start_of[ends]
        keep = np.zeros(len(ends), dtype=bool)
        keep[inside] = tok[first[inside]] == tail[P - 1 - l]
        if not keep.any():
            break
        ends = ends[keep]
        l += 1
    return l, ends


def build_draft_tree(corpus: Corpus, tail: np.ndarray, match_len: int, ends: np.ndarray, N: int, k: int,
                     min_match: int = 1, spec_factor=(0, 1), min_prob=(0, 1)):
    """Returns (ids, parent, count) int32 arrays of length num_nodes (see module docstring for the rules).

    Two thresholds of the SuffixDecoding method the paper builds on (Section 3.3 takes that method's code base;
    the paper itself names neither), both exact integer rules:
      spec_factor (a, b), a > 0: the tree has at most 1 + floor(match_len * a / b) slots (a longer match earns a
                  larger tree); (0, .) = no such cap.
      min_prob (a, b), a > 0:    a continuation is offered only if count(child) * b >= a * count(parent), i.e. its
                  empirical probability after the parent's string is at least a / b; (0, .) = every one is."""
    P = len(tail)
    if spec_factor[0] > 0:
        N = min(N, 1 + (match_len * spec_factor[0]) // spec_factor[1])
    tok = corpus.tokens
    ids, parent, count = [int(tail[P - 1])], [-1], [int(len(ends)) if match_len > 0 else 0]
    if match_len < max(1, min_match) or N <= 1:
        return np.array(ids, np.int32), np.array(parent, np.int32), np.array(count, np.int32)
    # per slot: flat positions of the token that FOLLOWS each occurrence of matched string + path, and the
    # flat end of the trajectory that occurrence lives in
    nxt = [ends + 1]
    lim = [corpus.end_of[ends]]

    def offers(slot):
        has_next = nxt[slot] < lim[slot]
        t = tok[nxt[slot][has_next]]
        if len(t) == 0:
            return []
        uniq, cnt = np.unique(t, return_counts=True)
        order = np.lexsort((uniq, -cnt))[:k]              # count descending, token id ascending
        return [(int(cnt[o]), slot, int(uniq[o])) for o in order
                if min_prob[0] == 0 or int(cnt[o]) * min_prob[1] >= min_prob[0] * len(nxt[slot])]

    frontier = offers(0)
    while len(ids) < N and frontier:
        best = min(range(len(frontier)), key=lambda e: (-frontier[e][0], frontier[e][1], frontier[e][2]))
        c, p, x = frontier.pop(best)
        has_next = nxt[p] < lim[p]
        sel = np.zeros(len(nxt[p]), dtype=bool)
        sel[has_next] = tok[nxt[p][has_next]] == x
        ids.append(x); parent.append(p); count.append(c)
        nxt.append(nxt[p][sel] + 1)
        lim.append(lim[p][sel])
        assert len(nxt[-1]) == c
        frontier.extend(offers(len(ids) - 1))
    return np.array(ids, np.int32), np.array(parent, np.int32), np.array(count, np.int32)


def suffix_occurrences(corpus: Corpus, tail: np.ndarray, l: int) -> np.ndarray:
    """Flat positions of the LAST token of every occurrence of the last l tokens of the tail (one plain scan per
    token of the suffix, written on its own rather than through `longest_suffix_match`)."""
    P = len(tail)
    tok = corpus.tokens
    ends = np.arange(len(tok), dtype=np.int64)
    for i in range(l):                                    # token i counted from the end of the suffix
        at = ends - i
        ok = at >= corpus.start_of[ends]
        ok[ok] = tok[at[ok]] == tail[P - 1 - i]
        ends = ends[ok]
    return ends


def tree_score(count: np.ndarray) -> Tuple[int, int]:
    """Score of a draft tree as an exact fraction (numerator, denominator) = (sum of the counts of slots 1.., count
    of the root).  count(slot) / count(root) is the empirical probability that the text continues with the slot's
    whole root path, so the fraction is the number of draft tokens one expects to be accepted if the continuation is
    drawn from the occurrences of the matched string.  The SuffixDecoding method scores candidate trees by the sum
    of such path probabilities (the product of the per-node probabilities along a path telescopes to this ratio)."""
    return int(np.sum(count[1:], dtype=np.int64)), int(count[0])


def draft_scored(corpus: Corpus, tail: np.ndarray, tail_len: int, N: int, k: int, n_lengths: int, min_match: int = 1,
                 spec_factor=(0, 1), min_prob=(0, 1)):
    """Draft from the best-scoring of several suffix lengths instead of from the longest match alone (a variant of
    the SuffixDecoding method the paper adopts in Section 3.3; the paper itself does not spell it out).

    Candidates are the lengths match_len, match_len - 1, ..., down n_lengths of them, never below max(1, min_match)
    (every shorter suffix of an occurring string occurs too).  Each candidate gets its own tree by the rules of
    `build_draft_tree` (its own root interval, its own node budget under spec_factor).  The tree with the largest
    `tree_score` wins; fractions are compared exactly (cross-multiplied integers); equal scores go to the longer
    suffix.  Returns (match_len, used_len, ids, parent, count): match_len is the longest match, used_len the
    length the returned tree was built from."""
    ml, _ = longest_suffix_match(corpus, tail, tail_len)
    best = None
    for c in range(max(1, n_lengths)):
        l = ml - c
        if c > 0 and l < max(1, min_match):
            break
        ends = suffix_occurrences(corpus, tail, l) if l > 0 else np.zeros(0, np.int64)
        tree = build_draft_tree(corpus, tail, l, ends, N, k, min_match, spec_factor, min_prob)
        num, den = tree_score(tree[2])
        if best is None or num * best[1] > best[0] * den:          # strictly better only: ties keep the longer suffix
            best = (num, den, l, tree)
    _, _, used, (ids, parent, count) = best
    return ml, used, ids, parent, count


def draft_scored_batch(corpus: Corpus, tails: np.ndarray, tail_len: np.ndarray, N: int, k: int, n_lengths: int,
                       min_match: int = 1, spec_batch_limit: int = 0, spec_factor=(0, 1), min_prob=(0, 1)):
    """Batched `draft_scored` with the library's output convention and the same switch as `draft_batch`
    (used_len is 0 wherever no tree is built)."""
    B = tails.shape[0]
    match_len = np.zeros(B, np.int32)
    used_len = np.zeros(B, np.int32)
    num_nodes = np.zeros(B, np.int32)
    ids = np.full((B, N), -1, np.int32)
    parent = np.full((B, N), -1, np.int32)
    count = np.zeros((B, N), np.int32)
    running = [i for i in range(B) if int(tail_len[i]) >= 0]
    plain = spec_batch_limit > 0 and len(running) > spec_batch_limit
    for i in running:
        if plain:
            num_nodes[i] = 1
            ids[i, 0] = tails[i, -1]
            continue
        ml, used, a, b, c = draft_scored(corpus, tails[i], int(tail_len[i]), N, k, n_lengths, min_match, spec_factor, min_prob)
        n = len(a)
        match_len[i], used_len[i], num_nodes[i] = ml, used, n
        ids[i, :n], parent[i, :n], count[i, :n] = a, b, c
    return match_len, used_len, num_nodes, ids, parent, count


def draft_batch(corpus: Corpus, tails: np.ndarray, tail_len: np.ndarray, N: int, k: int, min_match: int = 1,
                spec_batch_limit: int = 0, spec_factor=(0, 1), min_prob=(0, 1)):
    """Batched form with the library's output convention: unused slots hold ids = -1, parent = -1, count = 0.

    Workload-aware switch (paper, Section 3.3: speculation is switched on and off by the current batch size, and
    Section 5.3: beyond a batch of about 16 speculation costs more than it gains): a request with
    tail_len < 0 is not running (no tree at all); the effective batch size is the number of running requests;
    when spec_batch_limit > 0 and the effective batch size exceeds it, nothing is looked up and every running
    request gets the root alone (match_len 0, count 0), which makes the step a plain decode step."""
    B = tails.shape[0]
    match_len = np.zeros(B, np.int32)
    num_nodes = np.zeros(B, np.int32)
    ids = np.full((B, N), -1, np.int32)
    parent = np.full((B, N), -1, np.int32)
    count = np.zeros((B, N), np.int32)
    running = [i for i in range(B) if int(tail_len[i]) >= 0]
    plain = spec_batch_limit > 0 and len(running) > spec_batch_limit
    for i in running:
        if plain:
            num_nodes[i] = 1
            ids[i, 0] = tails[i, -1]
            continue
        ml, ends = longest_suffix_match(corpus, tails[i], int(tail_len[i]))
        a, b, c = build_draft_tree(corpus, tails[i], ml, ends, N, k, min_match, spec_factor, min_prob)
        n = len(a)
        match_len[i], num_nodes[i] = ml, n
        ids[i, :n], parent[i, :n], count[i, :n] = a, b, c
    return match_len, num_nodes, ids, parent, count
