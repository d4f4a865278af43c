"""Pins for the brute-force match / draft-tree checker: hand-worked cases, a definitional brute force written
differently, and invariants that hold by construction of the definition."""
import json
import os

import numpy as np
import pytest

from oracle import draft_oracle as D
from paper_2607_17299_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _load(name):
    with open(os.path.join(GOLD, name)) as f:
        return json.load(f)


def _window_occurrences(tokens, offsets, s):
    """Independent count: sliding windows per trajectory (no shared code with the checker)."""
    s = np.asarray(s, dtype=np.int32)
    out = []
    for t in range(len(offsets) - 1):
        tr = tokens[offsets[t]:offsets[t + 1]]
        if len(tr) < len(s):
            continue
        win = np.lib.stride_tricks.sliding_window_view(tr, len(s))
        for p in np.flatnonzero((win == s).all(axis=1)):
            out.append((t, int(p)))
    return out


@pytest.mark.parametrize("name", ["draft_case1.json", "draft_case2.json"])
def test_hand_worked_cases(name):
    g = _load(name)
    trajs = g["trajectories"]
    tail = np.array(g["tail"], dtype=np.int32)
    corpus = D.Corpus.from_lists(trajs)
    ml, ends = D.longest_suffix_match(corpus, tail, g["tail_len"])
    assert ml == g["match_len"]
    # occurrences: end position -> (t, p)
    occ = sorted((int(np.searchsorted(corpus.offsets, e, side="right") - 1),
                  int(e - (ml - 1) - corpus.start_of[e])) for e in ends)
    assert occ == sorted(map(tuple, g["occurrences"]))
    assert D.match_definitional(trajs, g["tail"], g["tail_len"]) == g["match_len"]
    for tr in g["trees"]:
        ids, parent, count = D.build_draft_tree(corpus, tail, ml, ends, tr["N"], tr["k"])
        assert ids.tolist() == tr["ids"]
        assert parent.tolist() == tr["parent"]
        assert count.tolist() == tr["count"]
        ml2, i2, p2, c2 = D.draft_definitional(trajs, g["tail"], g["tail_len"], tr["N"], tr["k"])
        assert (ml2, i2, p2, c2) == (g["match_len"], tr["ids"], tr["parent"], tr["count"])


@pytest.mark.parametrize("seed", range(40))
def test_numpy_version_equals_definitional_on_tiny_alphabets(seed):
    """Vocabularies of 2-5 symbols and corpora under 200 tokens force heavy count ties, so the
    (count, parent slot, token) ordering rules are exercised on almost every slot."""
    rng = np.random.default_rng(seed)
    vocab = int(rng.integers(2, 6))
    trajs = [rng.integers(0, vocab, size=int(rng.integers(1, 40))).tolist() for _ in range(int(rng.integers(1, 6)))]
    corpus = D.Corpus.from_lists(trajs)
    P = int(rng.integers(1, 9))
    N = int(rng.integers(1, 20))
    k = int(rng.integers(1, 5))
    for _ in range(5):
        tail = rng.integers(0, vocab + 1, size=P).astype(np.int32)     # vocab itself never occurs
        tail_len = int(rng.integers(0, P + 1))
        ml, ends = D.longest_suffix_match(corpus, tail, tail_len)
        ids, parent, count = D.build_draft_tree(corpus, tail, ml, ends, N, k)
        ml2, i2, p2, c2 = D.draft_definitional(trajs, tail.tolist(), tail_len, N, k)
        assert ml == ml2
        assert ids.tolist() == i2 and parent.tolist() == p2 and count.tolist() == c2


@pytest.fixture(scope="module")
def tiny():
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    # add structured tails: planted copies, out-of-vocabulary, short tail_len
    rng = np.random.default_rng(5)
    extra, extra_len, planted = [], [], []
    for _ in range(6):
        t = int(rng.integers(0, cfg.n_traj))
        dist = int(rng.integers(1, 200))                     # tokens from the trajectory start to the tail's end
        e = int(off[t]) + dist
        m = min(cfg.P, dist)
        row = np.full(cfg.P, -1, np.int32)
        row[cfg.P - m:] = tok[e - m:e]
        extra.append(row); extra_len.append(m); planted.append(min(cfg.P, dist))
    extra.append(np.full(cfg.P, cfg.vocab + 5, np.int32)); extra_len.append(cfg.P); planted.append(-1)
    short = tails[0].copy(); extra.append(short); extra_len.append(3); planted.append(-1)
    tails = np.concatenate([tails, np.stack(extra)])
    tl = np.concatenate([tl, np.array(extra_len, np.int32)])
    return cfg, tok, off, tails, tl, planted


def test_match_invariants_on_tiny_workload(tiny):
    cfg, tok, off, tails, tl, planted = tiny
    corpus = D.Corpus(tok, off)
    B0 = cfg.B
    for i in range(len(tails)):
        ml, ends = D.longest_suffix_match(corpus, tails[i], int(tl[i]))
        assert 0 <= ml <= tl[i]
        if ml > 0:
            s = tails[i, cfg.P - ml:]
            occ = _window_occurrences(tok, off, s)
            assert len(occ) == len(ends) > 0                 # it occurs, and the count is the brute-force count
            for e in ends[:50]:                              # reported places really hold the string
                assert (tok[e - ml + 1:e + 1] == s).all()
                assert e - ml + 1 >= corpus.start_of[e]
        if ml < tl[i]:                                       # no longer match exists (full independent scan)
            assert _window_occurrences(tok, off, tails[i, cfg.P - ml - 1:]) == []
        for l in range(1, ml):                               # monotone: every shorter suffix occurs too
            assert len(_window_occurrences(tok, off, tails[i, cfg.P - l:])) >= len(ends)
        j = i - B0
        if 0 <= j < len(planted) and planted[j] >= 0:
            assert ml >= planted[j]
    oov = B0 + 6
    assert D.longest_suffix_match(corpus, tails[oov], int(tl[oov]))[0] == 0
    assert D.longest_suffix_match(corpus, tails[oov + 1], 3)[0] <= 3


def test_tree_invariants_on_tiny_workload(tiny):
    cfg, tok, off, tails, tl, _ = tiny
    corpus = D.Corpus(tok, off)
    seen_unique = seen_branching = False
    for i in range(len(tails)):
        ml, ends = D.longest_suffix_match(corpus, tails[i], int(tl[i]))
        ids, parent, count = D.build_draft_tree(corpus, tails[i], ml, ends, cfg.N, cfg.topk)
        n = len(ids)
        assert 1 <= n <= cfg.N and parent[0] == -1 and ids[0] == tails[i, -1]
        if ml == 0:
            assert n == 1 and count[0] == 0
            continue
        s = tails[i, cfg.P - ml:].tolist()
        paths = [[]]
        for j in range(1, n):
            assert 0 <= parent[j] < j
            assert count[j] <= count[parent[j]]
            assert count[j] <= count[j - 1] or j == 1        # best-first => non-increasing after the root
            paths.append(paths[parent[j]] + [int(ids[j])])
        assert count[0] >= count[1:].max(initial=0)
        for j in range(n):
            kids = [int(ids[c]) for c in range(1, n) if parent[c] == j]
            assert len(kids) == len(set(kids)) <= cfg.topk
            occ = _window_occurrences(tok, off, s + paths[j])
            assert len(occ) == count[j]
            # all continuations of slot j (not only the kept ones) account for every occurrence that does not
            # end its trajectory
            nxt = {}
            ending = 0
            for (t, p) in occ:
                q = off[t] + p + len(s) + len(paths[j])
                if q < off[t + 1]:
                    nxt[int(tok[q])] = nxt.get(int(tok[q]), 0) + 1
                else:
                    ending += 1
            assert sum(nxt.values()) == count[j] - ending
            ranked = sorted(nxt.items(), key=lambda kv: (-kv[1], kv[0]))[:cfg.topk]
            if n < cfg.N:                                    # frontier emptied: every offered child is in the tree
                assert sorted(kids) == sorted(x for x, _ in ranked)
            else:                                            # kept children are a prefix of the ranking
                assert kids == [x for x, _ in ranked][:len(kids)] or set(kids) <= {x for x, _ in ranked}
            for c in range(1, n):
                if parent[c] == j:
                    assert nxt[int(ids[c])] == count[c]
        if count[0] == 1:                                    # unique occurrence => chain = corpus continuation
            seen_unique = True
            e = int(ends[0])
            room = int(corpus.end_of[e]) - (e + 1)
            m = min(cfg.N - 1, room)
            assert n == m + 1
            assert ids[1:].tolist() == tok[e + 1:e + 1 + m].tolist()
            assert parent[1:].tolist() == list(range(0, m))
        else:
            seen_branching = True
    assert seen_unique and seen_branching


def test_trajectory_order_does_not_matter(tiny):
    """Every worker must draft the same tokens once the caches hold the same trajectories, in whatever order
    they arrived (paper Section 3.3, cross-worker synchronisation)."""
    cfg, tok, off, tails, tl, _ = tiny
    rng = np.random.default_rng(11)
    order = rng.permutation(cfg.n_traj)
    trajs = [tok[off[t]:off[t + 1]] for t in order]
    tok2 = np.concatenate(trajs)
    off2 = np.zeros_like(off)
    off2[1:] = np.cumsum([len(t) for t in trajs])
    a = D.draft_batch(D.Corpus(tok, off), tails, tl, cfg.N, cfg.topk)
    b = D.draft_batch(D.Corpus(tok2, off2), tails, tl, cfg.N, cfg.topk)
    for x, y in zip(a, b):
        assert (x == y).all()


def test_no_match_across_trajectory_boundary():
    trajs = [[1, 2], [3, 4]]
    corpus = D.Corpus.from_lists(trajs)
    ml, ends = D.longest_suffix_match(corpus, np.array([1, 2, 3], np.int32), 3)
    assert ml == 1 and len(ends) == 1                        # [2,3] only exists across the boundary
    ids, parent, count = D.build_draft_tree(corpus, np.array([1, 2, 3], np.int32), ml, ends, 8, 4)
    assert ids.tolist() == [3, 4] and count.tolist() == [1, 1]


def test_min_match_and_budget_edges():
    trajs = [[1, 2, 3, 1, 2, 4]]
    corpus = D.Corpus.from_lists(trajs)
    tail = np.array([9, 1, 2], np.int32)
    ml, ends = D.longest_suffix_match(corpus, tail, 3)
    assert ml == 2
    ids, parent, count = D.build_draft_tree(corpus, tail, ml, ends, 8, 4, min_match=3)
    assert ids.tolist() == [2] and count.tolist() == [2]     # below min_match: root only, count still reported
    ids, parent, count = D.build_draft_tree(corpus, tail, ml, ends, 1, 4)
    assert ids.tolist() == [2]
    ids, parent, count = D.build_draft_tree(corpus, tail, ml, ends, 3, 1)
    assert ids.tolist() == [2, 3, 1] and parent.tolist() == [-1, 0, 1]   # k=1: chain along the smaller id on ties
    assert D.longest_suffix_match(corpus, tail, 0)[0] == 0


def test_workload_aware_switch():
    """Effective batch size = running requests (tail_len >= 0).  At or below the limit nothing changes; above it
    every running request gets the root alone; a request that is not running gets no tree in either mode."""
    rng = np.random.default_rng(3)
    toks = [rng.integers(0, 6, 40).astype(np.int32) for _ in range(5)]
    off = np.concatenate([[0], np.cumsum([len(t) for t in toks])]).astype(np.int64)
    corpus = D.Corpus(np.concatenate(toks), off)
    B, P, N = 6, 4, 5
    tails = rng.integers(0, 6, (B, P)).astype(np.int32)
    tl = np.array([4, 4, -1, 2, 0, 4], np.int32)                      # request 2 is not running: 5 running
    base = D.draft_batch(corpus, tails, tl, N, 2)
    for limit in (0, 5, 9):                                            # no limit, exactly at the limit, above
        got = D.draft_batch(corpus, tails, tl, N, 2, spec_batch_limit=limit)
        for g, w in zip(got, base):
            assert np.array_equal(g, w)
    assert base[1][2] == 0 and (base[2][2] == -1).all()                # not running: no slots
    assert base[1].max() > 1                                           # the speculative mode does draft here
    ml, nn, ids, par, cnt = D.draft_batch(corpus, tails, tl, N, 2, spec_batch_limit=4)
    assert nn.tolist() == [1, 1, 0, 1, 1, 1] and (ml == 0).all() and (cnt == 0).all()
    for i in (0, 1, 3, 4, 5):
        assert ids[i, 0] == tails[i, -1] and par[i, 0] == -1 and (ids[i, 1:] == -1).all()


def test_node_budget_and_probability_threshold():
    """spec_factor caps the tree at 1 + floor(match_len * a / b) slots; min_prob keeps a continuation only when
    count(child) / count(parent) >= a / b.  Checked on the hand-worked corpus and by properties on random ones."""
    with open(os.path.join(GOLD, "draft_case1.json")) as f:
        g = json.load(f)
    trajs = [np.array(t, np.int32) for t in g["trajectories"]]
    off = np.concatenate([[0], np.cumsum([len(t) for t in trajs])]).astype(np.int64)
    corpus = D.Corpus(np.concatenate(trajs), off)
    tail = np.array(g["tail"], np.int32)
    ml, ends = D.longest_suffix_match(corpus, tail, len(tail))
    assert ml == 3
    full = D.build_draft_tree(corpus, tail, ml, ends, 16, 4)
    # factor 1/1: 1 + 3 slots; 2/3: 1 + 2; the capped tree is a prefix of the uncapped one (best-first order)
    for fac, n in (((1, 1), 4), ((2, 3), 3), ((5, 1), 14), ((1, 4), 1)):
        ids, par, cnt = D.build_draft_tree(corpus, tail, ml, ends, 16, 4, spec_factor=fac)
        assert len(ids) == n and ids.tolist() == full[0][:n].tolist() and par.tolist() == full[1][:n].tolist()
    # min_prob 1/2: after [1,2,3] the continuations are 4 (2 of 3) and 5 (1 of 3): only 4 survives, then its own
    # continuations 1 and 8 have 1 of 2 each = exactly 1/2: both stay
    ids, par, cnt = D.build_draft_tree(corpus, tail, ml, ends, 6, 4, min_prob=(1, 2))
    assert ids.tolist()[:4] == [3, 4, 1, 8] and par.tolist()[:4] == [-1, 0, 1, 1] and 5 not in ids.tolist()[1:2]
    ids2, _, _ = D.build_draft_tree(corpus, tail, ml, ends, 6, 4, min_prob=(2, 3))
    assert ids2.tolist() == [3, 4]                                  # 2/3: 4 stays (2 of 3), its continuations (1 of 2) do not
    rng = np.random.default_rng(9)
    toks = [rng.integers(0, 4, 60).astype(np.int32) for _ in range(6)]
    off = np.concatenate([[0], np.cumsum([len(t) for t in toks])]).astype(np.int64)
    corpus = D.Corpus(np.concatenate(toks), off)
    for _ in range(50):
        tail = rng.integers(0, 4, 6).astype(np.int32)
        ml, ends = D.longest_suffix_match(corpus, tail, 6)
        a, b = int(rng.integers(1, 4)), int(rng.integers(1, 5))
        ids, par, cnt = D.build_draft_tree(corpus, tail, ml, ends, 20, 3, spec_factor=(a, b))
        assert len(ids) <= max(1, 1 + ml * a // b)
        pa, pb = int(rng.integers(1, 4)), 4
        ids, par, cnt = D.build_draft_tree(corpus, tail, ml, ends, 20, 3, min_prob=(pa, pb))
        for j in range(1, len(ids)):
            assert cnt[j] * pb >= pa * cnt[par[j]]
        # thresholds off = the plain rule
        x = D.build_draft_tree(corpus, tail, ml, ends, 20, 3, spec_factor=(0, 1), min_prob=(0, 1))
        y = D.build_draft_tree(corpus, tail, ml, ends, 20, 3)
        assert all(np.array_equal(p, q) for p, q in zip(x, y))


# ----------------------------------------------------------------------------------------------
# drafting from the best-scoring of several suffix lengths
# ----------------------------------------------------------------------------------------------

def _mean_accepted_by_enumeration(tokens, offsets, s, ids, parent):
    """Total number of draft tokens accepted when each occurrence of s in turn is taken as the true continuation
    (walks the tree along the text; shares nothing with the checker's score)."""
    children = {}
    for j in range(1, len(ids)):
        children.setdefault(int(parent[j]), {})[int(ids[j])] = j
    total, occ = 0, _window_occurrences(tokens, offsets, s)
    for t, p in occ:
        tr = tokens[offsets[t]:offsets[t + 1]]
        at, node = p + len(s), 0
        while at < len(tr) and int(tr[at]) in children.get(node, {}):
            node = children[node][int(tr[at])]
            at += 1
            total += 1
    return total, len(occ)


def test_scored_lengths_hand_worked_case():
    g = _load("draft_scored_case1.json")
    corpus = D.Corpus.from_lists(g["trajectories"])
    tail = np.array(g["tail"], np.int32)
    for l, want in g["candidates"].items():
        ends = D.suffix_occurrences(corpus, tail, int(l))
        ids, par, cnt = D.build_draft_tree(corpus, tail, int(l), ends, g["N"], g["k"])
        assert (ids.tolist(), par.tolist(), cnt.tolist()) == (want["ids"], want["parent"], want["count"])
        assert list(D.tree_score(cnt)) == want["score"]
    for nl, used in g["used_len"].items():
        ml, u, ids, par, cnt = D.draft_scored(corpus, tail, g["tail_len"], g["N"], g["k"], int(nl))
        assert (ml, u) == (g["match_len"], used)
        want = g["candidates"][str(used)]
        assert (ids.tolist(), par.tolist(), cnt.tolist()) == (want["ids"], want["parent"], want["count"])
    corpus2 = D.Corpus.from_lists(g["trajectories"][:-1])
    assert D.draft_scored(corpus2, tail, 3, g["N"], g["k"], 3)[1] == g["without_last_trajectory"]["used_len"]["3"]


@pytest.mark.parametrize("seed", range(12))
def test_score_is_the_mean_accepted_length_and_the_best_one_wins(seed):
    from fractions import Fraction
    rng = np.random.default_rng(100 + seed)
    V = int(rng.integers(2, 5))
    trajs = [rng.integers(0, V, int(rng.integers(1, 40))).astype(np.int32) for _ in range(int(rng.integers(1, 7)))]
    corpus = D.Corpus.from_lists(trajs)
    P = 6
    for _ in range(25):
        tail = rng.integers(0, V, P).astype(np.int32)
        tl = int(rng.integers(0, P + 1))
        N, k, nl, mm = int(rng.integers(1, 12)), int(rng.integers(1, 4)), int(rng.integers(1, 7)), int(rng.integers(0, 3))
        fac = (int(rng.integers(0, 3)), int(rng.integers(1, 3)))
        ml, used, ids, par, cnt = D.draft_scored(corpus, tail, tl, N, k, nl, mm, spec_factor=fac)
        assert ml == D.match_definitional(trajs, tail.tolist(), tl)
        lens = [l for c, l in enumerate(range(ml, ml - nl, -1)) if c == 0 or l >= max(1, mm)]
        assert used in lens
        scores = {}
        for l in lens:
            s = tail[P - l:] if l > 0 else tail[:0]
            ends = D.suffix_occurrences(corpus, tail, l) if l > 0 else np.zeros(0, np.int64)
            assert len(ends) == (len(_window_occurrences(corpus.tokens, corpus.offsets, s)) if l > 0 else 0)
            t_ids, t_par, t_cnt = D.build_draft_tree(corpus, tail, l, ends, N, k, mm, spec_factor=fac)
            num, den = D.tree_score(t_cnt)
            if l > 0:
                assert (num, den) == _mean_accepted_by_enumeration(corpus.tokens, corpus.offsets, s, t_ids, t_par)
            scores[l] = Fraction(num, den) if den else Fraction(0)
            if l == used:
                assert np.array_equal(t_ids, ids) and np.array_equal(t_par, par) and np.array_equal(t_cnt, cnt)
        top = max(scores.values())
        assert used == max(l for l in lens if scores[l] == top)


def test_one_scored_length_is_the_plain_draft(tiny):
    cfg, tok, off, tails, tl, _ = tiny
    corpus = D.Corpus(tok, off)
    a = D.draft_batch(corpus, tails, tl, cfg.N, cfg.topk)
    b = D.draft_scored_batch(corpus, tails, tl, cfg.N, cfg.topk, 1)
    assert np.array_equal(a[0], b[0]) and np.array_equal(b[1], np.where(b[2] > 0, b[0], 0))
    for x, y in zip(a[1:], b[2:]):
        assert np.array_equal(x, y)
    # more lengths never lower the score of the chosen tree
    c = D.draft_scored_batch(corpus, tails, tl, cfg.N, cfg.topk, 4)
    for i in range(len(tl)):
        n1, d1 = D.tree_score(b[5][i, :b[2][i]])
        n4, d4 = D.tree_score(c[5][i, :c[2][i]])
        assert n4 * max(d1, 1) >= n1 * max(d4, 1)
        assert c[0][i] == b[0][i] and c[1][i] <= c[0][i]
