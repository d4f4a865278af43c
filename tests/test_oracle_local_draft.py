"""Pins for the own-context draft checker and the choice between two trees: hand-worked cases, a definitional brute
force written differently, and properties that hold by construction."""
import json
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import draft_oracle as D
from oracle import local_draft_oracle as L

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold():
    with open(os.path.join(GOLD, "local_draft_case1.json")) as f:
        return json.load(f)


def test_hand_worked_cases():
    g = _gold()
    a = g["case_a"]
    for fn in (lambda c, *r: L.draft_local(np.array(c, np.int32), *r), L.draft_local_definitional):
        ml, ids, par, cnt = fn(a["ctx"], a["P"], a["tail_len"], a["N"], a["k"])
        assert ml == a["match_len"]
        assert (list(ids), list(par), list(cnt)) == (a["ids"], a["parent"], a["count"])
    b = g["case_b"]
    ctx = []
    for i in range(b["pairs"]):
        ctx += [7, b["first_value"] if i < b["first_count"] else b["second_value"]]
    ctx += [7]
    for fn in (lambda c, *r: L.draft_local(np.array(c, np.int32), *r), L.draft_local_definitional):
        ml, ids, par, cnt = fn(ctx, b["P"], b["tail_len"], b["N"], b["k"])
        assert ml == b["match_len"]
        assert (list(ids), list(par), list(cnt)) == (b["ids"], b["parent"], b["count"])
    assert len(L.local_occurrences(np.array(ctx, np.int32), 1)) == 40       # the window really cut something off


@pytest.mark.parametrize("seed", range(30))
def test_numpy_version_equals_definitional(seed):
    rng = np.random.default_rng(500 + seed)
    V = int(rng.integers(2, 5))
    for _ in range(12):
        Lc = int(rng.integers(0, 90))
        ctx = rng.integers(0, V, Lc).astype(np.int32)
        if Lc > 4 and rng.random() < 0.3:
            ctx[rng.integers(0, Lc, 2)] = -1                     # tokens < 0 behave like trajectory boundaries
        P, tl = int(rng.integers(1, 9)), int(rng.integers(0, 9))
        N, k, mm = int(rng.integers(1, 14)), int(rng.integers(1, 5)), int(rng.integers(0, 3))
        if Lc == 0:
            continue
        got = L.draft_local(ctx, P, tl, N, k, mm)
        want = L.draft_local_definitional(ctx.tolist(), P, tl, N, k, mm)
        assert got[0] == want[0]
        assert (got[1].tolist(), got[2].tolist(), got[3].tolist()) == (want[1], want[2], want[3])


def test_properties_on_a_long_repetitive_context():
    rng = np.random.default_rng(3)
    blocks = [rng.integers(0, 50, int(rng.integers(3, 20))).astype(np.int32) for _ in range(12)]
    ctx = np.concatenate([blocks[int(rng.integers(0, 12))] for _ in range(300)])
    for cut in (len(ctx), len(ctx) - 7, 1500, 400, 33, 2, 1):
        c = ctx[:cut]
        ml, ids, par, cnt = L.draft_local(c, 32, 32, 24, 4)
        n = len(ids)
        assert ids[0] == c[-1] and par[0] == -1 and cnt[0] <= L.MAX_OCC
        if ml > 0:
            # the matched suffix really occurs ending before the last position, and one more token does not
            ends = L.local_occurrences(c, ml)
            assert len(ends) > 0 and (ends <= len(c) - 2).all()
            assert cnt[0] == min(len(ends), L.MAX_OCC)
            if ml < min(32, len(c) - 1):
                assert len(L.local_occurrences(c, ml + 1)) == 0
        for j in range(1, n):
            assert 0 <= par[j] < j and 0 < cnt[j] <= cnt[par[j]]
            if j > 1:
                assert cnt[j] <= cnt[j - 1]                      # best-first: counts never grow
        # every slot's count is the number of window occurrences followed by its root path
        window = L.local_occurrences(c, ml)[-L.MAX_OCC:] if ml > 0 else []
        for j in range(1, n):
            path, q = [], j
            while q > 0:
                path.append(int(ids[q])); q = par[q]
            path = path[::-1]
            assert cnt[j] == sum(1 for e in window if e + len(path) <= len(c) - 1 and c[e + 1:e + 1 + len(path)].tolist() == path)


def test_switch_and_batch_convention():
    ctx = np.array([1, 2, 3, 1, 2, 3, 1, 2, 4, 4, 4, 4], np.int32)
    off = np.array([0, 8, 8, 12], np.int64)                      # the second request has an empty context
    tl = np.array([8, 8, -1], np.int32)
    ml, nn, ids, par, cnt = L.draft_local_batch(ctx, off, tl, 8, 6, 2)
    assert ml.tolist() == [5, 0, 0] and nn.tolist()[1:] == [1, 0]
    assert ids[1].tolist() == [-1] * 6 and ids[2].tolist() == [-1] * 6
    assert ids[0, :nn[0]].tolist()[:2] == [2, 3]                 # after 1 2 3 1 2 comes 3
    plain = L.draft_local_batch(ctx, off, np.array([8, 8, 8], np.int32), 8, 6, 2, spec_batch_limit=2)
    assert plain[1].tolist() == [1, 1, 1] and (plain[0] == 0).all() and (plain[4] == 0).all()
    assert plain[2][:, 0].tolist() == [2, -1, 4]


@pytest.mark.parametrize("seed", range(6))
def test_pick_by_score(seed):
    rng = np.random.default_rng(900 + seed)
    B, N = 40, 7

    def trees():
        nn = rng.integers(0, N + 1, B).astype(np.int32)
        ml = rng.integers(0, 9, B).astype(np.int32)
        ids = rng.integers(0, 5, (B, N)).astype(np.int32)
        par = np.full((B, N), -1, np.int32)
        cnt = np.zeros((B, N), np.int32)
        for i in range(B):
            c = int(rng.integers(0, 6))
            for j in range(nn[i]):
                cnt[i, j] = c
                c = int(rng.integers(0, c + 1))
                par[i, j] = -1 if j == 0 else int(rng.integers(0, j))
        return ml, nn, ids, par, cnt

    a, b = trees(), trees()
    src, ml, nn, ids, par, cnt = L.pick_by_score(a, b)
    for i in range(B):
        def score(t):
            n, c = int(t[1][i]), t[4][i]
            return Fraction(int(c[1:n].sum()), int(c[0])) if n > 0 and c[0] > 0 else Fraction(0)
        want = 1 if score(b) > score(a) else 0
        assert src[i] == want
        t = b if want else a
        assert ml[i] == t[0][i] and nn[i] == t[1][i]
        assert np.array_equal(ids[i], t[2][i]) and np.array_equal(par[i], t[3][i]) and np.array_equal(cnt[i], t[4][i])
    same = L.pick_by_score(a, a)
    assert (same[0] == 0).all()                                   # equal scores keep the first tree
