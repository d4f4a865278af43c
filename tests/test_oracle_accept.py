"""Pins for the acceptance checker: the hand-worked case, closed forms on chains, and a top-down walk that
is written differently from the checker's bottom-up path enumeration."""
import json
import os

import numpy as np
import pytest

from oracle import accept_oracle as C

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _walk_down(ids, parent, n, target):
    """Per-slot mode, distinct siblings: follow the child that equals the target's token, from the root."""
    cur, path = 0, []
    while True:
        nxt = [j for j in range(1, n) if parent[j] == cur and ids[j] == target[cur]]
        if not nxt:
            return len(path), path, int(target[cur])
        cur = nxt[0]
        path.append(cur)


def test_hand_worked_case():
    with open(os.path.join(GOLD, "draft_case1.json")) as f:
        g = json.load(f)
    tree = g["trees"][0]
    a = g["accept"]
    l, path, bonus = C.accept_request(tree["ids"], tree["parent"], len(tree["ids"]), a["target"], a["mode"])
    assert (l, path, bonus) == (a["accept_len"], a["accept_path"], a["bonus"])


@pytest.mark.parametrize("n", [1, 2, 5, 16])
def test_chain_closed_forms(n):
    ids = np.arange(100, 100 + n)
    parent = np.arange(-1, n - 1)
    target = np.concatenate([ids[1:], [777]])               # target after slot p = ids[p+1]: everything matches
    assert C.accept_request(ids, parent, n, target, 0) == (n - 1, list(range(1, n)), 777)
    for d in range(1, n):                                    # first wrong draft at depth d
        t = target.copy()
        t[d - 1] = -5
        l, path, bonus = C.accept_request(ids, parent, n, t, 0)
        assert l == d - 1 and path == list(range(1, d)) and bonus == t[d - 1]
    l, path, bonus = C.accept_request(ids, parent, n, np.full(n, -9), 0)
    assert (l, path, bonus) == (0, [], -9)                   # nothing accepted: plain decode, bonus = target[0]
    l, path, bonus = C.accept_request(ids, parent, n, ids, 1)
    assert (l, path, bonus) == (n - 1, list(range(1, n)), -1)


@pytest.mark.parametrize("seed", range(60))
def test_random_trees_against_top_down_walk(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 24))
    parent = np.array([-1] + [int(rng.integers(0, j)) for j in range(1, n)])
    ids = np.zeros(n, dtype=np.int64)
    for p in range(n):                                       # distinct ids among siblings, tiny alphabet
        kids = [j for j in range(1, n) if parent[j] == p]
        ids[kids] = rng.permutation(max(len(kids), 3))[:len(kids)]
    target = rng.integers(0, 3, size=n)
    l, path, bonus = C.accept_request(ids, parent, n, target, 0)
    assert (l, path, bonus) == _walk_down(ids, parent, n, target)
    if path:
        assert parent[path[0]] == 0
        for a, b in zip(path, path[1:]):
            assert parent[b] == a
    assert l <= n - 1
    # per-node mode: ok(j) = every slot on the path equals its own target; deepest, lowest slot on ties
    depth = np.zeros(n, dtype=int); ok = np.zeros(n, dtype=bool); ok[0] = True
    for j in range(1, n):
        depth[j] = depth[parent[j]] + 1
        ok[j] = ok[parent[j]] and ids[j] == target[j]
    best = max(range(n), key=lambda j: (ok[j] * (depth[j] + 1), -j))
    l1, path1, bonus1 = C.accept_request(ids, parent, n, target, 1)
    assert l1 == depth[best] and bonus1 == -1 and (path1[-1] == best if path1 else best == 0)


def test_duplicate_siblings_lowest_slot_wins():
    ids = np.array([5, 7, 7, 1, 2]); parent = np.array([-1, 0, 0, 1, 2]); target = np.array([7, 1, 2, 0, 0])
    l, path, _ = C.accept_request(ids, parent, 5, target, 0)
    assert l == 2 and path == [1, 3]


def test_batch_layout():
    ids = np.array([[3, 4, 5, 1, 8, 1], [9, -1, -1, -1, -1, -1]], np.int32)
    parent = np.array([[-1, 0, 0, 1, 1, 2], [-1, -1, -1, -1, -1, -1]], np.int32)
    target = np.array([[4, 1, 99, 7, 99, 99], [42, 0, 0, 0, 0, 0]], np.int32)
    alen, path, bonus = C.accept_batch(ids, parent, np.array([6, 1]), target, 0)
    assert alen.tolist() == [2, 0] and bonus.tolist() == [7, 42]
    assert path.tolist() == [[1, 3, -1, -1, -1, -1], [-1] * 6]
