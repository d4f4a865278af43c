"""GPU parity: acceptance, bit-exact against the path-enumerating checker."""
import numpy as np
import pytest

from oracle import accept_oracle as C
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _random_trees(rng, B, N, alphabet):
    ids = np.full((B, N), -1, np.int32); parent = np.full((B, N), -1, np.int32); nn = np.zeros(B, np.int32)
    for i in range(B):
        n = int(rng.integers(0, N + 1)); nn[i] = n
        for j in range(n):
            parent[i, j] = -1 if j == 0 else int(rng.integers(0, j))
        for p in range(n):
            kids = [j for j in range(1, n) if parent[i, j] == p]
            ids[i, kids] = rng.permutation(max(len(kids), alphabet))[:len(kids)]
        if n:
            ids[i, 0] = int(rng.integers(0, alphabet))
    return ids, parent, nn


@pytest.mark.parametrize("N,mode", [(1, 0), (8, 0), (16, 1), (33, 0), (64, 0), (64, 1)])
def test_random_trees(war, N, mode):
    rng = np.random.default_rng(N * 2 + mode)
    B = 301
    ids, parent, nn = _random_trees(rng, B, N, 3)
    target = rng.integers(0, 3, size=(B, N)).astype(np.int32)
    got = U.run_accept(war, ids, parent, nn, target, mode)
    want = C.accept_batch(ids, parent, nn, target, mode)
    for g, w in zip(got, want):
        assert (g == w).all()
    assert got[0].max() >= 2 or N < 8
    assert war.war_device_status() == 0


def test_chains_and_full_acceptance(war):
    N = 64
    ids = np.arange(N, dtype=np.int32)[None, :].repeat(3, 0) + 100
    parent = np.arange(-1, N - 1, dtype=np.int32)[None, :].repeat(3, 0)
    target = np.concatenate([ids[:, 1:], np.full((3, 1), 9, np.int32)], axis=1)
    target[1, 10] = -5                                                 # first wrong draft at depth 11
    target[2, 0] = -5                                                  # nothing accepted
    alen, path, bonus = U.run_accept(war, ids, parent, np.array([N, N, N], np.int32), target, 0)
    assert alen.tolist() == [N - 1, 10, 0] and bonus.tolist() == [9, -5, -5]
    assert path[0, :N - 1].tolist() == list(range(1, N)) and path[1, :10].tolist() == list(range(1, 11))
    assert (path[1, 10:] == -1).all() and (path[2] == -1).all()


def test_malformed_tree_sets_status_and_accepts_nothing(war):
    ids = np.array([[5, 6, 7, 8], [5, 6, 7, 8]], np.int32)
    parent = np.array([[-1, 0, 2, 1], [-1, 0, 0, 1]], np.int32)         # request 0: parent[2] = 2 is not < 2
    target = np.array([[6, 8, 0, 0], [6, 8, 0, 0]], np.int32)
    alen, path, bonus = U.run_accept(war, ids, parent, np.array([4, 4], np.int32), target, 0)
    assert alen.tolist() == [0, 2] and (path[0] == -1).all() and path[1, :2].tolist() == [1, 3]
    assert war.war_device_status() == 7
    assert war.war_device_status() == 0                                # reading clears it
