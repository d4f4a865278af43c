"""Pins for the commit checker (advance a request by its accepted tokens): a hand-worked case, identities that
hold for any tree, and a tie to the attention checker: attending over the compacted cache must equal attending
over the explicitly gathered rows."""
import json
import os

import numpy as np

from oracle import accept_oracle as ACC
from oracle import commit_oracle as C

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _tagged_kv(positions, Hkv=2, D=4):
    """Row p holds the value p everywhere (K) / -p (V), so a row's origin can be read off."""
    k = np.broadcast_to(np.arange(positions, dtype=np.float64)[:, None, None], (positions, Hkv, D)).copy()
    return k, -k


def test_hand_worked_case():
    with open(os.path.join(GOLD, "commit_case1.json")) as f:
        g = json.load(f)
    kv_k, kv_v = _tagged_kv(g["prefix_len"] + g["N"])
    for key, bonus in (("expect", g["bonus"]), ("no_bonus", -1)):
        nk, nv, npl, nt, ntl = C.commit_request(kv_k, kv_v, g["prefix_len"], g["ids"], g["accept_len"], g["accept_path"], bonus,
                                                np.array(g["tail"], np.int32), g["tail_len"])
        e = g[key]
        live = C.live_positions(npl, bonus >= 0)
        assert npl == e["prefix_len"] and live == len(e["row_source_position"])
        assert [int(x) for x in nk[:live, 0, 0]] == e["row_source_position"]
        assert [int(-x) for x in nv[:live, 1, 3]] == e["row_source_position"]
        assert nt.tolist() == e["tail"] and ntl == e["tail_len"]


def test_nothing_accepted_and_whole_chain():
    kv_k, kv_v = _tagged_kv(20)
    tail = np.array([0, 0, 3, 4], np.int32)
    # nothing accepted: only the bonus token enters the context, no row moves
    nk, nv, npl, nt, ntl = C.commit_request(kv_k, kv_v, 10, [4, 9, 9], 0, [-1, -1], 77, tail, 2)
    assert npl == 11 and np.array_equal(nk, kv_k) and nt.tolist() == [0, 3, 4, 77] and ntl == 3
    # a fully accepted chain is already in place: rows do not move either
    ids = [4, 5, 6, 7]
    nk, nv, npl, nt, ntl = C.commit_request(kv_k, kv_v, 10, ids, 3, [1, 2, 3], 8, tail, 2)
    assert npl == 14 and np.array_equal(nk[:14], kv_k[:14]) and nt.tolist() == [5, 6, 7, 8] and ntl == 4
    # no bonus, nothing accepted: nothing changes at all
    nk, nv, npl, nt, ntl = C.commit_request(kv_k, kv_v, 10, ids, 0, [-1, -1, -1], -1, tail, 2)
    assert npl == 10 and nt.tolist() == tail.tolist() and ntl == 2


def test_random_trees_rows_and_context():
    rng = np.random.default_rng(5)
    for _ in range(200):
        n = int(rng.integers(1, 17)); N = 16; P = 8
        parent = np.full(N, -1, np.int32); ids = rng.integers(0, 50, N).astype(np.int32)
        for j in range(1, n):
            parent[j] = rng.integers(0, j)
        for j in range(1, n):                                   # siblings must differ (the drafter guarantees it)
            while any(parent[q] == parent[j] and ids[q] == ids[j] for q in range(1, j)):
                ids[j] = rng.integers(0, 50)
        target = np.where(rng.random(N) < 0.6, np.array([ids[[c for c in range(1, n) if parent[c] == p][0]] if any(parent[c] == p for c in range(1, n)) else 0 for p in range(N)]), rng.integers(50, 60, N)).astype(np.int32)
        alen, path, bonus = ACC.accept_request(ids, parent, n, target, 0)
        pl = int(rng.integers(0, 30)); tl = int(rng.integers(0, P + 1))
        tail = np.zeros(P, np.int32); tail[P - tl:] = rng.integers(0, 50, tl)
        kv_k, kv_v = _tagged_kv(pl + N)
        pad = list(path) + [-1] * (N - len(path))
        nk, nv, npl, nt, ntl = C.commit_request(kv_k, kv_v, pl, ids, alen, pad, bonus, tail, tl)
        # rows: the prefix and the root are untouched, then the path's rows in order
        want = list(range(pl + 1)) + [pl + s for s in path]
        assert [int(x) for x in nk[:npl, 0, 0]] == want and npl == pl + alen + 1
        # context: the tail is the end of (old tail ++ accepted ids ++ bonus)
        ctx = tail[P - tl:].tolist() + [int(ids[s]) for s in path] + [int(bonus)]
        assert nt[P - ntl:].tolist() == ctx[-ntl:] and ntl == min(P, len(ctx)) and (nt[:P - ntl] == 0).all()
        # every accepted token is the target's own choice after its predecessor (lossless step)
        prev = 0
        for s in path:
            assert ids[s] == target[prev]; prev = s
        assert bonus == target[prev]


def test_attention_over_compacted_cache_equals_attention_over_the_path():
    """A one-slot tree attending over the compacted cache sees exactly prefix ++ root ++ path rows."""
    from oracle import attention_oracle as A
    rng = np.random.default_rng(11)
    Hkv, G, D, N, pl = 2, 2, 8, 6, 9
    parent = np.array([-1, 0, 0, 2, 3, 3], np.int32)
    path = [2, 3, 5]
    kv_k = rng.standard_normal((pl + N, Hkv, D)); kv_v = rng.standard_normal((pl + N, Hkv, D))
    ids = np.arange(N, dtype=np.int32)
    nk, nv, npl, _, _ = C.commit_request(kv_k, kv_v, pl, ids, 3, path + [-1] * 3, -1, np.zeros(4, np.int32), 0)
    assert npl == pl + 3                                            # no bonus: the last accepted token is the new root
    q = rng.standard_normal((1, Hkv * G, D))
    # (a) the new root (1-slot tree) over the compacted cache
    out_a, lse_a = A.verify_attention_request(q, nk[:npl + 1], nv[:npl + 1], npl, np.array([-1], np.int32), 1, 0.3)
    # (b) the same query as slot 5 of the old tree over the old cache (it sees prefix, root and its ancestors 2, 3)
    qq = np.zeros((N, Hkv * G, D)); qq[5] = q[0]
    out_b, lse_b = A.verify_attention_request(qq, kv_k, kv_v, pl, parent, N, 0.3)
    np.testing.assert_allclose(out_a[0], out_b[5], rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse_a[0], lse_b[5], rtol=1e-12, atol=1e-12)
