"""GPU parity: draft trees from the requests' own contexts and the choice between two trees, bit-exact against the
brute-force checker, through the C-ABI."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import draft_oracle as D
from oracle import local_draft_oracle as L
from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")
NAMES = ["match_len", "num_nodes", "ids", "parent", "count"]


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _run_local(war, ctxs, tail_len, P, N, k, min_match=1, with_count=True, **kw):
    d = U.dev()
    B = len(ctxs)
    off = np.zeros(B + 1, np.int64)
    off[1:] = np.cumsum([len(c) for c in ctxs])
    flat = np.concatenate([np.asarray(c, np.int32) for c in ctxs] + [np.zeros(1, np.int32)])      # never empty
    d_ctx, d_off = torch.from_numpy(flat).to(d), torch.from_numpy(off).to(d)
    d_tl = torch.from_numpy(np.ascontiguousarray(tail_len, dtype=np.int32)).to(d)
    ml, nn = (torch.full((B,), -7, dtype=torch.int32, device=d) for _ in range(2))
    ids, par = (torch.full((B, N), -7, dtype=torch.int32, device=d) for _ in range(2))
    cnt = torch.full((B, N), -7, dtype=torch.int32, device=d) if with_count else None
    war.war_draft_local(d_ctx, d_off, d_tl, P, N, k, min_match, ml, nn, ids, par, cnt, **kw)
    torch.cuda.synchronize()
    got = [x.cpu().numpy() for x in (ml, nn, ids, par)] + [cnt.cpu().numpy() if with_count else None]
    return got, flat[:-1], off


def _compare_local(war, ctxs, tail_len, P, N, k, min_match=1, **kw):
    got, flat, off = _run_local(war, ctxs, tail_len, P, N, k, min_match, **kw)
    want = L.draft_local_batch(flat, off, np.asarray(tail_len), P, N, k, min_match, **kw)
    for name, g, w in zip(NAMES, got, want):
        assert np.array_equal(g, w), f"{name} differs at request(s) {np.flatnonzero((g != w).reshape(len(g), -1).any(axis=1))[:8]}"
    assert war.war_device_status() == 0
    return got


def test_hand_worked_cases(war):
    with open(os.path.join(GOLD, "local_draft_case1.json")) as f:
        g = json.load(f)
    a, b = g["case_a"], g["case_b"]
    ctx_b = []
    for i in range(b["pairs"]):
        ctx_b += [7, b["first_value"] if i < b["first_count"] else b["second_value"]]
    ctx_b += [7]
    for case, ctx in ((a, a["ctx"]), (b, ctx_b)):
        got, _, _ = _run_local(war, [ctx], [case["tail_len"]], case["P"], case["N"], case["k"])
        n = len(case["ids"])
        assert got[0][0] == case["match_len"] and got[1][0] == n
        assert (got[2][0, :n].tolist(), got[3][0, :n].tolist(), got[4][0, :n].tolist()) == (case["ids"], case["parent"], case["count"])
        assert (got[2][0, n:] == -1).all() and (got[3][0, n:] == -1).all() and (got[4][0, n:] == 0).all()


@pytest.mark.parametrize("seed", range(10))
def test_tiny_alphabets(war, seed):
    """Few symbols: long matches, windows that overflow, heavy ties in every rule; empty, one-token and not-running
    requests and tokens < 0 ride along."""
    rng = np.random.default_rng(700 + seed)
    V = int(rng.integers(2, 6))
    B = 40
    ctxs = [rng.integers(0, V, int(rng.integers(0, 1500))).astype(np.int32) for _ in range(B)]
    ctxs[1] = np.zeros(0, np.int32)
    ctxs[2] = np.array([3], np.int32)
    for i in (5, 6, 7):
        if len(ctxs[i]) > 10:
            ctxs[i][rng.integers(0, len(ctxs[i]), 4)] = -1
    P, N, k = int(rng.integers(1, 33)), int(rng.integers(1, 65)), int(rng.integers(1, 9))
    tl = rng.integers(-1, P + 1, B).astype(np.int32)
    _compare_local(war, ctxs, tl, P, N, k, min_match=int(rng.integers(0, 4)),
                   spec_factor=(int(rng.integers(0, 3)), int(rng.integers(1, 4))),
                   min_prob=(int(rng.integers(0, 2)), int(rng.integers(2, 6))))


def test_long_repetitive_contexts(war):
    """Contexts of 10^4-10^5 tokens made of recurring blocks (what a rollout that re-reads files looks like): deep
    matches with few occurrences, a ragged last chunk, the scan running to the start of the context."""
    rng = np.random.default_rng(11)
    blocks = [rng.integers(0, 32000, int(rng.integers(8, 200))).astype(np.int32) for _ in range(40)]
    ctxs = []
    for Lc in (131072, 70001, 20000, 5000, 513, 512, 511, 40):
        parts, n = [], 0
        while n < Lc:
            x = blocks[int(rng.integers(0, 40))] if rng.random() < 0.6 else rng.integers(0, 32000, int(rng.integers(8, 200))).astype(np.int32)
            parts.append(x); n += len(x)
        c = np.concatenate(parts)[:Lc]
        m = min(int(rng.integers(3, 60)), Lc // 2)                       # the context ends with a repeat of its own start
        c[Lc - m:] = c[:m]
        ctxs.append(c)
    tl = np.full(len(ctxs), 32, np.int32)
    got = _compare_local(war, ctxs, tl, 32, 24, 4)
    assert got[0].max() >= 8 and (got[1] > 1).sum() >= 4                # real matches and real trees
    _compare_local(war, ctxs, tl, 32, 64, 8)
    _compare_local(war, ctxs, tl, 32, 24, 4, spec_batch_limit=4)         # over the limit: roots only
    nc, _, _ = _run_local(war, ctxs, tl, 32, 24, 4, with_count=False)
    assert all(np.array_equal(a, b) for a, b in zip(nc[:4], got[:4]))


def test_pick_between_stored_trajectories_and_own_context(war):
    """Both drafts on one batch and the choice between them, against the checker end to end."""
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    rng = np.random.default_rng(21)
    B, N, k, P = 24, 16, 4, cfg.P
    ctxs = []
    for i in range(B):
        t = int(rng.integers(0, cfg.n_traj))
        a = int(off[t]) + int(rng.integers(0, 500))
        own = tok[a:a + int(rng.integers(40, 400))]                      # a piece of a stored trajectory ...
        rep = own[:int(rng.integers(5, 30))]
        ctxs.append(np.concatenate([own, rng.integers(0, cfg.vocab, int(rng.integers(0, 50))).astype(np.int32), rep]))   # ... and a repeat of its start
    tails = np.full((B, P), -1, np.int32)
    tl = np.zeros(B, np.int32)
    for i, c in enumerate(ctxs):
        m = min(P, len(c)); tails[i, P - m:] = c[-m:]; tl[i] = m
    ix = U.build_index(war, tok, off, cfg.vocab)
    ga = U.run_draft(war, ix, tails, tl, N, k)
    gb, flat, coff = _run_local(war, ctxs, tl, P, N, k)
    wa = D.draft_batch(D.Corpus(tok, off), tails, tl, N, k)
    wb = L.draft_local_batch(flat, coff, tl, P, N, k)
    d = U.dev()
    ta = [torch.from_numpy(x).to(d) for x in ga]
    tb = [torch.from_numpy(x).to(d) for x in gb]
    src, ml, nn = (torch.full((B,), -7, dtype=torch.int32, device=d) for _ in range(3))
    ids, par, cnt = (torch.full((B, N), -7, dtype=torch.int32, device=d) for _ in range(3))
    war.war_draft_pick(ta, tb, src, ml, nn, ids, par, cnt)
    torch.cuda.synchronize()
    want = L.pick_by_score(wa, wb)
    for name, g, w in zip(["source"] + NAMES, (src, ml, nn, ids, par, cnt), want):
        assert np.array_equal(g.cpu().numpy(), w), name
    assert 0 < int(src.sum()) < B                                         # both sources win somewhere
    assert war.war_device_status() == 0
    ix.destroy()


@pytest.mark.parametrize("seed", range(3))
def test_pick_on_random_trees(war, seed):
    rng = np.random.default_rng(40 + seed)
    B, N = 70, int(rng.integers(1, 65))

    def trees():
        nn = rng.integers(0, N + 1, B).astype(np.int32)
        cnt = np.zeros((B, N), np.int32)
        for i in range(B):
            c = int(rng.integers(0, 2 ** int(rng.integers(1, 31))))
            for j in range(nn[i]):
                cnt[i, j] = c
                c = int(rng.integers(0, c + 1))
        return (rng.integers(0, 33, B).astype(np.int32), nn, rng.integers(0, 99, (B, N)).astype(np.int32),
                rng.integers(-1, 5, (B, N)).astype(np.int32), cnt)

    a, b = trees(), trees()
    d = U.dev()
    ta, tb = [torch.from_numpy(x).to(d) for x in a], [torch.from_numpy(x).to(d) for x in b]
    src, ml, nn = (torch.zeros(B, dtype=torch.int32, device=d) for _ in range(3))
    ids, par, cnt = (torch.zeros((B, N), dtype=torch.int32, device=d) for _ in range(3))
    war.war_draft_pick(ta, tb, src, ml, nn, ids, par, cnt)
    torch.cuda.synchronize()
    for name, g, w in zip(["source"] + NAMES, (src, ml, nn, ids, par, cnt), L.pick_by_score(a, b)):
        assert np.array_equal(g.cpu().numpy(), w), name
    war.war_draft_pick(ta, ta, src, ml, nn, ids, par, None)              # equal scores keep the first; no count output
    torch.cuda.synchronize()
    assert int(src.sum()) == 0


def test_argument_checks(war):
    d = U.dev()
    z = lambda *s: torch.zeros(s, dtype=torch.int32, device=d)
    ctx, off = z(4), torch.zeros(2, dtype=torch.int64, device=d)
    with pytest.raises(war.WarError):
        war.war_draft_local(ctx, off, z(1), 33, 8, 2, 1, z(1), z(1), z(1, 8), z(1, 8), None)          # P too large
    with pytest.raises(war.WarError):
        war.war_draft_local(ctx, off, z(1), 8, 65, 2, 1, z(1), z(1), z(1, 65), z(1, 65), None)        # N too large
    with pytest.raises(ValueError):
        war.war_draft_local(ctx, off.to(torch.int32), z(1), 8, 8, 2, 1, z(1), z(1), z(1, 8), z(1, 8), None)
    war.war_draft_local(ctx, torch.zeros(1, dtype=torch.int64, device=d), z(0), 8, 8, 2, 1, z(0), z(0), z(0, 8), z(0, 8), None)   # B = 0
