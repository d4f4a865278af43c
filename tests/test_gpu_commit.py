"""GPU parity: war_commit (the accepted tokens become context) against the plain CPU checker, through the C-ABI.
Rows are copies, so everything is compared bit for bit.  The last test runs whole steps in a row
(draft -> verify attention -> accept -> commit) on both sides."""
import numpy as np
import pytest
import torch

from oracle import accept_oracle as ACC
from oracle import attention_oracle as A
from oracle import commit_oracle as C
from oracle import draft_oracle as D
from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _pool(rng, B, positions, Hkv, pg, D=128, spare=3):
    """Random bf16 pools behind a shuffled page table with `positions[i]` logical positions per request."""
    n_pages = [(int(p) + pg - 1) // pg for p in positions]
    total = sum(n_pages) + spare
    perm = rng.permutation(total)
    max_pages = max(n_pages)
    pt = np.full((B, max_pages), -1, np.int32)
    at = 0
    for i in range(B):
        pt[i, :n_pages[i]] = perm[at:at + n_pages[i]]; at += n_pages[i]
    g = torch.Generator().manual_seed(int(rng.integers(1 << 30)))
    k = torch.randn((total, Hkv, pg, D), generator=g).to(torch.bfloat16).to(DEV)
    v = torch.randn((total, Hkv, pg, D), generator=g).to(torch.bfloat16).to(DEV)
    return k, v, pt


def _random_trees(rng, B, N, vocab=97):
    parent = np.full((B, N), -1, np.int32); nn = np.zeros(B, np.int32); ids = np.zeros((B, N), np.int32)
    for i in range(B):
        n = int(rng.integers(1, N + 1)); nn[i] = n
        ids[i, :n] = rng.integers(0, vocab, n)
        for j in range(1, n):
            parent[i, j] = int(rng.integers(0, j))
            while any(parent[i, q] == parent[i, j] and ids[i, q] == ids[i, j] for q in range(1, j)):
                ids[i, j] = rng.integers(0, vocab)
    return nn, parent, ids


def _targets(rng, nn, parent, ids, mode, p_match=0.7, vocab=97):
    B, N = ids.shape
    t = rng.integers(vocab, vocab + 50, size=(B, N)).astype(np.int32)          # tokens no draft has
    for i in range(B):
        for j in range(1, int(nn[i])):
            if rng.random() < p_match:
                if mode == 0: t[i, parent[i, j]] = ids[i, j]
                else: t[i, j] = ids[i, j]
    return t


def _dense(k_pool, v_pool, pt_row, n):
    return A.gather_request_kv(k_pool, v_pool, pt_row, n)


@pytest.mark.parametrize("N,pg,mode,token_major", [(8, 16, 0, False), (64, 16, 0, False), (24, 32, 0, False), (16, 16, 1, False),
                                                   (1, 16, 0, False), (32, 16, 0, True), (16, 64, 0, True)])
def test_commit_matches_checker(war, N, pg, mode, token_major):
    rng = np.random.default_rng(100 + N + pg + mode)
    B, Hkv, P = 37, 4, 32
    pl = rng.integers(0, 300, B).astype(np.int32)
    pl[:4] = [0, pg - 1, pg, 2 * pg - 1]                                       # page-boundary cases
    k_pool, v_pool, pt = _pool(rng, B, pl + N, Hkv, pg)
    if token_major:                                                            # same logical tensors, (page, token, head, d) in memory
        k_pool = k_pool.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        v_pool = v_pool.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    nn, parent, ids = _random_trees(rng, B, N)
    target = _targets(rng, nn, parent, ids, mode)
    alen, path, bonus = U.run_accept(war, ids, parent, nn, target, mode)
    tl = rng.integers(0, P + 1, B).astype(np.int32)
    tail = np.zeros((B, P), np.int32)
    for i in range(B):
        tail[i, P - tl[i]:] = rng.integers(0, 97, tl[i])
    before = [_dense(k_pool, v_pool, pt[i], int(pl[i]) + N) for i in range(B)]
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)
    d_pl, d_tail, d_tl = t(pl), t(tail), t(tl)
    war.war_commit(t(ids), t(alen), t(path), t(bonus), k_pool, v_pool, t(pt), d_pl, d_tail, d_tl)
    torch.cuda.synchronize()
    assert war.war_device_status() == 0
    got_pl, got_tail, got_tl = d_pl.cpu().numpy(), d_tail.cpu().numpy(), d_tl.cpu().numpy()
    moved = 0
    for i in range(B):
        a_l, a_p, b_ = ACC.accept_request(ids[i], parent[i], int(nn[i]), target[i], mode)
        assert a_l == alen[i] and b_ == bonus[i]
        wk, wv, wpl, wt, wtl = C.commit_request(before[i][0], before[i][1], int(pl[i]), ids[i], a_l,
                                                list(a_p) + [-1] * (N - len(a_p)), b_, tail[i], int(tl[i]))
        gk, gv = _dense(k_pool, v_pool, pt[i], int(pl[i]) + N)
        assert got_pl[i] == wpl and got_tl[i] == wtl and got_tail[i].tolist() == wt.tolist()
        # the whole allocation is compared, dead rows included: the checker leaves them as they were, so must the kernel
        assert np.array_equal(gk, wk) and np.array_equal(gv, wv)
        moved += sum(1 for d, s in enumerate(a_p) if s != d + 1)
    if N > 1:
        assert moved > 0 and alen.max() > 1                                   # the case really moves rows


def test_malformed_paths_and_pages_are_reported(war):
    rng = np.random.default_rng(7)
    B, N, Hkv, pg, P = 4, 8, 2, 16, 8
    pl = np.array([40, 41, 42, 43], np.int32)
    k_pool, v_pool, pt = _pool(rng, B, pl + N, Hkv, pg)
    ids = rng.integers(0, 50, (B, N)).astype(np.int32)
    alen = np.array([2, 2, 9, 1], np.int32)
    path = np.full((B, N), -1, np.int32)
    path[0, :2] = [3, 2]                                                       # not increasing
    path[1, :2] = [2, 5]                                                       # fine
    path[3, :1] = [0]                                                          # the root is not a draft
    bonus = np.array([5, 6, 7, 8], np.int32)
    tail = rng.integers(0, 50, (B, P)).astype(np.int32); tl = np.full(B, P, np.int32)
    k0, v0 = k_pool.clone(), v_pool.clone()
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)
    d_pl, d_tail, d_tl = t(pl), t(tail), t(tl)
    war.war_commit(t(ids), t(alen), t(path), t(bonus), k_pool, v_pool, t(pt), d_pl, d_tail, d_tl)
    torch.cuda.synchronize()
    assert war.war_device_status() == 7                                        # WAR_ERR_BAD_TREE
    got_pl = d_pl.cpu().numpy()
    assert got_pl.tolist() == [40, 44, 42, 43]                                 # only the well-formed request advanced
    assert torch.equal(d_tail.cpu()[[0, 2, 3]], torch.from_numpy(tail[[0, 2, 3]]))
    # request 1 moved rows 2 -> 1 and 5 -> 2 of its tree region; everything else is bit-identical
    b1 = _dense(k0, v0, pt[1], 41 + N); a1 = _dense(k_pool, v_pool, pt[1], 41 + N)
    assert np.array_equal(a1[0][42], b1[0][43]) and np.array_equal(a1[0][43], b1[0][46])
    for i in (0, 2, 3):
        b, a_ = _dense(k0, v0, pt[i], int(pl[i]) + N), _dense(k_pool, v_pool, pt[i], int(pl[i]) + N)
        assert np.array_equal(a_[0], b[0]) and np.array_equal(a_[1], b[1])
    # a page id outside the pool: reported, that row skipped, nothing faults
    pt_bad = pt.copy(); pt_bad[1, (41 + 1) // pg] = 10 ** 6
    d_pl = t(pl)
    war.war_commit(t(ids), t(np.array([0, 2, 0, 0], np.int32)), t(path), t(bonus), k_pool, v_pool, t(pt_bad), d_pl, t(tail), t(tl))
    torch.cuda.synchronize()
    assert war.war_device_status() == 8                                        # WAR_ERR_BAD_PAGE
    # a bad SOURCE page with a good destination: the destination row keeps what it held (it is not zeroed)
    pt_src = pt.copy(); pt_src[1, (41 + 7) // pg] = -5                         # slot 7 of request 1 lives on its own page
    assert (41 + 7) // pg != (41 + 1) // pg
    path2 = np.full((B, N), -1, np.int32); path2[1, 0] = 7
    kb, vb = k_pool.clone(), v_pool.clone()
    war.war_commit(t(ids), t(np.array([0, 1, 0, 0], np.int32)), t(path2), t(bonus), k_pool, v_pool, t(pt_src), t(pl), t(tail), t(tl))
    torch.cuda.synchronize()
    assert war.war_device_status() == 8
    assert torch.equal(k_pool, kb) and torch.equal(v_pool, vb)


def test_not_running_requests_are_left_alone(war):
    """tail_len < 0 marks a request that is not running (war_draft gives it no tree, war_accept an empty result):
    the commit must not touch it and must not report it as malformed."""
    rng = np.random.default_rng(8)
    B, N, Hkv, pg, P = 3, 8, 2, 16, 8
    pl = np.array([40, 41, 42], np.int32)
    k_pool, v_pool, pt = _pool(rng, B, pl + N, Hkv, pg)
    ids = rng.integers(0, 50, (B, N)).astype(np.int32)
    alen = np.array([1, 0, 0], np.int32)
    path = np.full((B, N), -1, np.int32); path[0, 0] = 3
    bonus = np.array([9, -1, 4], np.int32)
    tail = rng.integers(0, 50, (B, P)).astype(np.int32); tl = np.array([P, -1, 2], np.int32)
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)
    d_pl, d_tail, d_tl = t(pl), t(tail), t(tl)
    war.war_commit(t(ids), t(alen), t(path), t(bonus), k_pool, v_pool, t(pt), d_pl, d_tail, d_tl)
    torch.cuda.synchronize()
    assert war.war_device_status() == 0
    assert d_pl.cpu().tolist() == [42, 41, 43] and d_tl.cpu().tolist() == [P, -1, 3]
    assert torch.equal(d_tail.cpu()[1], torch.from_numpy(tail[1]))


def test_steps_in_a_row(war):
    """Three whole steps on the Tiny workload's corpus: draft, verify attention, accept, commit, with fresh K/V rows
    for the new root and the tree slots written before every step (a model forward would do that).  Every
    integer result is compared bit for bit each step, attention on all requests, and the caches at the end."""
    cfg = W.CONFIGS["tiny"]
    rng = np.random.default_rng(42)
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    corpus = D.Corpus(tok, off)
    ix = U.build_index(war, tok, off, cfg.vocab, cfg.P + cfg.N)
    B, N, P, Hkv, Hq, pg, steps = cfg.B, cfg.N, cfg.P, cfg.Hkv, cfg.Hq, cfg.page_size, 3
    pl = rng.integers(200, 700, B).astype(np.int32)
    k_pool, v_pool, pt = _pool(rng, B, pl + steps * N + N, Hkv, pg)
    t = lambda x: torch.from_numpy(np.ascontiguousarray(x, dtype=np.int32)).to(DEV)
    d_pt = t(pt)
    d_pl, d_tail, d_tl = t(pl), t(tails), t(tl)
    o_pl, o_tail, o_tl = pl.copy(), tails.copy(), tl.copy()
    dense = [list(_dense(k_pool, v_pool, pt[i], int(pl[i]) + (steps + 1) * N)) for i in range(B)]
    scale = 1.0 / np.sqrt(cfg.D)
    emitted = 0
    for step in range(steps):
        # fresh rows for positions prefix_len .. prefix_len + N - 1 on both sides
        g = torch.Generator().manual_seed(1000 + step)
        new_k = torch.randn((B, N, Hkv, cfg.D), generator=g).to(torch.bfloat16)
        new_v = torch.randn((B, N, Hkv, cfg.D), generator=g).to(torch.bfloat16)
        q = torch.randn((B, N, Hq, cfg.D), generator=g).to(torch.bfloat16).to(DEV)
        for i in range(B):
            pos = np.arange(o_pl[i], o_pl[i] + N)
            pages = torch.from_numpy(pt[i, pos // pg].astype(np.int64)).to(DEV); rows = torch.from_numpy(pos % pg).to(DEV)
            k_pool[pages, :, rows, :] = new_k[i].to(DEV); v_pool[pages, :, rows, :] = new_v[i].to(DEV)
            dense[i][0][pos] = new_k[i].double().numpy(); dense[i][1][pos] = new_v[i].double().numpy()
        # GPU step
        ml, nn, ids, par, cnt = U.run_draft(war, ix, d_tail.cpu().numpy(), d_tl.cpu().numpy(), N, cfg.topk)
        o_ml, o_nn, o_ids, o_par, o_cnt = D.draft_batch(corpus, o_tail, o_tl, N, cfg.topk)
        assert np.array_equal(ml, o_ml) and np.array_equal(nn, o_nn)
        for i in range(B):
            n = int(nn[i])
            assert np.array_equal(ids[i, :n], o_ids[i, :n]) and np.array_equal(par[i, :n], o_par[i, :n])
        params = war.attn_params(q, k_pool, v_pool, d_pt, scale, 0)
        ws = war.new_workspace(params, DEV)
        out = torch.zeros_like(q); lse = torch.zeros(q.shape[:3], dtype=torch.float32, device=DEV)
        war.war_verify_attn(q, k_pool, v_pool, d_pt, d_pl, t(nn), t(par), params, ws, out, lse)
        torch.cuda.synchronize()
        for i in range(B):
            n = int(nn[i])
            w_out, w_lse = A.verify_attention_request(q[i].double().cpu().numpy(), dense[i][0], dense[i][1], int(o_pl[i]), o_par[i], n, scale)
            U.assert_attention_close(out[i].float().cpu().numpy(), lse[i].cpu().numpy(), w_out, w_lse, n)
        target = W.make_targets(cfg, o_ids, o_par, o_nn, 0)
        alen, path, bonus = U.run_accept(war, ids, par, nn, target, 0)
        war.war_commit(t(ids), t(alen), t(path), t(bonus), k_pool, v_pool, d_pt, d_pl, d_tail, d_tl)
        torch.cuda.synchronize()
        for i in range(B):
            a_l, a_p, b_ = ACC.accept_request(o_ids[i], o_par[i], int(o_nn[i]), target[i], 0)
            assert a_l == alen[i] and b_ == bonus[i] and list(a_p) == path[i, :a_l].tolist()
            dense[i][0], dense[i][1], o_pl[i], o_tail[i], o_tl[i] = C.commit_request(
                dense[i][0], dense[i][1], int(o_pl[i]), o_ids[i], a_l, list(a_p) + [-1] * (N - a_l), b_, o_tail[i], int(o_tl[i]))
            emitted += a_l + 1
        assert np.array_equal(d_pl.cpu().numpy(), o_pl) and np.array_equal(d_tl.cpu().numpy(), o_tl)
        gt = d_tail.cpu().numpy()
        for i in range(B):
            assert np.array_equal(gt[i, P - o_tl[i]:], o_tail[i, P - o_tl[i]:])
    assert war.war_device_status() == 0
    assert emitted > steps * B                                                 # some drafts were accepted on the way
    for i in range(B):
        gk, gv = _dense(k_pool, v_pool, pt[i], int(o_pl[i]))
        assert np.array_equal(gk, dense[i][0][:o_pl[i]]) and np.array_equal(gv, dense[i][1][:o_pl[i]])
    ix.destroy()
