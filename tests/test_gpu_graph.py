"""The three calls of a step enqueue work and return without touching the host, so a whole step can be captured
in a CUDA graph and replayed (the paper's engine keeps separate CUDA graphs for speculative and plain decoding,
Section 3.3).  Replays must reproduce the eager results bit for bit, also after the inputs change in place."""
import numpy as np
import pytest
import torch

from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def test_step_replays_from_a_cuda_graph(war):
    dev = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["tiny"], B=6, N=16)
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    ctx = np.array([4096, 777, 1300, 2049, 40, 3000])
    ix = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + cfg.N)
    a = W.make_attention_inputs(cfg, ctx, device=dev)
    B, N = cfg.B, cfg.N
    i32 = dict(dtype=torch.int32, device=dev)
    d_tails, d_tl = torch.from_numpy(tails).to(dev), torch.from_numpy(tl).to(dev)
    ml, nn = torch.zeros(B, **i32), torch.zeros(B, **i32)
    ids, par, cnt = torch.zeros((B, N), **i32), torch.zeros((B, N), **i32), torch.zeros((B, N), **i32)
    alen, path, bonus = torch.zeros(B, **i32), torch.zeros((B, N), **i32), torch.zeros(B, **i32)
    target = torch.randint(0, cfg.vocab, (B, N), dtype=torch.int32, device=dev)
    out = torch.zeros_like(a.q)
    lse = torch.zeros(a.q.shape[:3], dtype=torch.float32, device=dev)
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, 1.0 / np.sqrt(cfg.D), 0)
    ws = war.new_workspace(params, dev)

    def step():
        war.war_draft(ix, d_tails, d_tl, N, cfg.topk, 1, ml, nn, ids, par, cnt)
        war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, nn, par, params, ws, out, lse)
        war.war_accept(ids, par, nn, target, 0, alen, path, bonus)

    def snapshot():
        torch.cuda.synchronize()
        return [t.clone() for t in (ml, nn, ids, par, cnt, out, lse, alen, path, bonus)]

    step()                                                    # eager: also does the one-time per-device set-up
    eager = snapshot()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for t in (ml, nn, ids, par, cnt, out, lse, alen, path, bonus):
        t.zero_()
    g.replay()
    for x, y in zip(snapshot(), eager):
        assert torch.equal(x, y)
    # new inputs in the same buffers: the replay recomputes everything on the device
    d_tails.copy_(torch.roll(d_tails, 1, dims=0)); d_tl.copy_(torch.roll(d_tl, 1, dims=0))
    a.q.copy_(torch.roll(a.q, 1, dims=0))
    g.replay()
    replayed = snapshot()
    step()
    for x, y in zip(replayed, snapshot()):
        assert torch.equal(x, y)
    assert not torch.equal(replayed[2], eager[2])
    assert war.war_device_status() == 0
    ix.destroy()


def test_one_graph_serves_speculative_and_plain_steps(war):
    """Workload-aware switch inside a captured step (paper Section 3.3: adaptive enabling by batch size, stateless
    switching, CUDA-graph compatibility): the number of running requests is read on the device, so the same graph
    speculates while few requests run and does plain decode steps (root-only trees) when many do."""
    from oracle import draft_oracle as D
    dev = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["tiny"], B=12, N=16)
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    corpus = D.Corpus(tok, off)
    ix = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + cfg.N)
    a = W.make_attention_inputs(cfg, W.context_lengths(cfg)[:cfg.B] // 4 + 100, device=dev)
    B, N, limit = cfg.B, cfg.N, 8
    i32 = dict(dtype=torch.int32, device=dev)
    d_tails, d_tl = torch.from_numpy(tails).to(dev), torch.from_numpy(tl).to(dev)
    ml, nn = torch.zeros(B, **i32), torch.zeros(B, **i32)
    ids, par, cnt = torch.zeros((B, N), **i32), torch.zeros((B, N), **i32), torch.zeros((B, N), **i32)
    alen, path, bonus = torch.zeros(B, **i32), torch.zeros((B, N), **i32), torch.zeros(B, **i32)
    target = torch.randint(0, cfg.vocab, (B, N), dtype=torch.int32, device=dev)
    out = torch.zeros_like(a.q)
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, 1.0 / np.sqrt(cfg.D), 0)
    ws = war.new_workspace(params, dev)

    # the commit works on copies (made inside the step), so that every replay starts from the same request state
    c_k, c_v = a.k_pool.clone(), a.v_pool.clone()
    c_pl, c_tails, c_tl = a.prefix_len.clone(), d_tails.clone(), d_tl.clone()

    def step():
        war.war_draft(ix, d_tails, d_tl, N, cfg.topk, 1, ml, nn, ids, par, cnt, limit)
        war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, nn, par, params, ws, out, None)
        war.war_accept(ids, par, nn, target, 0, alen, path, bonus)
        c_pl.copy_(a.prefix_len); c_tails.copy_(d_tails); c_tl.copy_(d_tl)
        war.war_commit(ids, alen, path, bonus, c_k, c_v, a.page_table, c_pl, c_tails, c_tl)

    step()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    with torch.cuda.graph(g):
        step()
    for running in (12, 8, 3, 9):                                     # above, at, below, above the limit again
        h_tl = tl.copy(); h_tl[running:] = -1
        d_tl.copy_(torch.from_numpy(h_tl).to(dev))
        out.fill_(7.0)
        g.replay()
        torch.cuda.synchronize()
        want = D.draft_batch(corpus, tails, h_tl, N, cfg.topk, spec_batch_limit=limit)
        for got, w in zip((ml, nn, ids, par, cnt), want):
            assert np.array_equal(got.cpu().numpy(), w), running
        h_nn = nn.cpu().numpy()
        assert (h_nn.max() > 1) == (running <= limit)
        assert (alen.cpu().numpy()[h_nn <= 1] == 0).all()
        o = out.float().cpu().numpy()
        for i in range(B):                                             # rows beyond num_nodes are never written
            assert (o[i, h_nn[i]:] == 7.0).all() and (h_nn[i] == 0 or (o[i, 0] != 7.0).any())
        # the commit leaves requests that are not running alone (and does not call them malformed) and advances the others
        h_cpl, h_ctl, h_ct = c_pl.cpu().numpy(), c_tl.cpu().numpy(), c_tails.cpu().numpy()
        h_pl, h_alen = a.prefix_len.cpu().numpy(), alen.cpu().numpy()
        assert (h_cpl[running:] == h_pl[running:]).all() and (h_ctl[running:] == -1).all()
        assert (h_ct[running:] == tails[running:]).all()
        assert (h_cpl[:running] == h_pl[:running] + h_alen[:running] + 1).all()
        assert war.war_device_status() == 0
    assert war.war_device_status() == 0
    ix.destroy()


def test_drafting_variants_replay_from_a_graph(war):
    """war_draft_scored, war_draft_local (a cluster launch) and war_draft_pick enqueue work only: captured once,
    replayed on new inputs in the same buffers, bit-identical to eager calls."""
    from oracle import draft_oracle as D
    from oracle import local_draft_oracle as L
    cfg = W.scaled(W.CONFIGS["tiny"], B=6)
    dev = U.dev()
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    ctx_len = np.array([900, 3000, 64, 5000, 1200, 700])
    h_ctx, h_off = W.make_request_contexts(cfg, ctx_len)
    ix = U.build_index(war, tok, off, cfg.vocab)
    B, N, k, P = cfg.B, cfg.N, cfg.topk, cfg.P
    i32 = dict(dtype=torch.int32, device=dev)
    d_tails, d_tl = torch.from_numpy(tails).to(dev), torch.from_numpy(tl).to(dev)
    d_ctx, d_off = torch.from_numpy(h_ctx).to(dev), torch.from_numpy(h_off).to(dev)
    tree = lambda: [torch.zeros(B, **i32), torch.zeros(B, **i32)] + [torch.zeros((B, N), **i32) for _ in range(3)]
    s_tree, l_tree, p_tree = tree(), tree(), tree()
    used, src = torch.zeros(B, **i32), torch.zeros(B, **i32)
    sws = torch.zeros(war.war_draft_scored_workspace_bytes(B, P, N, k, 3), dtype=torch.uint8, device=dev)

    def drafts():
        war.war_draft_scored(ix, d_tails, d_tl, N, k, 1, 3, sws, s_tree[0], used, *s_tree[1:])
        war.war_draft_local(d_ctx, d_off, d_tl, P, N, k, 1, *l_tree)
        war.war_draft_pick(s_tree, l_tree, src, *p_tree)

    def snapshot():
        torch.cuda.synchronize()
        return [t.clone() for t in (used, src, *s_tree, *l_tree, *p_tree)]

    drafts()
    eager = snapshot()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        drafts()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        drafts()
    for t in (used, src, *s_tree, *l_tree, *p_tree):
        t.fill_(-3)
    g.replay()
    for x, y in zip(snapshot(), eager):
        assert torch.equal(x, y)
    # new inputs in the same buffers
    d_tails.copy_(torch.roll(d_tails, 1, dims=0)); d_tl.copy_(torch.roll(d_tl, 1, dims=0))
    d_ctx.copy_(torch.roll(d_ctx, 17))
    g.replay()
    replayed = snapshot()
    drafts()
    for x, y in zip(replayed, snapshot()):
        assert torch.equal(x, y)
    # and the replay is the checker's answer
    t2, l2 = d_tails.cpu().numpy(), d_tl.cpu().numpy()
    w_s = D.draft_scored_batch(D.Corpus(tok, off), t2, l2, N, k, 3)
    w_l = L.draft_local_batch(d_ctx.cpu().numpy(), h_off, l2, P, N, k)
    w_p = L.pick_by_score((w_s[0],) + tuple(w_s[2:]), w_l)
    for gpu, want in zip([src] + p_tree, w_p):
        assert np.array_equal(gpu.cpu().numpy(), want)
    assert war.war_device_status() == 0
    ix.destroy()


def test_a_captured_draft_follows_the_index_through_updates(war):
    """The draft kernel picks the published set of index arrays when it starts, from device memory, so a launch that
    was captured before an update answers from the updated index when it is replayed: capture, append, replay, append
    again (the first captured set is being rebuilt now), evict, replay -- every replay equals the checker on the corpus
    as it is at that moment."""
    from oracle import draft_oracle as D
    dev = U.dev()
    cfg = W.scaled(W.CONFIGS["tiny"], B=8, n_traj=40)
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    N, k = cfg.N, cfg.topk
    first, second = 20, 30                                            # 20 trajectories, then +10, then +10
    cap = len(tok) + cfg.n_traj
    ix = U.build_index(war, tok[:off[first]], off[:first + 1], cfg.vocab, max_depth=cfg.P + N, capacity=cap)
    i32 = dict(dtype=torch.int32, device=dev)
    d_tails, d_tl = torch.from_numpy(tails).to(dev), torch.from_numpy(tl).to(dev)
    ml, nn = torch.zeros(cfg.B, **i32), torch.zeros(cfg.B, **i32)
    ids, par, cnt = (torch.zeros((cfg.B, N), **i32) for _ in range(3))

    def draft():
        war.war_draft(ix, d_tails, d_tl, N, k, 1, ml, nn, ids, par, cnt)

    def check(n_from, n_to):
        torch.cuda.synchronize()
        o = off[n_from:n_to + 1] - off[n_from]
        want = D.draft_batch(D.Corpus(tok[off[n_from]:off[n_to]], o), tails, tl, N, k)
        for got, w in zip((ml, nn, ids, par, cnt), want):
            assert np.array_equal(got.cpu().numpy(), w), (n_from, n_to)

    draft()
    check(0, first)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        draft()
    torch.cuda.current_stream().wait_stream(side)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        draft()
    g.replay()
    check(0, first)
    d_tok = torch.from_numpy(tok).to(dev)
    war.war_index_append(ix, d_tok[off[first]:off[second]], off[first:second + 1] - off[first])
    g.replay()
    check(0, second)
    war.war_index_append(ix, d_tok[off[second]:], off[second:] - off[second])
    g.replay()
    check(0, cfg.n_traj)
    war.war_index_evict(ix, 5)
    g.replay()
    check(5, cfg.n_traj)
    assert war.war_device_status() == 0
    del g
    ix.destroy()
