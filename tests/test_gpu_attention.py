"""GPU parity: tree-masked verify attention against the fp64 checker, through the C-ABI.

Bar: atol 1e-2 / rtol 1e-2 on the fp32 cast of both sides (the stated tolerance), plus a per-row relative L2
bound of 1e-2 and lse within 1e-3, because the stated absolute bar is loose at long context."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import attention_oracle as A
from oracle import draft_oracle as D
from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")
KERNELS = [0, 1, 2]          # 0 default (one launch for up to 64 requests), 1 plain CUDA-core kernel, 2 tensor-core kernel with separate plan / combine launches


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _random_trees(rng, B, N, n_fixed=None):
    parent = np.full((B, N), -1, np.int32); nn = np.zeros(B, np.int32)
    for i in range(B):
        n = int(rng.integers(1, N + 1)) if n_fixed is None else n_fixed[i]
        nn[i] = n
        for j in range(1, n):
            parent[i, j] = int(rng.integers(0, j))
    return nn, parent


def _check(war, cfg, ctx, nn, parent, kernel, scale=None, a=None):
    scale = 1.0 / np.sqrt(cfg.D) if scale is None else scale
    if a is None:
        a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    got, got_lse, raw = U.run_attn(war, a, nn, parent, scale, kernel)
    want = A.verify_attention(a.q, a.k_pool, a.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(),
                              nn, parent, scale)
    for i in range(cfg.B):
        n = int(nn[i])
        if n:
            U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], n)
        assert (got[i, n:] == 7.0).all() and (got_lse[i, n:] == 7.0).all()       # rows beyond num_nodes untouched
    assert war.war_device_status() == 0
    return a, raw


@pytest.mark.parametrize("kernel", KERNELS)
def test_tiny_config(war, kernel):
    """8 requests x 4096 context, trees from the brute-force drafter; the plan splits every request into several
    KV chunks here, so the combine pass is exercised as well."""
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    _, nn, _, parent, _ = D.draft_batch(D.Corpus(tok, off), tails, tl, cfg.N, cfg.topk)
    ctx = W.context_lengths(cfg)
    a, raw1 = _check(war, cfg, ctx, nn, parent, kernel)
    _, _, raw2 = U.run_attn(war, a, nn, parent, 1.0 / np.sqrt(cfg.D), kernel)
    assert torch.equal(raw1, raw2)                                           # deterministic


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("case", ["ragged16", "ragged32", "wide", "single", "deep", "many", "rows256", "page8", "page64", "page128"])
def test_shapes_and_ragged_lengths(war, kernel, case):
    rng = np.random.default_rng(["ragged16", "ragged32", "wide", "single", "deep", "many", "rows256", "page8", "page64", "page128"].index(case))
    base = W.CONFIGS["tiny"]
    if case == "ragged16":       # lengths around page and tile edges, empty prefix, an unused request
        ctx = np.array([1, 2, 15, 16, 17, 113, 127, 128, 129, 1000, 1024, 1025, 2049, 3000])
        cfg = W.scaled(base, B=len(ctx), N=16)
        nn, parent = _random_trees(rng, cfg.B, cfg.N)
        nn[3] = 0
    elif case == "ragged32":     # page size 32, 24 slots (96 rows)
        ctx = np.array([1, 31, 33, 500, 2047, 5000])
        cfg = W.scaled(base, B=len(ctx), N=24, page_size=32)
        nn, parent = _random_trees(rng, cfg.B, cfg.N)
    elif case in ("page8", "page64", "page128"):    # the other page sizes a 128-key tile can be cut into
        pg = int(case[4:])
        ctx = np.array([1, pg - 1, pg, pg + 1, 127, 129, 700, 2049, 4100])
        cfg = W.scaled(base, B=len(ctx), N=16, page_size=pg)
        nn, parent = _random_trees(rng, cfg.B, cfg.N)
    elif case == "wide":         # 64 query heads on 8 kv heads, 64 slots: 512 rows per kv head, four row blocks
        ctx = np.array([700, 2500, 40])
        cfg = W.scaled(base, B=len(ctx), N=64, Hq=64)
        nn, parent = _random_trees(rng, cfg.B, cfg.N, n_fixed=[64, 37, 5])
    elif case == "single":       # one slot per request: ordinary decode attention
        ctx = np.array([300, 4000, 9])
        cfg = W.scaled(base, B=len(ctx), N=8)
        nn, parent = _random_trees(rng, cfg.B, cfg.N, n_fixed=[1, 1, 1])
    elif case == "many":         # more requests than one planning pass handles per thread, all short
        ctx = rng.integers(1, 300, size=1500)
        cfg = W.scaled(base, B=len(ctx), N=4)
        nn, parent = _random_trees(rng, cfg.B, cfg.N)
    elif case == "rows256":      # 4 heads per group x 64 slots: two row blocks per kv head, the second partly filled
        ctx = np.array([900, 130, 2000])
        cfg = W.scaled(base, B=len(ctx), N=64)
        nn, parent = _random_trees(rng, cfg.B, cfg.N, n_fixed=[64, 40, 33])
    else:                        # chains as deep as the budget allows (every ancestor bit set)
        ctx = np.array([257, 1500])
        cfg = W.scaled(base, B=len(ctx), N=32)
        nn = np.array([32, 32], np.int32)
        parent = np.tile(np.arange(-1, 31, dtype=np.int32), (2, 1))
    _check(war, cfg, ctx, nn, parent, kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_structured_values_with_order_one_outputs(war, kernel):
    """Zero queries give a uniform softmax, so outputs are plain means of V rows (order one, exactly known), and a
    sibling's V must not leak: the hand-worked case scaled to head size 128."""
    with open(os.path.join(GOLD, "attention_case3.json")) as f:
        g = json.load(f)
    cfg = W.scaled(W.CONFIGS["tiny"], B=1, N=8)
    ctx = np.array([g["prefix_len"] + 1])
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    a.q.zero_(); a.v_pool.zero_()
    rows = g["prefix_v"] + g["slot_v"]
    page = int(a.page_table[0, 0])
    for pos, v in enumerate(rows):
        a.v_pool[page, :, pos, 0] = v[0]
        a.v_pool[page, :, pos, 1] = v[1]
    nn = np.array([3], np.int32)
    parent = np.array([g["parent"] + [-1] * 5], np.int32)
    got, lse, _ = U.run_attn(war, a, nn, parent, g["scale"], kernel)
    for j in range(3):
        np.testing.assert_allclose(got[0, j, :, :2], np.tile(np.array(g["out"][j]), (cfg.Hq, 1)), atol=4e-3)
        np.testing.assert_allclose(np.exp(lse[0, j]), g["lse_exp"][j], rtol=1e-4)
    assert np.abs(got[0, :3, :, 2:]).max() == 0.0


@pytest.mark.parametrize("kernel", KERNELS)
def test_needle_key_and_large_logits(war, kernel):
    """One key with a huge logit deep inside a long context: the output is that key's V row (order-one values,
    also a test of the running-max rescale: the needle sits after many ordinary tiles)."""
    cfg = W.scaled(W.CONFIGS["tiny"], B=2, N=4)
    ctx = np.array([3000, 2000])
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    nn = np.array([2, 1], np.int32)
    parent = np.array([[-1, 0, -1, -1], [-1, -1, -1, -1]], np.int32)
    pos = 2500
    page = int(a.page_table[0, pos // cfg.page_size])
    qv = a.q[0, 1, :, :].float()
    a.k_pool[page, :, pos % cfg.page_size, :] = (qv.view(cfg.Hkv, -1, cfg.D)[:, 0, :] * 3).to(torch.bfloat16)
    _check(war, cfg, ctx, nn, parent, kernel, a=a)
    got, _, _ = U.run_attn(war, a, nn, parent, 1.0 / np.sqrt(cfg.D), kernel)
    G = cfg.Hq // cfg.Hkv
    want = a.v_pool[page, :, pos % cfg.page_size, :].float().cpu().numpy()
    np.testing.assert_allclose(got[0, 1, ::G, :], want, atol=2e-2, rtol=2e-2)


def test_lse_is_optional_and_scale_is_an_argument(war):
    cfg = W.scaled(W.CONFIGS["tiny"], B=2, N=8)
    ctx = np.array([1300, 77])
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    nn, parent = _random_trees(np.random.default_rng(3), cfg.B, cfg.N)
    d_nn = torch.from_numpy(nn).to("cuda:0"); d_par = torch.from_numpy(parent).to("cuda:0")
    for scale in (0.02, 0.3):
        params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, scale, 0)
        ws = war.new_workspace(params, "cuda:0")
        out = torch.zeros_like(a.q)
        war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, d_nn, d_par, params, ws, out, None)
        torch.cuda.synchronize()
        want = A.verify_attention(a.q, a.k_pool, a.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(), nn, parent, scale)
        for i in range(cfg.B):
            n = int(nn[i])
            np.testing.assert_allclose(out[i, :n].float().cpu().numpy(), want[i][0].astype(np.float32), atol=1e-2, rtol=1e-2)
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, 0.0, 0)
    assert war.war_verify_attn_workspace_bytes(params) == 0          # scale must be positive


@pytest.mark.parametrize("kernel", KERNELS)
def test_page_permutation_leaves_bits_unchanged(war, kernel):
    cfg = W.scaled(W.CONFIGS["tiny"], B=3, N=16)
    ctx = np.array([1500, 700, 3100])
    rng = np.random.default_rng(2)
    nn, parent = _random_trees(rng, cfg.B, cfg.N)
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    _, _, raw1 = U.run_attn(war, a, nn, parent, 0.1, kernel)
    perm = torch.randperm(a.num_pages, generator=torch.Generator().manual_seed(1)).to("cuda:0")
    inv = torch.empty_like(perm); inv[perm] = torch.arange(a.num_pages, device="cuda:0")
    a.k_pool = a.k_pool[perm].contiguous(); a.v_pool = a.v_pool[perm].contiguous()
    pt = a.page_table.long()
    a.page_table = torch.where(pt >= 0, inv[pt.clamp(min=0)], pt).to(torch.int32)
    _, _, raw2 = U.run_attn(war, a, nn, parent, 0.1, kernel)
    assert torch.equal(raw1, raw2)


def test_kv_head_shards_equal_the_unsharded_call(war):
    """Tensor-parallel replicas shard the kv heads (and their query-head groups): a rank calls the library on its
    own slice of the pools and of q.  Outputs of the shards, put side by side, must equal the unsharded call bit for
    bit (each kv head is an independent problem)."""
    cfg = W.scaled(W.CONFIGS["tiny"], B=3, N=16)
    ctx = np.array([2100, 400, 900])
    rng = np.random.default_rng(5)
    nn, parent = _random_trees(rng, cfg.B, cfg.N)
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    _, _, full = U.run_attn(war, a, nn, parent, 0.09, 0)
    G = cfg.Hq // cfg.Hkv
    shards = []
    for r in range(2):                                                     # two ranks, four kv heads each
        h0, h1 = r * cfg.Hkv // 2, (r + 1) * cfg.Hkv // 2
        b = W.AttnInputs(q=a.q[:, :, h0 * G:h1 * G, :].contiguous(), k_pool=a.k_pool[:, h0:h1].contiguous(),
                         v_pool=a.v_pool[:, h0:h1].contiguous(), page_table=a.page_table, prefix_len=a.prefix_len,
                         num_pages=a.num_pages, max_pages=a.max_pages)
        _, _, part = U.run_attn(war, b, nn, parent, 0.09, 0)
        shards.append(part)
    assert torch.equal(torch.cat(shards, dim=2), full)


@pytest.mark.parametrize("kernel", KERNELS)
def test_malformed_inputs_are_reported_not_faulted(war, kernel):
    cfg = W.scaled(W.CONFIGS["tiny"], B=2, N=8)
    ctx = np.array([200, 300])
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    nn = np.array([3, 3], np.int32)
    parent = np.array([[-1, 0, 5, -1, -1, -1, -1, -1], [-1, 0, 1, -1, -1, -1, -1, -1]], np.int32)
    got, lse, _ = U.run_attn(war, a, nn, parent, 0.1, kernel)
    assert (got[0] == 7.0).all()                                             # the bad request is skipped
    assert (got[1, :3] != 7.0).any()
    assert war.war_device_status() == 7
    a.page_table[1, 2] = a.num_pages + 5                                     # a page index outside the pool
    U.run_attn(war, a, np.array([0, 3], np.int32), parent, 0.1, kernel)
    assert war.war_device_status() == 8


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("pg", [16, 32, 128])
def test_token_major_pools(war, kernel, pg):
    """Engines that store a page as [token][head][d] pass the same logical tensor with other strides.  The result
    must equal the head-major call bit for bit (same arithmetic, other addressing) and the checker within tolerance."""
    cfg = W.scaled(W.CONFIGS["tiny"], B=5, N=24, page_size=pg)
    ctx = np.array([1, pg + 1, 900, 2049, 5000])
    rng = np.random.default_rng(31 + pg)
    nn, parent = _random_trees(rng, cfg.B, cfg.N)
    a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    _, _, head_major = U.run_attn(war, a, nn, parent, 0.088, kernel)
    tm = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)       # same shape, (page, token, head, d) in memory
    b = W.AttnInputs(q=a.q, k_pool=tm(a.k_pool), v_pool=tm(a.v_pool), page_table=a.page_table, prefix_len=a.prefix_len,
                     num_pages=a.num_pages, max_pages=a.max_pages)
    assert b.k_pool.stride() == (pg * cfg.Hkv * cfg.D, cfg.D, cfg.Hkv * cfg.D, 1)
    _, raw = _check(war, cfg, ctx, nn, parent, kernel, scale=0.088, a=b)
    assert torch.equal(raw, head_major)
    # mixed layouts are refused
    c = W.AttnInputs(q=a.q, k_pool=b.k_pool, v_pool=a.v_pool, page_table=a.page_table, prefix_len=a.prefix_len,
                     num_pages=a.num_pages, max_pages=a.max_pages)
    assert war.war_verify_attn_workspace_bytes(war.attn_params(c.q, c.k_pool, c.v_pool, c.page_table, 0.088, kernel)) == 0


@pytest.mark.parametrize("seed", range(6))
def test_random_shapes_against_the_checker(war, seed):
    """Shapes drawn at random: batch, slots, heads per group, page size, pool layout, contexts from 1 token to a few
    thousand (so that single-tile requests, split requests, one-wave and many-unit plans, ragged last tiles and empty
    requests all occur together), random trees.  Every request is compared; the call is repeated for determinism."""
    rng = np.random.default_rng(900 + seed)
    for _ in range(4):
        G = int(rng.choice([1, 2, 4, 8]))
        Hkv = int(rng.choice([1, 2, 8]))
        N = int(rng.choice([1, 3, 8, 16, 33, 64]))
        while G * N > 512:
            N //= 2
        pg = int(rng.choice([8, 16, 32, 64, 128]))
        B = int(rng.integers(1, 12))
        ctx = rng.integers(1, int(rng.choice([40, 300, 2500, 6000])), size=B)
        cfg = W.scaled(W.CONFIGS["tiny"], B=B, N=N, Hq=G * Hkv, Hkv=Hkv, page_size=pg)
        nn, parent = _random_trees(rng, B, N)
        if B > 2:
            nn[int(rng.integers(0, B))] = 0                                   # a request that is not running
        a = W.make_attention_inputs(cfg, ctx, device="cuda:0")
        if rng.random() < 0.5:                                                # token-major pools
            tm = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            a = W.AttnInputs(q=a.q, k_pool=tm(a.k_pool), v_pool=tm(a.v_pool), page_table=a.page_table, prefix_len=a.prefix_len,
                             num_pages=a.num_pages, max_pages=a.max_pages)
        scale = float(rng.choice([0.05, 0.088, 0.2]))
        _, raw1 = _check(war, cfg, ctx, nn, parent, 0, scale=scale, a=a)
        _, _, raw2 = U.run_attn(war, a, nn, parent, scale, 0)
        assert torch.equal(raw1, raw2)


@pytest.mark.parametrize("kernel", [0, 2])
def test_workspace_contents_do_not_matter(war, kernel):
    """The workspace is scratch: whatever it holds before the call (zeros, ones, a pattern, another call's leftovers,
    noise), the results are the same bits.  On the one-launch path this is what the call numbers in the arrival
    counters of split requests are for; the contexts are long enough that every request is split."""
    rng = np.random.default_rng(77)
    cfg = W.scaled(W.CONFIGS["low"], B=5, N=12)
    ctx = np.array([9000, 14000, 700, 20000, 4100])
    a = W.make_attention_inputs(cfg, ctx, device=U.dev())
    nn, parent = _random_trees(rng, cfg.B, cfg.N)
    d_nn, d_par = torch.from_numpy(nn).to(U.dev()), torch.from_numpy(parent).to(U.dev())
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, 0.088, kernel)
    n_bytes = war.war_verify_attn_workspace_bytes(params)
    outs = []
    fills = [lambda n: torch.zeros(n, dtype=torch.uint8, device=U.dev()),
             lambda n: torch.full((n,), 0xFF, dtype=torch.uint8, device=U.dev()),
             lambda n: torch.full((n,), 0xA5, dtype=torch.uint8, device=U.dev()),
             lambda n: torch.randint(0, 256, (n,), dtype=torch.uint8, device=U.dev())]
    for fill in fills:
        ws = fill(n_bytes)
        for _ in range(2):                                                    # the second call finds the first one's leftovers
            out = torch.full(a.q.shape, 7.0, dtype=torch.bfloat16, device=U.dev())
            lse = torch.full(a.q.shape[:3], 7.0, dtype=torch.float32, device=U.dev())
            war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, d_nn, d_par, params, ws, out, lse)
            torch.cuda.synchronize()
            outs.append((out, lse))
    for out, lse in outs[1:]:
        assert torch.equal(out, outs[0][0]) and torch.equal(lse, outs[0][1])
    assert war.war_device_status() == 0
    want = A.verify_attention(a.q, a.k_pool, a.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(), nn, parent, 0.088)
    got, got_lse = outs[0][0].float().cpu().numpy(), outs[0][1].cpu().numpy()
    for i in range(cfg.B):
        U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], int(nn[i]))


@pytest.mark.parametrize("seed", range(12))
def test_mid_size_batches_through_every_plan(war, seed):
    """2-64 requests of four length mixes (long and uniform: the contiguous split when the trees have more than 64
    rows; short; lognormal; one very long among short ones: the chunk-length search), random trees, sampled requests
    against the fp64 checker."""
    rng = np.random.default_rng(7000 + seed)
    B = int(rng.integers(2, 65))
    Hkv, G, N, pg = int(rng.choice([2, 4, 8])), int(rng.choice([2, 4])), int(rng.integers(4, 33)), int(rng.choice([16, 32]))
    kind = seed % 4
    if kind == 0:
        ctx = rng.integers(16000, 30000, B)
    elif kind == 1:
        ctx = rng.integers(200, 9000, B)
    elif kind == 2:
        ctx = np.clip(np.exp(rng.normal(np.log(6000), 0.8, B)), 130, 40000).astype(int)
    else:
        ctx = np.concatenate([rng.integers(500, 3000, B - 1), rng.integers(30000, 60000, 1)])
    budget = 3e9                                                        # bytes of K/V held on the device
    if ctx.sum() * Hkv * 512 > budget:
        ctx = (ctx * (budget / (ctx.sum() * Hkv * 512))).astype(int) + 130
    cfg = W.scaled(W.CONFIGS["low"], B=B, N=N, Hkv=Hkv, Hq=Hkv * G, page_size=pg)
    a = W.make_attention_inputs(cfg, np.asarray(ctx), device=U.dev())
    nn = rng.integers(1, N + 1, B).astype(np.int32)
    par = np.full((B, N), -1, np.int32)
    for i in range(B):
        for j in range(1, nn[i]):
            par[i, j] = int(rng.integers(0, j))
    scale = 1.0 / np.sqrt(cfg.D)
    got, got_lse, raw = U.run_attn(war, a, nn, par, scale, 0)
    # the one-launch path (every CTA plans for itself, the last CTA of a split unit merges) takes the same decisions as
    # the three-launch path and adds the partials in the same order: the bits are the same
    got3, got3_lse, raw3 = U.run_attn(war, a, nn, par, scale, 2)
    assert torch.equal(raw, raw3) and (got_lse == got3_lse).all()
    sample = sorted({0, B - 1, int(np.argmax(ctx)), int(rng.integers(0, B))})
    want = A.verify_attention(a.q, a.k_pool, a.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(), nn, par, scale,
                              requests=sample)
    for i in sample:
        U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], int(nn[i]))
    assert war.war_device_status() == 0
    del a
    torch.cuda.empty_cache()


@pytest.mark.parametrize("B,N,G", [(1, 32, 4), (2, 32, 4), (3, 24, 4), (2, 8, 4), (1, 64, 8), (4, 16, 4)])
def test_few_requests_whose_merges_are_shared_out(war, B, N, G):
    """With a handful of long requests every (request, kv head, row block) is cut into many chunks and its merge is
    shared out to two, four or eight CTAs, a share of the rows each, which count themselves on a second counter word
    before the last one clears both.  Checked against the fp64 checker, bit for bit against the three-launch path, and
    on repeated calls and graph replays with one and the same workspace (the counters must come back to a state in which
    the next call, or the replay with its frozen call number, starts from nothing)."""
    rng = np.random.default_rng(4100 + 10 * B + N)
    Hkv = 8
    ctx = rng.integers(14000, 26000, B)
    cfg = W.scaled(W.CONFIGS["low"], B=B, N=N, Hkv=Hkv, Hq=Hkv * G, page_size=16)
    a = W.make_attention_inputs(cfg, np.asarray(ctx), device=U.dev())
    nn = np.full(B, N, np.int32)
    nn[-1] = max(1, N - 3)
    par = np.full((B, N), -1, np.int32)
    for i in range(B):
        for j in range(1, nn[i]):
            par[i, j] = int(rng.integers(0, j))
    scale = 1.0 / np.sqrt(cfg.D)
    d = U.dev()
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, scale, 0)
    ws = torch.full((war.war_verify_attn_workspace_bytes(params),), 0xa5, dtype=torch.uint8, device=d)
    d_nn, d_par = torch.from_numpy(nn).to(d), torch.from_numpy(par).to(d)
    outs = []
    for _ in range(3):
        out = torch.full(a.q.shape, 7.0, dtype=torch.bfloat16, device=d)
        lse = torch.full(a.q.shape[:3], 7.0, dtype=torch.float32, device=d)
        war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, d_nn, d_par, params, ws, out, lse)
        torch.cuda.synchronize()
        outs.append((out, lse))
    g_out = torch.full(a.q.shape, 7.0, dtype=torch.bfloat16, device=d)
    g_lse = torch.full(a.q.shape[:3], 7.0, dtype=torch.float32, device=d)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, d_nn, d_par, params, ws, g_out, g_lse)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        g_out.fill_(7.0)
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(g_out, outs[0][0]) and torch.equal(g_lse, outs[0][1])
    assert all(torch.equal(o, outs[0][0]) and torch.equal(l, outs[0][1]) for o, l in outs[1:])
    got3, got3_lse, raw3 = U.run_attn(war, a, nn, par, scale, 2)
    live = torch.arange(N, device=d)[None, :] < d_nn[:, None]
    assert torch.equal(outs[0][0][live], raw3[live]) and torch.equal(outs[0][1][live], torch.from_numpy(got3_lse).to(d)[live])
    want = A.verify_attention(a.q, a.k_pool, a.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(), nn, par, scale)
    got, got_lse = outs[0][0].float().cpu().numpy(), outs[0][1].cpu().numpy()
    for i in range(B):
        U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], int(nn[i]))
    assert war.war_device_status() == 0
    del a
    torch.cuda.empty_cache()


def test_a_wait_that_runs_out_ends_with_an_error_not_a_hang(war):
    """Every wait inside the tensor-core kernel has a time budget.  The library's self-test runs the same wait routine
    on a barrier that nobody completes: the waiter gives up after its budget (here 1 ms instead of the kernel's 2 s),
    WAR_ERR_TIMEOUT is recorded, a second waiter is released by the first one's abort flag long before its own budget,
    the kernel returns normally, and the library works afterwards."""
    d = U.dev()
    assert war.war_device_status() == 0
    res = torch.full((4,), -1, dtype=torch.int64, device=d)
    war.war_selftest_bounded_wait(1000, res)
    torch.cuda.synchronize()
    ok0, ok1, ns0, ns1 = res.cpu().tolist()
    assert ok0 == 0 and ok1 == 0                                     # both waits gave up
    assert 1_000_000 <= ns0 < 200_000_000                            # the first after its budget (not the 2 s default)
    assert ns1 < 200_000_000                                         # the second because the first raised the flag
    assert war.war_device_status() == 5                              # WAR_ERR_TIMEOUT, read and cleared
    assert war.war_device_status() == 0
    with pytest.raises(war.WarError):
        war.war_selftest_bounded_wait(0, res)
    # the context is intact: an ordinary call right after
    rng = np.random.default_rng(5)
    cfg = W.scaled(W.CONFIGS["tiny"], B=3, N=8)
    nn, parent = _random_trees(rng, cfg.B, cfg.N)
    _check(war, cfg, np.array([900, 130, 2500]), nn, parent, 0)
