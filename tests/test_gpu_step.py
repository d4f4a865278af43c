"""GPU parity of the whole step (draft -> verify attention -> accept) on the small configuration, and, at the
benchmark's full sizes, on sampled requests the checker can afford one by one."""
import numpy as np
import pytest
import torch

from oracle import accept_oracle as C
from oracle import attention_oracle as A
from oracle import draft_oracle as D
from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _step(war, cfg, sample, kernel=0, draft_sample=None):
    """`sample`: requests whose attention is checked; `draft_sample`: requests whose trees are checked (default: the same)."""
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    ctx = W.context_lengths(cfg)
    ix = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + cfg.N)
    ml, nn, ids, par, cnt = U.run_draft(war, ix, tails, tl, cfg.N, cfg.topk)
    corpus = D.Corpus(tok, off)
    for i in (sample if draft_sample is None else draft_sample):        # brute-force scan per sampled request
        m, ends = D.longest_suffix_match(corpus, tails[i], int(tl[i]))
        a, b, c = D.build_draft_tree(corpus, tails[i], m, ends, cfg.N, cfg.topk)
        n = len(a)
        assert ml[i] == m and nn[i] == n
        assert (ids[i, :n] == a).all() and (par[i, :n] == b).all() and (cnt[i, :n] == c).all()
        assert (ids[i, n:] == -1).all()
    ix.destroy()
    # properties that hold at any size
    assert (nn >= 1).all() and (nn <= cfg.N).all() and (ml <= tl).all()
    for i in range(cfg.B):
        n = int(nn[i])
        assert par[i, 0] == -1 and (par[i, 1:n] < np.arange(1, n)).all() and (par[i, 1:n] >= 0).all()
        assert (cnt[i, 1:n] <= cnt[i, par[i, 1:n]]).all()
        assert (np.diff(cnt[i, 1:n]) <= 0).all()
    a_in = W.make_attention_inputs(cfg, ctx, device="cuda:0")
    scale = 1.0 / np.sqrt(cfg.D)
    got, got_lse, _ = U.run_attn(war, a_in, nn, par, scale, kernel)
    pt = a_in.page_table.cpu().numpy(); pl = a_in.prefix_len.cpu().numpy()
    want = A.verify_attention(a_in.q, a_in.k_pool, a_in.v_pool, pt, pl, nn, par, scale, requests=sample)
    for i in sample:
        U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], int(nn[i]))
    assert np.isfinite(got[np.arange(cfg.N)[None, :] < nn[:, None]]).all()
    del a_in
    target = W.make_targets(cfg, ids, par, nn, mode=0)
    alen, path, bonus = U.run_accept(war, ids, par, nn, target, 0)
    w_alen, w_path, w_bonus = C.accept_batch(ids, par, nn, target, 0)
    assert (alen == w_alen).all() and (path == w_path).all() and (bonus == w_bonus).all()
    assert war.war_device_status() == 0
    return ml, nn, alen


def test_tiny_step_every_request(war):
    cfg = W.CONFIGS["tiny"]
    _step(war, cfg, sample=list(range(cfg.B)))


@pytest.mark.parametrize("name,sample", [("high", [0, 17, 101, 255]), ("low", [3, 30]), ("longtail", [5, 41]), ("wide", [7])])
def test_full_size_sampled(war, name, sample):
    cfg = W.CONFIGS[name]
    ctx = W.context_lengths(cfg)
    longest, shortest = int(np.argmax(ctx)), int(np.argmin(ctx))
    ml, nn, alen = _step(war, cfg, sample=sorted(set(sample + [longest, shortest])))
    torch.cuda.empty_cache()


@pytest.mark.slow
def test_high_workload_every_request(war):
    """The configuration the metric is quoted on, in full: match lengths, trees and counts of all 256 requests against
    the brute-force checker, acceptance of all 256 by path enumeration, attention of 32 requests (every eighth, plus
    the longest and the shortest context) against the fp64 checker."""
    cfg = W.CONFIGS["high"]
    ctx = W.context_lengths(cfg)
    sample = sorted(set(range(0, cfg.B, 8)) | {int(np.argmax(ctx)), int(np.argmin(ctx))})
    _step(war, cfg, sample=sample, draft_sample=list(range(cfg.B)))
    torch.cuda.empty_cache()


def test_contiguous_split_beyond_32_requests(war):
    """48 requests of the Low recipe (128 query rows per kv head, pairs of 128-256 tiles): the attention plan cuts the
    whole tile sequence into equal ranges, two requests per planning lane; sampled requests against the checker."""
    cfg = W.scaled(W.CONFIGS["low"], B=48)
    ctx = W.context_lengths(cfg)
    _step(war, cfg, sample=sorted({0, 23, 47, int(np.argmax(ctx)), int(np.argmin(ctx))}))
    torch.cuda.empty_cache()
