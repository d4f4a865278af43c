"""GPU parity: suffix index and draft trees, bit-exact against the brute-force checker, through the C-ABI."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import draft_oracle as D
from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _flat(trajs):
    off = np.zeros(len(trajs) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(t) for t in trajs])
    tok = np.concatenate([np.asarray(t, dtype=np.int32) for t in trajs]) if len(trajs) else np.zeros(0, np.int32)
    return tok, off


def _read_device(ptr, nbytes):
    """Copies raw device memory to the host (test-only peek at the index internals)."""
    import ctypes
    cudart = ctypes.CDLL("libcudart.so.12")
    host = np.empty(nbytes, dtype=np.uint8)
    rc = cudart.cudaMemcpy(ctypes.c_void_p(host.ctypes.data), ctypes.c_void_p(ptr), ctypes.c_size_t(nbytes), 2)
    assert rc == 0
    return host


def _compare_with_oracle(war, tok, off, vocab, tails, tl, N, k, min_match=1, ix=None):
    own = ix is None
    if own:
        ix = U.build_index(war, tok, off, vocab)
    got = U.run_draft(war, ix, tails, tl, N, k, min_match)
    want = D.draft_batch(D.Corpus(tok, off), tails, tl, N, k, min_match)
    names = ["match_len", "num_nodes", "ids", "parent", "count"]
    for name, g, w in zip(names, got, want):
        assert (g == w).all(), f"{name} differs at request(s) {np.flatnonzero((g != w).reshape(len(g), -1).any(axis=1))[:8]}"
    assert war.war_device_status() == 0
    if own:
        ix.destroy()
    return got


def test_textbook_suffix_array_and_lcp(war):
    """'banana$' with a=1, b=2, n=3: the suffix array and LCP array every textbook prints."""
    tok, off = _flat([[2, 1, 3, 1, 3, 1]])
    ix = U.build_index(war, tok, off, vocab=4)
    info = war.war_index_info(ix)
    assert info.M == 7 and info.T == 1
    sa = _read_device(info.d_sa, 7 * 4).view(np.int32)
    lcp = _read_device(info.d_lcp, 7)
    corpus = _read_device(info.d_corpus, 7 * 4).view(np.int32)
    bucket = _read_device(info.d_bucket, 5 * 4).view(np.int32)
    assert corpus.tolist() == [2, 1, 3, 1, 3, 1, -1]
    assert sa.tolist() == [6, 5, 3, 1, 0, 4, 2]
    assert lcp.tolist() == [0, 0, 1, 3, 0, 0, 2]
    assert bucket.tolist() == [1, 1, 4, 5, 7]
    ix.destroy()


@pytest.mark.parametrize("seed", range(3))
def test_suffix_array_equals_naive_sort(war, seed):
    rng = np.random.default_rng(seed)
    trajs = [rng.integers(0, 4, size=int(rng.integers(0, 300))).tolist() for _ in range(7)]
    tok, off = _flat(trajs)
    depth = 96
    ix = U.build_index(war, tok, off, vocab=4, max_depth=depth)
    info = war.war_index_info(ix)
    M = int(info.M)
    assert M == len(tok) + len(trajs)
    sa = _read_device(info.d_sa, M * 4).view(np.int32)
    lcp = _read_device(info.d_lcp, M)
    corpus = _read_device(info.d_corpus, M * 4).view(np.int32).tolist()
    assert sorted(sa.tolist()) == list(range(M))                       # a permutation
    naive = sorted(range(M), key=lambda i: corpus[i:])                 # separators are negative and unique
    # order is only promised to depth 128 (the doubling's reach); beyond that ties may remain in any order
    key = lambda i: corpus[i:i + 128]
    assert [key(i) for i in sa] == [key(i) for i in naive]
    for i in range(1, M):
        a, b = corpus[sa[i - 1]:], corpus[sa[i]:]
        l = 0
        while l < min(len(a), len(b), depth) and a[l] == b[l]:
            l += 1
        assert lcp[i] == l
    ix.destroy()


@pytest.mark.parametrize("name", ["draft_case1.json", "draft_case2.json"])
def test_hand_worked_cases(war, name):
    with open(os.path.join(GOLD, name)) as f:
        g = json.load(f)
    tok, off = _flat(g["trajectories"])
    ix = U.build_index(war, tok, off, vocab=16)
    tail = np.array([g["tail"]], dtype=np.int32)
    for tr in g["trees"]:
        ml, nn, ids, par, cnt = U.run_draft(war, ix, tail, np.array([g["tail_len"]]), tr["N"], tr["k"])
        n = len(tr["ids"])
        assert ml[0] == g["match_len"] and nn[0] == n
        assert ids[0, :n].tolist() == tr["ids"] and par[0, :n].tolist() == tr["parent"] and cnt[0, :n].tolist() == tr["count"]
        assert (ids[0, n:] == -1).all() and (par[0, n:] == -1).all() and (cnt[0, n:] == 0).all()
    ix.destroy()


@pytest.mark.parametrize("seed", range(12))
def test_tiny_alphabets_force_ties(war, seed):
    rng = np.random.default_rng(100 + seed)
    vocab = int(rng.integers(2, 6))
    trajs = [rng.integers(0, vocab, size=int(rng.integers(0, 120))).tolist() for _ in range(int(rng.integers(1, 9)))]
    tok, off = _flat(trajs)
    P = int(rng.integers(1, 33))
    N = int(rng.integers(1, 65))
    k = int(rng.integers(1, 9))
    B = 24
    tails = rng.integers(0, vocab + 1, size=(B, P)).astype(np.int32)
    tails[0, :] = -1                                                   # negative ids must never match a separator
    tl = rng.integers(0, P + 1, size=B).astype(np.int32)
    _compare_with_oracle(war, tok, off, vocab + 1, tails, tl, N, k, min_match=int(rng.integers(0, 4)))


def test_tiny_config_with_structured_tails(war):
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    rng = np.random.default_rng(5)
    extra, extra_len = [], []
    for _ in range(24):                                                # tails planted inside the corpus
        t = int(rng.integers(0, cfg.n_traj)); dist = int(rng.integers(1, 300))
        e = int(off[t]) + dist; m = min(cfg.P, dist)
        row = np.full(cfg.P, -1, np.int32); row[cfg.P - m:] = tok[e - m:e]
        extra.append(row); extra_len.append(m)
    for v in (0, 1, 2, 5, 17):                                         # one-token matches on the most frequent ids:
        row = np.full(cfg.P, cfg.vocab + 3, np.int32); row[-1] = v      # the largest intervals (block-wide scans)
        extra.append(row); extra_len.append(cfg.P)
    row = np.full(cfg.P, cfg.vocab + 9, np.int32); extra.append(row); extra_len.append(cfg.P)   # never seen
    for t in range(3):                                                 # the very end of a trajectory: no continuation
        row = tok[off[t + 1] - cfg.P:off[t + 1]].copy(); extra.append(row); extra_len.append(cfg.P)
    tails = np.concatenate([tails, np.stack(extra)]); tl = np.concatenate([tl, np.array(extra_len, np.int32)])
    got = _compare_with_oracle(war, tok, off, cfg.vocab, tails, tl, cfg.N, cfg.topk)
    assert got[4][:, 0].max() >= 8192                                  # a block-wide scan really happened
    for N, k in ((64, 8), (8, 4), (2, 1), (1, 4), (33, 3)):
        _compare_with_oracle(war, tok, off, cfg.vocab, tails, tl, N, k)


def test_append_equals_rebuild_and_order_independence(war):
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    T = cfg.n_traj
    cut1, cut2 = 20, 45
    cap = len(tok) + T
    ix = U.build_index(war, tok[:off[cut1]], off[:cut1 + 1], cfg.vocab, capacity=cap)
    d_tok = torch.from_numpy(tok).to("cuda:0")
    war.war_index_append(ix, d_tok, off[cut1:cut2 + 1])                # offsets index into d_tok
    war.war_index_append(ix, d_tok, off[cut2:])
    assert war.war_index_info(ix).M == cap and war.war_index_info(ix).T == T
    _compare_with_oracle(war, tok, off, cfg.vocab, tails, tl, cfg.N, cfg.topk, ix=ix)
    with pytest.raises(war.WarError) as e:
        war.war_index_append(ix, d_tok, off[:2])
    assert e.value.code == 3                                           # capacity; the index is unchanged
    assert war.war_index_info(ix).M == cap
    _compare_with_oracle(war, tok, off, cfg.vocab, tails, tl, cfg.N, cfg.topk, ix=ix)
    ix.destroy()
    # same trajectories in another arrival order: same drafts
    order = np.random.default_rng(3).permutation(T)
    trajs = [tok[off[t]:off[t + 1]] for t in order]
    tok2, off2 = _flat(trajs)
    ix2 = U.build_index(war, tok2, off2, cfg.vocab)
    a = U.run_draft(war, ix2, tails, tl, cfg.N, cfg.topk)
    want = D.draft_batch(D.Corpus(tok, off), tails, tl, cfg.N, cfg.topk)
    for g, w in zip(a, want):
        assert (g == w).all()
    ix2.destroy()


@pytest.mark.parametrize("seed", range(3))
def test_incremental_appends_keep_a_valid_suffix_array(war, seed):
    """Small appends take the merge path (new suffixes sorted on their own, then merged into the old order).  After
    every append the suffix array must be a depth-ordered permutation with correct LCP and buckets, and drafts must
    equal the brute-force checker's on everything stored so far."""
    rng = np.random.default_rng(40 + seed)
    vocab = 5
    trajs = [rng.integers(0, vocab, size=int(rng.integers(0, 400))).tolist() for _ in range(14)]
    tok, off = _flat(trajs)
    d_tok = torch.from_numpy(tok).to("cuda:0")
    cap = len(tok) + len(trajs)
    ix = U.build_index(war, tok[:off[6]], off[:7], vocab, max_depth=96, capacity=cap)
    tails = rng.integers(0, vocab, size=(40, 12)).astype(np.int32)
    tl = rng.integers(0, 13, size=40).astype(np.int32)
    done = 6
    for step in (1, 2, 1, 3, 1):                                        # each addition is smaller than what is stored
        war.war_index_append(ix, d_tok, off[done:done + step + 1])
        done += step
        info = war.war_index_info(ix)
        M = int(info.M)
        assert M == off[done] + done and info.T == done
        sa = _read_device(info.d_sa, M * 4).view(np.int32)
        lcp = _read_device(info.d_lcp, M)
        corpus = _read_device(info.d_corpus, M * 4).view(np.int32).tolist()
        bucket = _read_device(info.d_bucket, (vocab + 1) * 4).view(np.int32)
        assert sorted(sa.tolist()) == list(range(M))
        key = lambda i: corpus[i:i + 128]
        naive = sorted(range(M), key=lambda i: corpus[i:])
        assert [key(i) for i in sa] == [key(i) for i in naive]
        for i in range(1, M):
            a, b = corpus[sa[i - 1]:], corpus[sa[i]:]
            l = 0
            while l < min(len(a), len(b), 96) and a[l] == b[l]:
                l += 1
            assert lcp[i] == l
        firsts = np.array([corpus[i] for i in sa])
        for v in range(vocab + 1):
            assert bucket[v] == int((firsts < v).sum())
        _compare_with_oracle(war, tok[:off[done]], off[:done + 1], vocab, tails, tl, 24, 4, ix=ix)
    ix.destroy()


def test_empty_and_degenerate_inputs(war):
    ix = U.build_index(war, np.zeros(0, np.int32), np.zeros(1, np.int64), vocab=10, capacity=64)   # no trajectories
    tails = np.array([[1, 2, 3, 4]], np.int32)
    ml, nn, ids, par, cnt = U.run_draft(war, ix, tails, np.array([4]), 8, 4)
    assert ml[0] == 0 and nn[0] == 1 and ids[0, 0] == 4 and cnt[0, 0] == 0
    d_tok = torch.tensor([1, 2, 3, 4, 5], dtype=torch.int32, device="cuda:0")
    war.war_index_append(ix, d_tok, np.array([0, 0, 5, 5]))            # empty trajectories around a real one
    ml, nn, ids, par, cnt = U.run_draft(war, ix, tails, np.array([4]), 8, 4, with_count=False)
    assert ml[0] == 4 and nn[0] == 2 and ids[0, :2].tolist() == [4, 5] and cnt is None
    for bad in (10, -1):                                               # ids outside [0, vocab) are refused, nothing changes
        with pytest.raises(war.WarError) as e:
            war.war_index_append(ix, torch.tensor([1, bad, 3], dtype=torch.int32, device="cuda:0"), np.array([0, 3]))
        assert e.value.code == 1
    assert war.war_index_info(ix).M == 8 and war.war_index_info(ix).T == 3
    ml, nn, ids, par, cnt = U.run_draft(war, ix, tails, np.array([4]), 8, 4)
    assert ml[0] == 4 and nn[0] == 2 and ids[0, :2].tolist() == [4, 5]
    ix.destroy()


def test_workload_aware_switch(war):
    """Requests with tail_len < 0 are not running; above the limit every running request gets the root alone."""
    cfg = W.scaled(W.CONFIGS["tiny"], B=24)
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    tl = tl.copy(); tl[[3, 11, 17]] = -1                               # 21 running
    corpus = D.Corpus(tok, off)
    ix = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + cfg.N)
    for limit in (0, 21, 20, 1):
        got = U.run_draft(war, ix, tails, tl, cfg.N, cfg.topk, spec_batch_limit=limit)
        want = D.draft_batch(corpus, tails, tl, cfg.N, cfg.topk, spec_batch_limit=limit)
        for g, w in zip(got, want):
            assert np.array_equal(g, w), limit
        assert (got[1][[3, 11, 17]] == 0).all()
        assert (got[1].max() > 1) == (limit in (0, 21))
    ix.destroy()


@pytest.mark.parametrize("seed", range(2))
def test_evicting_the_oldest_trajectories_equals_a_fresh_build(war, seed):
    """A sliding window over the trajectory stream: append, evict the oldest, append again.  After every change the
    suffix array must be a depth-ordered permutation of what is stored, with exact LCP and buckets and separators
    numbered from the first stored trajectory, and drafts must equal the brute-force checker's on the window."""
    rng = np.random.default_rng(70 + seed)
    vocab = 5
    trajs = [rng.integers(0, vocab, size=int(rng.integers(0, 300))).tolist() for _ in range(16)]
    tok, off = _flat(trajs)
    d_tok = torch.from_numpy(tok).to("cuda:0")
    ix = U.build_index(war, tok[:off[8]], off[:9], vocab, max_depth=96, capacity=len(tok) + len(trajs))
    tails = rng.integers(0, vocab, size=(40, 12)).astype(np.int32)
    tl = rng.integers(0, 13, size=40).astype(np.int32)
    first, done = 0, 8

    def check():
        info = war.war_index_info(ix)
        M = int(info.M)
        assert info.T == done - first and M == (off[done] - off[first]) + (done - first)
        wtok, woff = tok[off[first]:off[done]], off[first:done + 1] - off[first]
        if M:
            sa = _read_device(info.d_sa, M * 4).view(np.int32)
            lcp = _read_device(info.d_lcp, M)
            corpus = _read_device(info.d_corpus, (M + 8) * 4).view(np.int32).tolist()
            assert corpus[M:] == [-1] * 8                                # the vacated end reads as "no token"
            corpus = corpus[:M]
            assert [v for v in corpus if v < 0] == [-(t + 1) for t in range(done - first)]
            assert [v for v in corpus if v >= 0] == wtok.tolist()
            assert sorted(sa.tolist()) == list(range(M))
            naive = sorted(range(M), key=lambda i: corpus[i:])
            assert [corpus[i:i + 128] for i in sa] == [corpus[i:i + 128] for i in naive]
            for i in range(1, M):
                a, b = corpus[sa[i - 1]:], corpus[sa[i]:]
                l = 0
                while l < min(len(a), len(b), 96) and a[l] == b[l]:
                    l += 1
                assert lcp[i] == l
            bucket = _read_device(info.d_bucket, (vocab + 1) * 4).view(np.int32)
            firsts = np.array([corpus[i] for i in sa])
            for v in range(vocab + 1):
                assert bucket[v] == int((firsts < v).sum())
        _compare_with_oracle(war, wtok, woff, vocab, tails, tl, 24, 4, ix=ix)

    for evict, add in ((3, 2), (0, 1), (4, 3), (1, 2)):
        war.war_index_evict(ix, evict); first += evict
        check()
        war.war_index_append(ix, d_tok, off[done:done + add + 1]); done += add
        check()
    with pytest.raises(war.WarError):
        war.war_index_evict(ix, done - first + 1)                        # more than is stored
    war.war_index_evict(ix, done - first); first = done                  # everything: an empty index still answers
    check()
    war.war_index_append(ix, d_tok, off[0:3]); first, done = 0, 2       # and can be filled again
    check()
    ix.destroy()


@pytest.mark.parametrize("spec_factor,min_prob", [((1, 1), (0, 1)), ((2, 3), (0, 1)), ((0, 1), (1, 2)), ((0, 1), (1, 10)),
                                                  ((3, 1), (1, 4)), ((1, 8), (1, 1))])
def test_node_budget_and_probability_threshold(war, spec_factor, min_prob):
    """The two thresholds against the brute-force checker: the Tiny workload (template matches and junk matches) and
    a tiny alphabet with heavy ties and large intervals (block-wide scans, chains)."""
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(W.scaled(cfg, B=48))
    ix = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + 64)
    corpus = D.Corpus(tok, off)
    for N, k in ((16, 4), (64, 8)):
        got = U.run_draft(war, ix, tails, tl, N, k, spec_factor=spec_factor, min_prob=min_prob)
        want = D.draft_batch(corpus, tails, tl, N, k, spec_factor=spec_factor, min_prob=min_prob)
        for g, w in zip(got, want):
            assert np.array_equal(g, w)
    ix.destroy()
    rng = np.random.default_rng(17)
    trajs = [rng.integers(0, 3, size=int(rng.integers(50, 3000))).tolist() for _ in range(12)]
    tok2, off2 = _flat(trajs)
    tails2 = rng.integers(0, 3, size=(40, 10)).astype(np.int32)
    tl2 = rng.integers(0, 11, size=40).astype(np.int32)
    ix2 = U.build_index(war, tok2, off2, 3, max_depth=96)
    got = U.run_draft(war, ix2, tails2, tl2, 32, 3, spec_factor=spec_factor, min_prob=min_prob)
    want = D.draft_batch(D.Corpus(tok2, off2), tails2, tl2, 32, 3, spec_factor=spec_factor, min_prob=min_prob)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    assert war.war_device_status() == 0
    ix2.destroy()


def test_drafts_keep_running_while_the_index_is_updated(war):
    """war_index_append builds the new arrays beside the published ones and publishes them when they are complete
    (the paper updates the cache asynchronously so that the update does not block the pipeline, Section 3.3).  One
    thread drafts in a loop on its own stream while another appends twice; every draft result must equal the
    brute-force checker's answer on one of the three corpus states, and the states must appear in order."""
    import threading
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(W.scaled(cfg, B=32))
    T = cfg.n_traj
    cuts = [T - 24, T - 10, T]
    d_tok = torch.from_numpy(tok).to("cuda:0")
    ix = U.build_index(war, tok[:off[cuts[0]]], off[:cuts[0] + 1], cfg.vocab, max_depth=cfg.P + cfg.N, capacity=len(tok) + T)
    wants = [D.draft_batch(D.Corpus(tok[:off[c]], off[:c + 1]), tails, tl, cfg.N, cfg.topk) for c in cuts]
    assert not all(np.array_equal(a, b) for a, b in zip(wants[0], wants[2]))     # the appends change some draft
    results, errors, stop = [], [], threading.Event()

    def drafter():
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                while not stop.is_set() or len(results) < 3:
                    results.append(U.run_draft(war, ix, tails, tl, cfg.N, cfg.topk))
                    if len(results) > 4000:
                        break
        except Exception as e:                                       # noqa: BLE001
            errors.append(e)

    th = threading.Thread(target=drafter)
    th.start()
    s2 = torch.cuda.Stream()
    with torch.cuda.stream(s2):
        while len(results) < 5 and th.is_alive():
            pass
        war.war_index_append(ix, d_tok, off[cuts[0]:cuts[1] + 1])
        n1 = len(results)
        while len(results) < n1 + 5 and th.is_alive():
            pass
        war.war_index_append(ix, d_tok, off[cuts[1]:cuts[2] + 1])
        n2 = len(results)
        while len(results) < n2 + 5 and th.is_alive():
            pass
    stop.set()
    th.join(timeout=60)
    assert not errors and not th.is_alive()
    state = 0
    for got in results:
        while state < 3 and not all(np.array_equal(g, w) for g, w in zip(got, wants[state])):
            state += 1
        assert state < 3, "a draft matched none of the corpus states (or went back to an older one)"
    assert state == 2                                                 # the last drafts saw everything
    assert war.war_device_status() == 0
    ix.destroy()


def test_stream_ordered_append_from_one_thread(war):
    """war_index_append_async only enqueues the update: ONE host thread starts it on a side stream and goes on
    drafting on its main stream.  Every draft enqueued meanwhile equals the checker's answer on the corpus before or
    after the update (never anything else), drafts ordered behind the update see the grown corpus, two updates
    enqueued back to back on one stream land in order, a full re-sort (the addition larger than what is stored) and a
    merge both come out as a fresh build would, and a token outside the vocabulary becomes an end-of-trajectory mark
    with WAR_ERR_INVALID_ARG in the device status."""
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(W.scaled(cfg, B=32))
    T = cfg.n_traj
    cuts = [6, 20, 44, T]                                             # 6 -> 20 is a full re-sort, the others merge
    dev = U.dev()
    d_tok = torch.from_numpy(tok).to(dev)
    N, k = cfg.N, cfg.topk
    ix = U.build_index(war, tok[:off[cuts[0]]], off[:cuts[0] + 1], cfg.vocab, max_depth=cfg.P + N, capacity=len(tok) + T + 64)
    wants = [D.draft_batch(D.Corpus(tok[:off[c]], off[:c + 1]), tails, tl, N, k) for c in cuts]
    same = lambda got, want: all(np.array_equal(g, w) for g, w in zip(got, want))
    side = torch.cuda.Stream()
    main = torch.cuda.current_stream()
    i32 = dict(dtype=torch.int32, device=dev)
    d_tails, d_tl = torch.from_numpy(tails).to(dev), torch.from_numpy(tl).to(dev)

    def enqueue_draft():
        bufs = [torch.full((32,), -7, **i32), torch.full((32,), -7, **i32)] + [torch.full((32, N), -7, **i32) for _ in range(3)]
        war.war_draft(ix, d_tails, d_tl, N, k, 1, *bufs)
        return bufs

    for step in range(1, 4):
        side.wait_stream(main)
        with torch.cuda.stream(side):
            war.war_index_append_async(ix, d_tok[off[cuts[step - 1]]:off[cuts[step]]], off[cuts[step - 1]:cuts[step] + 1] - off[cuts[step - 1]])
        assert war.war_index_info(ix).T == cuts[step]                 # the handle's host side has advanced already
        during = [enqueue_draft() for _ in range(6)]                  # not ordered against the update: old or new
        main.wait_stream(side)
        after = enqueue_draft()                                       # ordered behind it: new
        torch.cuda.synchronize()
        for bufs in during:
            got = [b.cpu().numpy() for b in bufs]
            assert same(got, wants[step - 1]) or same(got, wants[step])
        assert same([b.cpu().numpy() for b in after], wants[step])
    # the arrays themselves equal a fresh build's up to the order of suffixes that agree to the full depth: compare lcp and buckets
    info = war.war_index_info(ix)
    fresh = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + N)
    f_info = war.war_index_info(fresh)
    M = int(info.M)
    assert M == int(f_info.M)
    torch.cuda.synchronize()
    lcp_a = _read_device(info.d_lcp, M); lcp_b = _read_device(f_info.d_lcp, M)
    assert np.array_equal(lcp_a, lcp_b)
    fresh.destroy()
    # two updates back to back on one stream, then an eviction ordered behind them
    ix2 = U.build_index(war, tok[:off[30]], off[:31], cfg.vocab, max_depth=cfg.P + N, capacity=len(tok) + T + 64)
    with torch.cuda.stream(side):
        war.war_index_append_async(ix2, d_tok[off[30]:off[40]], off[30:41] - off[30])
        war.war_index_append_async(ix2, d_tok[off[40]:off[T]], off[40:T + 1] - off[40])
        war.war_index_evict(ix2, 7)                                   # (synchronises the side stream itself)
    got = U.run_draft(war, ix2, tails, tl, N, k)
    want = D.draft_batch(D.Corpus(tok[off[7]:], off[7:] - off[7]), tails, tl, N, k)
    assert same(got, want)
    assert war.war_device_status() == 0
    # a token outside the vocabulary: recorded, stored as an end-of-trajectory mark
    bad = np.array([5, 9, cfg.vocab + 3, 9, 5, 9], np.int32)
    with torch.cuda.stream(side):
        war.war_index_append_async(ix2, torch.from_numpy(bad).to(dev), np.array([0, 6], np.int64))
    side.synchronize()
    assert war.war_device_status() == 1                               # WAR_ERR_INVALID_ARG
    hist_tok = np.concatenate([tok[off[7]:], bad[:2], bad[3:]])
    hist_off = np.concatenate([off[7:] - off[7], [off[T] - off[7] + 2, off[T] - off[7] + 5]])
    got = U.run_draft(war, ix2, tails, tl, N, k)
    want = D.draft_batch(D.Corpus(hist_tok, hist_off), tails, tl, N, k)
    assert same(got, want)
    with pytest.raises(war.WarError) as e:                            # over capacity: refused, nothing enqueued
        war.war_index_append_async(ix2, d_tok, off)
    assert e.value.code == 3
    ix.destroy(); ix2.destroy()


def test_memo_of_node_expansions_never_changes_an_answer(war):
    """The index caches the expansions of large nodes.  Same answers on an empty and on a filled memo, for different
    k on the same nodes, and after an append (which must drop the entries of the old suffix array)."""
    rng = np.random.default_rng(23)
    vocab = 3                                                          # tiny alphabet: every node near the root is large
    trajs = [rng.integers(0, vocab, size=int(rng.integers(500, 4000))).tolist() for _ in range(10)]
    tok, off = _flat(trajs)
    tails = rng.integers(0, vocab, size=(64, 8)).astype(np.int32)
    tl = rng.integers(0, 9, size=64).astype(np.int32)
    d_tok = torch.from_numpy(tok).to("cuda:0")
    ix = U.build_index(war, tok[:off[7]], off[:8], vocab, max_depth=96, capacity=len(tok) + len(trajs))
    corpus = D.Corpus(tok[:off[7]], off[:8])
    first = {}
    for rep in range(3):
        for k in (1, 3, 2, 8):
            got = U.run_draft(war, ix, tails, tl, 40, k)
            if rep == 0:
                want = D.draft_batch(corpus, tails, tl, 40, k)
                for g, w in zip(got, want):
                    assert np.array_equal(g, w)
                first[k] = got
                assert got[4][:, 0].max() > 1000                        # large nodes were expanded
            else:
                for g, w in zip(got, first[k]):
                    assert np.array_equal(g, w)
    war.war_index_append(ix, d_tok, off[7:])
    want = D.draft_batch(D.Corpus(tok, off), tails, tl, 40, 3)
    got = U.run_draft(war, ix, tails, tl, 40, 3)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    assert not all(np.array_equal(g, w) for g, w in zip(got, first[3]))   # the append did change the answers
    assert war.war_device_status() == 0
    ix.destroy()


def test_export_and_import(war):
    """An imported index answers exactly as the exported one, can be appended to, and bad buffers are refused."""
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(W.scaled(cfg, B=24))
    cut = cfg.n_traj - 9
    ix = U.build_index(war, tok[:off[cut]], off[:cut + 1], cfg.vocab, max_depth=cfg.P + cfg.N)
    buf = war.war_index_export(ix)
    want = U.run_draft(war, ix, tails, tl, cfg.N, cfg.topk)
    ix.destroy()
    ix2 = war.war_index_import(buf, len(tok) + cfg.n_traj)
    info = war.war_index_info(ix2)
    assert info.T == cut and info.M == off[cut] + cut and info.capacity_tokens == len(tok) + cfg.n_traj
    got = U.run_draft(war, ix2, tails, tl, cfg.N, cfg.topk)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    assert np.array_equal(war.war_index_export(ix2), buf)                  # a fixed point
    war.war_index_append(ix2, torch.from_numpy(tok).to("cuda:0"), off[cut:])
    _compare_with_oracle(war, tok, off, cfg.vocab, tails, tl, cfg.N, cfg.topk, ix=ix2)
    ix2.destroy()
    bad = buf.copy(); bad[0] ^= 0xFF                                       # magic
    with pytest.raises(war.WarError):
        war.war_index_import(bad, len(tok) + cfg.n_traj)
    with pytest.raises(war.WarError):
        war.war_index_import(buf[:len(buf) // 2], len(tok) + cfg.n_traj)   # truncated
    with pytest.raises(war.WarError) as e:
        war.war_index_import(buf, 10)                                      # does not fit
    assert e.value.code == 3
    empty = U.build_index(war, np.zeros(0, np.int32), np.zeros(1, np.int64), vocab=10, capacity=64)
    ix3 = war.war_index_import(war.war_index_export(empty), 64)
    assert war.war_index_info(ix3).M == 0
    empty.destroy(); ix3.destroy()


# ----------------------------------------------------------------------------------------------
# drafting from the best-scoring of several suffix lengths
# ----------------------------------------------------------------------------------------------

def _compare_scored(war, ix, corpus, tails, tl, N, k, n_lengths, **kw):
    got = U.run_draft_scored(war, ix, tails, tl, N, k, n_lengths, **kw)
    want = D.draft_scored_batch(corpus, tails, tl, N, k, n_lengths, **kw)
    for name, g, w in zip(["match_len", "used_len", "num_nodes", "ids", "parent", "count"], got, want):
        assert np.array_equal(g, w), f"{name} differs at request(s) {np.flatnonzero((g != w).reshape(len(g), -1).any(axis=1))[:8]}"
    assert war.war_device_status() == 0
    return got


def test_scored_lengths_hand_worked_case(war):
    with open(os.path.join(GOLD, "draft_scored_case1.json")) as f:
        g = json.load(f)
    tok, off = _flat(g["trajectories"])
    ix = U.build_index(war, tok, off, vocab=10)
    tails = np.array([g["tail"]], np.int32)
    tl = np.array([g["tail_len"]], np.int32)
    for nl, used in g["used_len"].items():
        ml, ul, nn, ids, par, cnt = U.run_draft_scored(war, ix, tails, tl, g["N"], g["k"], int(nl))
        want = g["candidates"][str(used)]
        n = len(want["ids"])
        assert (ml[0], ul[0], nn[0]) == (g["match_len"], used, n)
        assert (ids[0, :n].tolist(), par[0, :n].tolist(), cnt[0, :n].tolist()) == (want["ids"], want["parent"], want["count"])
        assert (ids[0, n:] == -1).all() and (par[0, n:] == -1).all() and (cnt[0, n:] == 0).all()
    ix.destroy()


@pytest.mark.parametrize("seed", range(8))
def test_scored_lengths_on_tiny_alphabets(war, seed):
    """Few symbols: every suffix length has many occurrences, scores tie often, every rule of the choice is exercised."""
    rng = np.random.default_rng(300 + seed)
    vocab = int(rng.integers(2, 6))
    trajs = [rng.integers(0, vocab, size=int(rng.integers(0, 200))).tolist() for _ in range(int(rng.integers(1, 9)))]
    tok, off = _flat(trajs)
    P = int(rng.integers(1, 33))
    N = int(rng.integers(1, 65))
    k = int(rng.integers(1, 9))
    B = 24
    tails = rng.integers(0, vocab + 1, size=(B, P)).astype(np.int32)
    tails[0, :] = -1
    tl = rng.integers(-1, P + 1, size=B).astype(np.int32)              # -1: not running
    ix = U.build_index(war, tok, off, vocab + 1)
    corpus = D.Corpus(tok, off)
    for nl in (1, 2, 5, 32):
        _compare_scored(war, ix, corpus, tails, tl, N, k, nl, min_match=int(rng.integers(0, 4)),
                        spec_factor=(int(rng.integers(0, 3)), int(rng.integers(1, 4))),
                        min_prob=(int(rng.integers(0, 2)), int(rng.integers(2, 6))))
    ix.destroy()


def test_scored_lengths_on_the_tiny_workload(war):
    cfg = W.CONFIGS["tiny"]
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(W.scaled(cfg, B=40))
    ix = U.build_index(war, tok, off, cfg.vocab, max_depth=cfg.P + 64)
    corpus = D.Corpus(tok, off)
    one = U.run_draft_scored(war, ix, tails, tl, cfg.N, cfg.topk, 1)
    plain = U.run_draft(war, ix, tails, tl, cfg.N, cfg.topk)
    assert np.array_equal(one[0], plain[0]) and all(np.array_equal(a, b) for a, b in zip(one[2:], plain[1:]))
    picked_shorter = 0
    for nl, N, k in ((4, cfg.N, cfg.topk), (8, 64, 8), (3, 2, 1)):
        got = _compare_scored(war, ix, corpus, tails, tl, N, k, nl)
        picked_shorter += int((got[1] < got[0]).sum())
    assert picked_shorter > 0                                           # the choice is not always the longest match
    # the switch: over the limit nothing is looked up
    got = _compare_scored(war, ix, corpus, tails, tl, cfg.N, cfg.topk, 4, spec_batch_limit=8)
    assert (got[2] == 1).all() and (got[1] == 0).all()
    # no count output
    nc = U.run_draft_scored(war, ix, tails, tl, cfg.N, cfg.topk, 4, with_count=False)
    ref = U.run_draft_scored(war, ix, tails, tl, cfg.N, cfg.topk, 4)
    assert all(np.array_equal(a, b) for a, b in zip(nc[:5], ref[:5]))
    ix.destroy()


def test_searches_that_stop_early_never_change_an_answer(war):
    """The match gives up the suffix lengths that cannot matter (above a length that does not occur, or too far below
    one that does).  Here the lengths differ as much as they can in how long their searches take: one token makes up
    half of the corpus (a bucket many steps deep), the others are rare (shallow buckets), and the tails put the frequent
    token at every position while their longest matches run from nothing to the whole tail."""
    rng = np.random.default_rng(77)
    vocab, F = 400, 7
    trajs = []
    for _ in range(6):
        t = rng.integers(0, vocab, size=3000)
        t[rng.random(3000) < 0.5] = F
        trajs.append(t.tolist())
    tok, off = _flat(trajs)
    P, B = 32, 64
    tails = np.empty((B, P), np.int32)
    for i in range(B):
        at = int(rng.integers(P, len(tok)))
        tails[i] = tok[at - P:at]                                         # occurs as a whole ...
        cut = P if i == 1 else int(rng.integers(0, P + 1))                # ... then only its last `cut` tokens do
        if cut < P:
            tails[i, :P - cut] = rng.integers(0, vocab, size=P - cut)
            tails[i, P - cut - 1] = vocab - 1 - (tails[i, P - cut - 1] % 2)
        if i % 3 == 0:
            tails[i, int(rng.integers(0, P))] = F
    tl = np.full(B, P, np.int32)
    tl[5], tl[6] = 3, 0
    ix = U.build_index(war, tok, off, vocab, max_depth=P + 16)
    corpus = D.Corpus(tok, off)
    got = _compare_with_oracle(war, tok, off, vocab, tails, tl, 16, 4, ix=ix)
    assert got[0].min() == 0 and got[0].max() == P and len(np.unique(got[0])) > 8
    for nl in (2, 5, 32):
        _compare_scored(war, ix, corpus, tails, tl, 16, 4, nl)
    ix.destroy()


def test_scored_lengths_argument_checks(war):
    tok, off = _flat([[1, 2, 3, 1, 2, 3]])
    ix = U.build_index(war, tok, off, vocab=4)
    assert war.war_draft_scored_workspace_bytes(4, 8, 8, 2, 0) == 0
    assert war.war_draft_scored_workspace_bytes(4, 8, 8, 2, 33) == 0
    assert war.war_draft_scored_workspace_bytes(4, 8, 8, 2, 3) >= 4 * (3 * 12 + 3 * 12 * 8)
    tails = np.array([[1, 2, 3]], np.int32)
    with pytest.raises(ValueError):
        U.run_draft_scored(war, ix, tails, np.array([3], np.int32), 8, 2, 0)
    got = U.run_draft_scored(war, ix, np.zeros((0, 3), np.int32), np.zeros(0, np.int32), 8, 2, 2)      # B = 0
    assert got[0].shape == (0,)
    ix.destroy()
