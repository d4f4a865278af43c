"""The synthetic input generators: determinism, shapes, and the bit-exact logical keying of K/V."""
import numpy as np
import torch

from paper_2607_17299_b200 import workloads as W


def test_corpus_is_deterministic_and_has_template_repeats():
    cfg = W.CONFIGS["tiny"]
    a, off = W.make_corpus(cfg)
    b, _ = W.make_corpus(cfg)
    assert (a == b).all() and len(a) == 64 * 2048 and off[-1] == len(a)
    assert a.min() >= 0 and a.max() < cfg.vocab
    freq = np.bincount(a, minlength=cfg.vocab) / len(a)
    assert 0.10 < freq[0] < 0.18                              # Zipf s=1.1 head mass ~0.142


def test_context_length_recipes():
    hi = W.context_lengths(W.CONFIGS["high"])
    assert len(hi) == 256 and hi.max() <= 65536 and hi.min() >= 256 and 9000 < np.median(hi) < 16000
    lt = np.sort(W.context_lengths(W.CONFIGS["longtail"]))
    assert (lt[:60] == 8192).all() and (lt[60:] >= 98304).all() and (lt[60:] <= 131072).all()
    assert abs(W.trajectory_lengths(W.CONFIGS["longtail"]).sum() / 64e6 - 1) < 0.1


def test_kv_values_depend_on_logical_position_only():
    cfg = W.scaled(W.CONFIGS["tiny"], B=3)
    ctx = np.array([40, 300, 17])
    a = W.make_attention_inputs(cfg, ctx)
    table = W.normal_table()
    for i in range(3):
        pos = torch.arange(int(ctx[i]) - 1 + cfg.N)
        want = W.logical_kv(cfg, i, pos, 1, table)
        pages = torch.from_numpy(a.page_table[i].numpy().astype(np.int64))[pos // cfg.page_size]
        got = a.v_pool[pages, :, pos % cfg.page_size, :]
        assert torch.equal(got, want)
    assert abs(a.k_pool.float().std().item() - 1.0) < 0.02
    assert a.q.shape == (3, cfg.N, cfg.Hq, cfg.D) and a.prefix_len.tolist() == [39, 299, 16]


def test_targets_follow_first_child_at_zero_mismatch():
    cfg = W.scaled(W.CONFIGS["tiny"], B=1, mismatch=0.0)
    ids = np.array([[3, 4, 5, 1, 8, 1] + [-1] * 10], np.int32)
    parent = np.array([[-1, 0, 0, 1, 1, 2] + [-1] * 10], np.int32)
    t = W.make_targets(cfg, ids, parent, np.array([6]))
    assert t[0, 0] == 4 and t[0, 1] == 1 and t[0, 2] == 1
