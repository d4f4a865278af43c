"""World-size-2 CPU test (gloo) of the replica plumbing: end-of-step trajectory exchange and request sharding."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import draft_oracle as D
from paper_2607_17299_b200 import replica
from paper_2607_17299_b200 import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_trajectories(rank):
    rng = np.random.default_rng(100 + rank)
    n = 3 + rank                                              # ranks contribute different numbers of trajectories
    trajs = [rng.integers(0, 6, size=int(rng.integers(0, 50))).astype(np.int32) for _ in range(n)]
    off = np.zeros(n + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(t) for t in trajs])
    tok = np.concatenate(trajs) if n else np.zeros(0, np.int32)
    return tok, off


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        tok, off = _rank_trajectories(rank)
        all_tok, all_off = replica.gather_trajectories(tok, off, "cpu")
        all_tok = all_tok.numpy()
        # drafts from the merged history, for a fixed set of probes
        corpus = D.Corpus(all_tok, all_off)
        rng = np.random.default_rng(7)
        tails = rng.integers(0, 6, size=(16, 6)).astype(np.int32)
        res = D.draft_batch(corpus, tails, np.full(16, 6, np.int32), 8, 3)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), tok=all_tok, off=all_off, ids=res[2], parent=res[3], count=res[4],
                 ml=res[0])
        sl = replica.shard_requests(11, rank, world)
        np.save(os.path.join(out_dir, f"shard{rank}.npy"), np.arange(11)[sl])
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_trajectory_exchange_and_sharding(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    r0 = np.load(tmp_path / "rank0.npz")
    r1 = np.load(tmp_path / "rank1.npz")
    for k in r0.files:                                        # every rank ends with the same history and the same drafts
        assert (r0[k] == r1[k]).all(), k
    t0, o0 = _rank_trajectories(0)
    t1, o1 = _rank_trajectories(1)
    assert (r0["tok"] == np.concatenate([t0, t1])).all()      # rank order
    assert (r0["off"] == np.concatenate([o0, o1[1:] + o0[-1]])).all()
    # the same trajectories arriving in the other order give the same drafts (order independence of the cache)
    corpus = D.Corpus(np.concatenate([t1, t0]), np.concatenate([o1, o0[1:] + o1[-1]]))
    rng = np.random.default_rng(7)
    tails = rng.integers(0, 6, size=(16, 6)).astype(np.int32)
    res = D.draft_batch(corpus, tails, np.full(16, 6, np.int32), 8, 3)
    assert (res[2] == r0["ids"]).all() and (res[3] == r0["parent"]).all() and (res[4] == r0["count"]).all()
    shards = [np.load(tmp_path / f"shard{r}.npy") for r in range(world)]
    assert np.concatenate(shards).tolist() == list(range(11)) and abs(len(shards[0]) - len(shards[1])) <= 1


def test_one_rank_alone_needs_no_process_group():
    tok, off = _rank_trajectories(1)
    got_tok, got_off = replica.gather_trajectories(tok, off, "cpu")
    assert (got_tok.numpy() == tok).all() and (got_off == off).all()
    with pytest.raises(ValueError):
        replica.gather_trajectories(tok[:-1], off, "cpu")


def test_kv_head_shards_cover_the_heads():
    assert [replica.kv_head_shard(8, r, 4) for r in range(4)] == [slice(0, 2), slice(2, 4), slice(4, 6), slice(6, 8)]
    with pytest.raises(ValueError):
        replica.kv_head_shard(8, 0, 3)


def test_window_eviction_policy():
    """Host logic of the sliding window: stored + incoming never exceeds the window, never evicts more than stored."""
    assert replica.window_eviction(10, 3, 0) == 0                  # no window
    assert replica.window_eviction(10, 3, 20) == 0
    assert replica.window_eviction(10, 3, 13) == 0
    assert replica.window_eviction(10, 3, 12) == 1
    assert replica.window_eviction(10, 3, 3) == 10
    assert replica.window_eviction(2, 9, 4) == 2                   # more incoming than the window holds
    for stored in range(0, 12):
        for incoming in range(0, 12):
            for window in range(1, 12):
                e = replica.window_eviction(stored, incoming, window)
                assert 0 <= e <= stored and (stored - e + min(incoming, window) <= window or e == stored)
