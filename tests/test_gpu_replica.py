"""GPU tests of the multi-rank plumbing: the end-of-step trajectory exchange followed by the replicated append
(paper Section 3.3, cross-worker synchronisation of the suffix cache) and the tensor-parallel split of the
verification by kv heads (the paper's rollout workers run with tensor parallelism 4).

Both run through NCCL and the library, on as many GPUs as there are: always as a process group of one rank, and as two
ranks (child processes, one GPU each) when two GPUs are visible.  No kernel ever reads another GPU's memory: the
exchange is an NCCL all-gather into each rank's own buffer."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import attention_oracle as A
from oracle import draft_oracle as D
from paper_2607_17299_b200 import replica
from paper_2607_17299_b200 import workloads as W
from tests import gpu_util as U

pytestmark = pytest.mark.gpu


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _setup(cfg):
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    return tok, off, tails, tl


def _rank_share(off, base, rank, world):
    """Trajectories [base, T) dealt to the ranks in contiguous, unequal shares (rank 0 gets the larger one)."""
    T = len(off) - 1
    cut = [base, base + (2 * (T - base)) // 3, T] if world == 2 else [base, T]
    return cut[rank], cut[rank + 1]


def _exchange_and_check(rank, world, dev):
    """Every rank: an index over the first `base` trajectories, the rest arrives through the exchange; afterwards the
    library's drafts equal the checker's on the whole history, on every rank."""
    from paper_2607_17299_b200 import binding as war
    cfg = W.scaled(W.CONFIGS["tiny"], B=8, n_traj=24)
    tok, off, tails, tl = _setup(cfg)
    base = 12
    N, k = cfg.N, cfg.topk
    ix = U.build_index(war, tok[:off[base]], off[:base + 1], cfg.vocab, max_depth=cfg.P + N, capacity=len(tok) + cfg.n_traj)
    t0, t1 = _rank_share(off, base, rank, world)
    mine_tok = torch.from_numpy(tok[off[t0]:off[t1]]).to(dev)               # the rank's finished trajectories are on its GPU
    got_tok, got_off = replica.append_step_trajectories(ix, mine_tok, off[t0:t1 + 1] - off[t0], dev)
    assert got_tok.is_cuda and got_tok.dtype == torch.int32
    assert np.array_equal(got_tok.cpu().numpy(), tok[off[base]:]) and np.array_equal(got_off, off[base:] - off[base])
    assert war.war_index_info(ix).T == cfg.n_traj
    got = U.run_draft(war, ix, tails, tl, N, k)
    want = D.draft_batch(D.Corpus(tok, off), tails, tl, N, k)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    # a sliding window over the trajectory stream: the same eviction on every rank, then the same append
    extra = tok[off[2]:off[6]]
    e0, e1 = (0, 4) if world == 1 else ((0, 3), (3, 4))[rank]
    o = off[2:7] - off[2]
    replica.append_step_trajectories(ix, torch.from_numpy(extra[o[e0]:o[e1]]).to(dev), o[e0:e1 + 1] - o[e0], dev, window=20)
    assert war.war_index_info(ix).T == 20
    hist_tok = np.concatenate([tok[off[8]:], extra])
    hist_off = np.concatenate([off[8:] - off[8], (off[-1] - off[8]) + o[1:]])
    got = U.run_draft(war, ix, tails, tl, N, k)
    want = D.draft_batch(D.Corpus(hist_tok, hist_off), tails, tl, N, k)
    for g, w in zip(got, want):
        assert np.array_equal(g, w)
    assert war.war_device_status() == 0
    ix.destroy()


def _head_shard_check(rank, world):
    """A tensor-parallel rank verifies its own kv heads on its own slice of q and of the pools; checked against the
    fp64 checker restricted to those heads."""
    from paper_2607_17299_b200 import binding as war
    cfg = W.scaled(W.CONFIGS["tiny"], B=3, N=16)
    ctx = np.array([2100, 400, 900])
    rng = np.random.default_rng(5)
    nn = rng.integers(1, cfg.N + 1, cfg.B).astype(np.int32)
    parent = np.full((cfg.B, cfg.N), -1, np.int32)
    for i in range(cfg.B):
        for j in range(1, nn[i]):
            parent[i, j] = int(rng.integers(0, j))
    a = W.make_attention_inputs(cfg, ctx, device=U.dev())                  # every rank generates the same full tensors ...
    G = cfg.Hq // cfg.Hkv
    hs = replica.kv_head_shard(cfg.Hkv, rank, world)                       # ... and keeps its heads
    mine = W.AttnInputs(q=a.q[:, :, hs.start * G:hs.stop * G, :].contiguous(), k_pool=a.k_pool[:, hs].contiguous(),
                        v_pool=a.v_pool[:, hs].contiguous(), page_table=a.page_table, prefix_len=a.prefix_len,
                        num_pages=a.num_pages, max_pages=a.max_pages)
    got, got_lse, _ = U.run_attn(war, mine, nn, parent, 0.09, 0)
    want = A.verify_attention(mine.q, mine.k_pool, mine.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(), nn,
                              parent, 0.09)
    for i in range(cfg.B):
        U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], int(nn[i]))
    assert war.war_device_status() == 0


def _worker(rank, world, port):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ.setdefault("NCCL_NVLS_ENABLE", "0")
    torch.cuda.set_device(rank)
    dev = torch.device("cuda", rank)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    try:
        _exchange_and_check(rank, world, dev)
        if rank == 0 or torch.cuda.device_count() >= world:
            _head_shard_check(rank, world)
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_exchange_and_append_in_a_process_group_of_one():
    port = _free_port()
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dev = U.dev()
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    try:
        _exchange_and_check(0, 1, dev)
    finally:
        dist.destroy_process_group()


def test_head_shards_against_the_checker_one_rank_after_the_other():
    for rank in range(2):
        _head_shard_check(rank, 2)


@pytest.mark.timeout(600)
def test_exchange_and_head_shards_on_two_gpus():
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs")
    mp.spawn(_worker, args=(2, _free_port()), nprocs=2, join=True)
