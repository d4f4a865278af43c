"""The allocation-free verify-attention entry point (collected last on purpose).

Some users of the library cannot allocate device memory where they call it (a frozen memory pool, a plugin that
only sees its input and output buffers), so war_verify_attn_noalloc keeps its scratch in a fixed array inside the
library.  It must give what war_verify_attn gives, call after call, although the array still holds the previous
call's contents."""
import numpy as np
import pytest
import torch

from paper_2607_17299_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def war():
    from paper_2607_17299_b200 import binding
    return binding


def _trees(rng, B, N):
    parent = np.full((B, N), -1, np.int32); nn = np.zeros(B, np.int32)
    for i in range(B):
        nn[i] = int(rng.integers(1, N + 1))
        for j in range(1, nn[i]):
            parent[i, j] = int(rng.integers(0, j))
    return nn, parent


def _both(war, cfg, ctx, seed):
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(seed)
    a = W.make_attention_inputs(cfg, ctx, device=dev)
    nn, parent = _trees(rng, cfg.B, cfg.N)
    d_nn, d_par = torch.from_numpy(nn).to(dev), torch.from_numpy(parent).to(dev)
    scale = 1.0 / float(np.sqrt(cfg.D))
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, scale, 0)
    assert 0 < war.war_verify_attn_workspace_bytes(params) <= war.NOALLOC_MAX_BYTES
    ws = war.new_workspace(params, dev)
    ref_out = torch.full(a.q.shape, 3.0, dtype=torch.bfloat16, device=dev)
    ref_lse = torch.full(a.q.shape[:3], 3.0, dtype=torch.float32, device=dev)
    war.war_verify_attn(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, d_nn, d_par, params, ws, ref_out, ref_lse)
    out = torch.full(a.q.shape, 3.0, dtype=torch.bfloat16, device=dev)
    lse = torch.full(a.q.shape[:3], 3.0, dtype=torch.float32, device=dev)
    war.war_verify_attn_noalloc(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, d_nn, d_par, params, out, lse)
    torch.cuda.synchronize()
    # the two entry points run the same kernels on the same plan: the same bits, not merely close ones
    assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)
    assert (ref_out.float() != 3.0).any()
    assert war.war_device_status() == 0
    return a, nn, parent, scale, out, lse


def test_matches_the_workspace_entry_point_on_two_calls_in_a_row(war):
    # two different shapes back to back: the second call finds the first call's work list and partials in the array
    cfg1 = W.scaled(W.CONFIGS["tiny"], B=6, N=16)
    _both(war, cfg1, np.array([4096, 3000, 17, 1025, 2500, 129]), seed=1)
    cfg2 = W.scaled(W.CONFIGS["tiny"], B=3, N=8, page_size=32)
    _both(war, cfg2, np.array([700, 5000, 64]), seed=2)
    _both(war, cfg1, np.array([100, 200, 300, 400, 500, 4000]), seed=3)


def test_matches_the_cpu_checker(war):
    """The allocation-free entry point against the fp64 checker itself (not only against the other entry point)."""
    from oracle import attention_oracle as A
    from tests import gpu_util as U
    cfg = W.scaled(W.CONFIGS["tiny"], B=4, N=16)
    a, nn, parent, scale, out, lse = _both(war, cfg, np.array([3000, 129, 4096, 640]), seed=4)
    want = A.verify_attention(a.q, a.k_pool, a.v_pool, a.page_table.cpu().numpy(), a.prefix_len.cpu().numpy(), nn, parent, scale)
    got, got_lse = out.float().cpu().numpy(), lse.cpu().numpy()
    for i in range(cfg.B):
        U.assert_attention_close(got[i], got_lse[i], want[i][0], want[i][1], int(nn[i]))


def test_refuses_shapes_beyond_the_fixed_scratch(war):
    dev = torch.device("cuda:0")
    cfg = W.scaled(W.CONFIGS["tiny"], B=64, N=64, Hq=64)             # 512 rows per kv head: scratch far above the limit
    a = W.make_attention_inputs(cfg, np.full(cfg.B, 40), device=dev)
    params = war.attn_params(a.q, a.k_pool, a.v_pool, a.page_table, 0.1, 0)
    assert war.war_verify_attn_workspace_bytes(params) > war.NOALLOC_MAX_BYTES
    nn = torch.ones(cfg.B, dtype=torch.int32, device=dev)
    par = torch.full((cfg.B, cfg.N), -1, dtype=torch.int32, device=dev)
    out = torch.zeros_like(a.q)
    with pytest.raises(war.WarError) as e:
        war.war_verify_attn_noalloc(a.q, a.k_pool, a.v_pool, a.page_table, a.prefix_len, nn, par, params, out, None)
    assert e.value.code == 3
