"""Pins for the fp64 tree-masked attention checker: a hand-worked case, reductions to a library routine
(torch scaled_dot_product_attention in fp64), and invariants of the definition."""
import json
import os

import numpy as np
import pytest
import torch

from oracle import attention_oracle as A

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _random_case(seed, n, prefix_len, Hq=4, Hkv=2, D=8, pg=4, parent=None, scramble=True):
    g = torch.Generator().manual_seed(seed)
    L = prefix_len + n
    n_pages = (L + pg - 1) // pg
    pool_pages = n_pages + 3
    k_pool = torch.randn((pool_pages, Hkv, pg, D), generator=g).to(torch.bfloat16)
    v_pool = torch.randn((pool_pages, Hkv, pg, D), generator=g).to(torch.bfloat16)
    q = torch.randn((1, n, Hq, D), generator=g).to(torch.bfloat16)
    perm = torch.randperm(pool_pages, generator=g).numpy() if scramble else np.arange(pool_pages)
    page_table = perm[None, :n_pages].astype(np.int32)
    if parent is None:
        rs = np.random.default_rng(seed)
        parent = np.array([-1] + [int(rs.integers(0, j)) for j in range(1, n)], dtype=np.int32)
    return q, k_pool, v_pool, page_table, np.array([prefix_len], np.int32), np.array([n], np.int32), parent[None, :]


def _logical(k_pool, v_pool, page_table, L):
    return A.gather_request_kv(k_pool, v_pool, page_table[0], L)


def test_hand_worked_uniform_softmax():
    with open(os.path.join(GOLD, "attention_case3.json")) as f:
        g = json.load(f)
    V = np.array(g["prefix_v"] + g["slot_v"], dtype=np.float64)[:, None, :]
    K = np.random.default_rng(0).normal(size=V.shape)        # irrelevant: q = 0
    q = np.zeros((3, 1, g["D"]))
    out, lse = A.verify_attention_request(q, K, V, g["prefix_len"], np.array(g["parent"]), 3, g["scale"])
    np.testing.assert_allclose(out[:, 0, :], np.array(g["out"]), rtol=0, atol=1e-15)
    np.testing.assert_allclose(np.exp(lse[:, 0]), np.array(g["lse_exp"], dtype=np.float64), rtol=1e-14)


@pytest.mark.parametrize("seed,n,prefix", [(0, 1, 37), (1, 1, 0), (2, 5, 19), (3, 7, 0), (4, 6, 64)])
def test_chain_tree_is_causal_attention(seed, n, prefix):
    """parent[j] = j-1 makes slot j see the prefix and slots 0..j: plain causal attention of n new tokens
    (n = 1: ordinary decode attention).  Cross-checked against the library routine, which also pins the
    query-head -> kv-head grouping (h // G, i.e. repeat_interleave of the kv heads)."""
    Hq, Hkv, D = 6, 2, 8
    chain = np.arange(-1, n - 1, dtype=np.int32)
    q, kp, vp, pt, pl, nn, par = _random_case(seed, n, prefix, Hq, Hkv, D, parent=chain)
    scale = 0.37
    res = A.verify_attention(q, kp, vp, pt, pl, nn, par, scale)[0]
    K, V = _logical(kp, vp, pt, prefix + n)
    Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)     # [Hq, L, D]
    Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
    Qt = q[0].to(torch.float64).permute(1, 0, 2)                                       # [Hq, n, D]
    L = prefix + n
    mask = torch.zeros((n, L), dtype=torch.bool)
    for j in range(n):
        mask[j, :prefix + j + 1] = True
    ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, attn_mask=mask, scale=scale)
    np.testing.assert_allclose(res[0], ref.permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-13)
    z = scale * torch.einsum("hnd,hld->hnl", Qt, Kt).masked_fill(~mask, float("-inf"))
    np.testing.assert_allclose(res[1], torch.logsumexp(z, dim=-1).T.numpy(), rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("seed", range(4))
def test_tree_equals_per_slot_decode_over_its_root_path(seed):
    """Slot j of any tree equals single-token decode attention over [prefix, ancestors..., j] gathered in a
    dense buffer: the tree mask is nothing more than that selection."""
    n, prefix, Hq, Hkv, D = 7, 21, 4, 2, 8
    q, kp, vp, pt, pl, nn, par = _random_case(seed, n, prefix, Hq, Hkv, D)
    scale = 1 / np.sqrt(D)
    out, lse = A.verify_attention(q, kp, vp, pt, pl, nn, par, scale)[0]
    K, V = _logical(kp, vp, pt, prefix + n)
    for j in range(n):
        cols = list(range(prefix)) + [prefix + a for a in sorted(A.ancestors_or_self(par[0], j))]
        Kt = torch.from_numpy(K[cols]).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
        Vt = torch.from_numpy(V[cols]).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)
        Qt = q[0, j].to(torch.float64)[:, None, :]
        ref = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, scale=scale)
        np.testing.assert_allclose(out[j], ref[:, 0, :].numpy(), rtol=1e-12, atol=1e-13)


def test_constant_v_and_weights_sum_to_one():
    q, kp, vp, pt, pl, nn, par = _random_case(7, 6, 33)
    vp = torch.full_like(vp, 1.5)
    out, _ = A.verify_attention(q, kp, vp, pt, pl, nn, par, 0.5)[0]
    np.testing.assert_allclose(out, 1.5, rtol=1e-14)


def test_non_ancestors_do_not_matter_and_siblings_are_hidden():
    parent = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    q, kp, vp, pt, pl, nn, par = _random_case(9, 5, 10, parent=parent, scramble=False, pg=4)
    base, _ = A.verify_attention(q, kp, vp, pt, pl, nn, par, 0.3)[0]
    # overwrite K/V of slot 2 (logical position 12 -> page 3, row 0): slots 0, 1, 3 must not change, 2 and 4 must
    kp2, vp2 = kp.clone(), vp.clone()
    kp2[3, :, 0, :] += 1.0
    vp2[3, :, 0, :] -= 2.0
    out2, _ = A.verify_attention(q, kp2, vp2, pt, pl, nn, par, 0.3)[0]
    for j in (0, 1, 3):
        assert (out2[j] == base[j]).all()
    for j in (2, 4):
        assert np.abs(out2[j] - base[j]).max() > 1e-3


def test_page_permutation_and_group_symmetry():
    q, kp, vp, pt, pl, nn, par = _random_case(13, 5, 27, Hq=4, Hkv=2)
    q[:, :, 1, :] = q[:, :, 0, :]                           # heads 0 and 1 share kv head 0
    out, lse = A.verify_attention(q, kp, vp, pt, pl, nn, par, 0.4)[0]
    assert (out[:, 0] == out[:, 1]).all() and (lse[:, 0] == lse[:, 1]).all()
    assert np.abs(out[:, 2] - out[:, 0]).max() > 1e-3        # head 2 reads kv head 1
    perm = torch.randperm(kp.shape[0], generator=torch.Generator().manual_seed(3))
    inv = torch.empty_like(perm); inv[perm] = torch.arange(len(perm))
    kp2, vp2 = kp[perm], vp[perm]                            # physical page x now sits at inv[x]
    pt2 = inv.numpy()[pt].astype(np.int32)
    out2, lse2 = A.verify_attention(q, kp2, vp2, pt2, pl, nn, par, 0.4)[0]
    assert (out2 == out).all() and (lse2 == lse).all()


def test_needle_key_dominates():
    """A key aligned with the query with a large logit takes essentially all the weight: output = its V."""
    n, prefix, D = 1, 50, 8
    q, kp, vp, pt, pl, nn, par = _random_case(17, n, prefix, Hq=2, Hkv=1, D=D, scramble=False, pg=4)
    q[:] = 0
    q[0, 0, :, 0] = 8.0
    kp[:] = 0
    kp[5, 0, 2, 0] = 8.0                                     # logical position 22
    out, lse = A.verify_attention(q, kp, vp, pt, pl, nn, par, 1.0)[0]
    want = vp[5, 0, 2, :].to(torch.float64).numpy()
    np.testing.assert_allclose(out[0, 0], want, atol=1e-20 + 51 * np.exp(-64.0) * 8)
    np.testing.assert_allclose(lse[0, 0], 64.0, atol=1e-12)
