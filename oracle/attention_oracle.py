"""Tree-masked GQA verification attention in fp64 (test infrastructure).

The verifier scores all draft tokens of a request in one forward pass (paper, Section 3.3: the target model
checks the predicted tokens together, in one pass; Sections 2.3 and 5.3 name the auxiliary attention / tree mask
this needs).  The attention of that pass, for request i, slot j, query head h
(kv head g = h // G):

    visible(j) = { all prefix positions 0 .. prefix_len-1 }  U  { prefix_len + a : a == j or a is an ancestor of j }
    z_c   = scale * <q[i, j, h, :], K[c, g, :]>            for c in visible(j)
    out   = sum_c softmax(z)_c * V[c, g, :]                 lse = log sum_c exp(z_c)      (natural log)

computed in float64 from the bf16 input values.  Slot a's K/V sit at logical position prefix_len + a;
logical position p lives in physical page page_table[i, p // page_size], row p % page_size.
"""
from __future__ import annotations

import numpy as np
import torch


def ancestors_or_self(parent: np.ndarray, j: int):
    out = []
    a = int(j)
    while a >= 0:
        out.append(a)
        a = int(parent[a])
    return out


def gather_request_kv(k_pool: torch.Tensor, v_pool: torch.Tensor, page_row: np.ndarray, n_tokens: int):
    """float64 [n_tokens, Hkv, D] K and V of one request, in logical order."""
    pg = k_pool.shape[2]
    n_pages = (n_tokens + pg - 1) // pg
    pages = torch.as_tensor(np.asarray(page_row[:n_pages], dtype=np.int64), device=k_pool.device)
    def one(pool):
        x = pool[pages]                                   # [n_pages, Hkv, pg, D]
        x = x.permute(0, 2, 1, 3).reshape(n_pages * pg, pool.shape[1], pool.shape[3])[:n_tokens]
        return x.to("cpu").to(torch.float64).numpy()
    return one(k_pool), one(v_pool)


def verify_attention_request(q: np.ndarray, K: np.ndarray, V: np.ndarray, prefix_len: int, parent: np.ndarray,
                             n: int, scale: float):
    """q float64 [N, Hq, D]; K, V float64 [>= prefix_len + n, Hkv, D].  Returns out [n, Hq, D], lse [n, Hq]."""
    Hq, D = q.shape[1], q.shape[2]
    Hkv = K.shape[1]
    G = Hq // Hkv
    L = prefix_len + n
    # visible[j, c]: every prefix column, and tree column prefix_len + a iff a is j or an ancestor of j
    visible = np.zeros((n, L), dtype=bool)
    visible[:, :prefix_len] = True
    for j in range(n):
        for a in ancestors_or_self(parent, j):
            visible[j, prefix_len + a] = True
    out = np.zeros((n, Hq, D), dtype=np.float64)
    lse = np.zeros((n, Hq), dtype=np.float64)
    for h in range(Hq):
        g = h // G
        z = scale * (q[:n, h, :] @ K[:L, g, :].T)          # [n, L] logits against every stored position
        z = np.where(visible, z, -np.inf)
        m = z.max(axis=1, keepdims=True)
        w = np.exp(z - m)
        den = w.sum(axis=1, keepdims=True)
        out[:, h, :] = (w @ V[:L, g, :]) / den
        lse[:, h] = (m + np.log(den))[:, 0]
    return out, lse


def verify_attention(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: np.ndarray,
                     prefix_len: np.ndarray, num_nodes: np.ndarray, parent: np.ndarray, scale: float,
                     requests=None):
    """Batched wrapper.  Returns {i: (out float64 [n_i, Hq, D], lse float64 [n_i, Hq])} for the chosen requests."""
    res = {}
    B = q.shape[0]
    for i in (range(B) if requests is None else requests):
        n = int(num_nodes[i])
        if n == 0:
            res[i] = (np.zeros((0,) + tuple(q.shape[2:])), np.zeros((0, q.shape[2])))
            continue
        K, V = gather_request_kv(k_pool, v_pool, np.asarray(page_table[i]), int(prefix_len[i]) + n)
        qi = q[i].to("cpu").to(torch.float64).numpy()
        res[i] = verify_attention_request(qi, K, V, int(prefix_len[i]), np.asarray(parent[i]), n, scale)
    return res
