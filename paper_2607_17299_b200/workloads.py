"""Seeded synthetic workloads for the speculate-and-verify step.

This module only *produces inputs*: token corpora, request tails, context lengths, paged
bf16 K/V pools, queries and target ids.  It contains none of the method's arithmetic (no
matching, no tree building, no attention, no acceptance), so that both the CUDA path and
the independent CPU checker can be fed the very same bits.

The paper evaluates on a private software-engineering agent dataset (Section 5, setup) with
contexts of 10K-100K tokens (Section 3) in which recurring code snippets provide the suffix
matches (Section 5.3).  None of that data exists here; the five configurations below are
seeded stand-ins with the same scales: Zipf-distributed tokens with a share of spans copied
from a fixed pool of templates (the "recurring snippets"), long and long-tailed contexts,
GQA head shapes of the served model family.

Everything is a pure function of (configuration, seed).  The corpus / request generators
use numpy's PCG64; the bf16 tensors use a counter hash written with exact integer torch ops
so that the same call yields identical bits on CPU and on a CUDA device.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

VOCAB = 32000
ZIPF_S = 1.1
TEMPLATE_POOL = 256
PATTERN_LEN = 32          # P: how many trailing context tokens are matched
TOPK = 4                  # k: branching of the draft tree
HEAD_DIM = 128


@dataclass(frozen=True)
class WorkloadConfig:
    name: str
    index: int                    # position in the benchmark's configuration list (seeds derive from it)
    n_traj: int
    traj_len: int                 # fixed length, or the median when traj_sigma > 0
    traj_sigma: float             # lognormal sigma of trajectory lengths (0 = fixed)
    traj_clip: Tuple[int, int]
    B: int                        # live requests
    ctx: str                      # "fixed" | "uniform" | "lognormal" | "longtail"
    ctx_a: int
    ctx_b: int
    ctx_sigma: float
    N: int                        # tree slots per request, root slot included
    Hq: int
    Hkv: int
    page_size: int
    p_tmpl: float
    tmpl_lo: int
    tmpl_hi: int
    mismatch: float               # per-node probability that the target disagrees with the draft
    P: int = PATTERN_LEN
    topk: int = TOPK
    D: int = HEAD_DIM
    vocab: int = VOCAB


CONFIGS: Dict[str, WorkloadConfig] = {
    "tiny": WorkloadConfig("tiny", 0, 64, 2048, 0.0, (2048, 2048), 8, "fixed", 4096, 4096, 0.0,
                           16, 32, 8, 16, 0.2, 8, 64, 0.30),
    "low": WorkloadConfig("low", 1, 512, 16384, 0.0, (16384, 16384), 32, "uniform", 16384, 32768, 0.0,
                          32, 32, 8, 16, 0.2, 8, 64, 0.25),
    "high": WorkloadConfig("high", 2, 2048, 16384, 0.0, (16384, 16384), 256, "lognormal", 12288, 65536, 0.6,
                           8, 32, 8, 16, 0.2, 8, 64, 0.40),
    "longtail": WorkloadConfig("longtail", 3, 4096, 8192, 1.18, (256, 131072), 64, "longtail", 8192, 131072, 0.0,
                               24, 32, 8, 32, 0.2, 8, 64, 0.25),
    "wide": WorkloadConfig("wide", 4, 1024, 32768, 0.0, (32768, 32768), 128, "uniform", 24576, 49152, 0.0,
                           64, 64, 8, 16, 0.5, 128, 1024, 0.15),
}


def scaled(cfg: WorkloadConfig, **kw) -> WorkloadConfig:
    """A copy of a configuration with some fields replaced (used by tests for reduced sizes)."""
    return replace(cfg, **kw)


def seed_streams(cfg: WorkloadConfig) -> List[np.random.SeedSequence]:
    """Six independent streams: templates, corpus, requests, kv, page table, targets."""
    return np.random.SeedSequence(1000 + cfg.index).spawn(6)


# ----------------------------------------------------------------------------------------------
# tokens
# ----------------------------------------------------------------------------------------------

def zipf_cdf(vocab: int = VOCAB, s: float = ZIPF_S) -> np.ndarray:
    r = np.arange(1, vocab + 1, dtype=np.float64)
    p = r ** (-s)
    cdf = np.cumsum(p / p.sum())
    cdf[-1] = 1.0
    return cdf


def zipf_tokens(rng: np.random.Generator, n: int, cdf: np.ndarray) -> np.ndarray:
    """n token ids; id = Zipf rank - 1, drawn by inverse-CDF lookup."""
    u = rng.random(n)
    return np.minimum(np.searchsorted(cdf, u, side="left"), len(cdf) - 1).astype(np.int32)


def make_templates(cfg: WorkloadConfig, cdf: np.ndarray) -> List[np.ndarray]:
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[0]))
    lens = rng.integers(cfg.tmpl_lo, cfg.tmpl_hi + 1, size=TEMPLATE_POOL)
    return [zipf_tokens(rng, int(l), cdf) for l in lens]


def _span_sequence(rng: np.random.Generator, length: int, cfg: WorkloadConfig, templates: List[np.ndarray],
                   tmpl_flat: np.ndarray, tmpl_off: np.ndarray, cdf: np.ndarray) -> np.ndarray:
    """Spans are appended until `length` tokens exist, then the sequence is truncated.  A span is a
    whole template (probability p_tmpl) or a fresh Zipf span whose length is uniform in the
    templates' length range."""
    n_spans = length // cfg.tmpl_lo + 2
    is_t = rng.random(n_spans) < cfg.p_tmpl
    tid = rng.integers(0, TEMPLATE_POOL, size=n_spans)
    fresh_len = rng.integers(cfg.tmpl_lo, cfg.tmpl_hi + 1, size=n_spans)
    tlen = (tmpl_off[1:] - tmpl_off[:-1])[tid]
    lens = np.where(is_t, tlen, fresh_len).astype(np.int64)
    ends = np.cumsum(lens)
    used = int(np.searchsorted(ends, length, side="left")) + 1
    is_t, tid, lens, ends = is_t[:used], tid[:used], lens[:used], ends[:used]
    total = int(ends[-1])
    starts = ends - lens
    span_of = np.repeat(np.arange(used), lens)
    within = np.arange(total, dtype=np.int64) - starts[span_of]
    from_t = is_t[span_of]
    out = np.empty(total, dtype=np.int32)
    out[from_t] = tmpl_flat[tmpl_off[tid[span_of[from_t]]] + within[from_t]]
    n_fresh = int((~from_t).sum())
    out[~from_t] = zipf_tokens(rng, n_fresh, cdf)
    return out[:length]


def _flatten(templates: List[np.ndarray]) -> Tuple[np.ndarray, np.ndarray]:
    off = np.zeros(len(templates) + 1, dtype=np.int64)
    off[1:] = np.cumsum([len(t) for t in templates])
    return np.concatenate(templates).astype(np.int32), off


def trajectory_lengths(cfg: WorkloadConfig) -> np.ndarray:
    if cfg.traj_sigma <= 0:
        return np.full(cfg.n_traj, cfg.traj_len, dtype=np.int64)
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[1].spawn(1)[0]))
    l = np.exp(rng.normal(math.log(cfg.traj_len), cfg.traj_sigma, size=cfg.n_traj))
    return np.clip(np.rint(l), cfg.traj_clip[0], cfg.traj_clip[1]).astype(np.int64)


def make_corpus(cfg: WorkloadConfig) -> Tuple[np.ndarray, np.ndarray]:
    """Returns (tokens int32[sum len], offsets int64[T+1]): trajectory t is tokens[offsets[t]:offsets[t+1]]."""
    cdf = zipf_cdf(cfg.vocab)
    templates = make_templates(cfg, cdf)
    tmpl_flat, tmpl_off = _flatten(templates)
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[1]))
    lens = trajectory_lengths(cfg)
    offsets = np.zeros(cfg.n_traj + 1, dtype=np.int64)
    offsets[1:] = np.cumsum(lens)
    tokens = np.empty(int(offsets[-1]), dtype=np.int32)
    for t in range(cfg.n_traj):
        tokens[offsets[t]:offsets[t + 1]] = _span_sequence(rng, int(lens[t]), cfg, templates, tmpl_flat, tmpl_off, cdf)
    return tokens, offsets


def context_lengths(cfg: WorkloadConfig) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[2].spawn(1)[0]))
    if cfg.ctx == "fixed":
        return np.full(cfg.B, cfg.ctx_a, dtype=np.int64)
    if cfg.ctx == "uniform":
        return rng.integers(cfg.ctx_a, cfg.ctx_b + 1, size=cfg.B).astype(np.int64)
    if cfg.ctx == "lognormal":
        l = np.exp(rng.normal(math.log(cfg.ctx_a), cfg.ctx_sigma, size=cfg.B))
        return np.clip(np.rint(l), 256, cfg.ctx_b).astype(np.int64)
    if cfg.ctx == "longtail":
        n_long = max(1, cfg.B // 16)
        out = np.full(cfg.B, cfg.ctx_a, dtype=np.int64)
        where = rng.choice(cfg.B, size=n_long, replace=False)
        out[where] = rng.integers((cfg.ctx_b * 3) // 4, cfg.ctx_b + 1, size=n_long)
        return out
    raise ValueError(cfg.ctx)


def make_request_tails(cfg: WorkloadConfig, ctx_len: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """The last P tokens of each live request's context, right-aligned in an int32[B, P] array, and how many
    of them are real (tail_len = min(P, context length)).  Contexts come from the corpus generator and the
    same template pool, on their own seed stream; only their final tokens matter to the step, so only the
    final stretch (up to 2048 tokens) of each context is synthesised."""
    cdf = zipf_cdf(cfg.vocab)
    templates = make_templates(cfg, cdf)
    tmpl_flat, tmpl_off = _flatten(templates)
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[2]))
    if ctx_len is None:
        ctx_len = context_lengths(cfg)
    tails = np.full((cfg.B, cfg.P), -1, dtype=np.int32)
    tail_len = np.zeros(cfg.B, dtype=np.int32)
    for i in range(cfg.B):
        n = int(min(ctx_len[i], max(2048, 2 * cfg.tmpl_hi)))
        seq = _span_sequence(rng, n, cfg, templates, tmpl_flat, tmpl_off, cdf)
        m = min(cfg.P, n)
        tails[i, cfg.P - m:] = seq[n - m:]
        tail_len[i] = m
    return tails, tail_len


def make_request_contexts(cfg: WorkloadConfig, ctx_len: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Whole contexts of the live requests, back to back (int32) with int64 bounds [B+1]: the final stretch of each is
    the one `make_request_tails` synthesises (so the last P tokens agree with its tails), the part before it comes
    from the same span recipe on a seed stream of its own.  Templates recur inside a context, which is the
    self-repetition that drafting from the own context feeds on."""
    cdf = zipf_cdf(cfg.vocab)
    templates = make_templates(cfg, cdf)
    tmpl_flat, tmpl_off = _flatten(templates)
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[2]))
    rng_head = np.random.Generator(np.random.PCG64(seed_streams(cfg)[2].spawn(1)[0]))
    if ctx_len is None:
        ctx_len = context_lengths(cfg)
    parts = []
    for i in range(cfg.B):
        n = int(min(ctx_len[i], max(2048, 2 * cfg.tmpl_hi)))
        seq = _span_sequence(rng, n, cfg, templates, tmpl_flat, tmpl_off, cdf)
        head = int(ctx_len[i]) - n
        if head > 0:
            parts.append(_span_sequence(rng_head, head, cfg, templates, tmpl_flat, tmpl_off, cdf))
        parts.append(seq)
    off = np.zeros(cfg.B + 1, dtype=np.int64)
    off[1:] = np.cumsum(np.asarray(ctx_len[:cfg.B], dtype=np.int64))
    return np.concatenate(parts).astype(np.int32), off


# ----------------------------------------------------------------------------------------------
# bf16 tensors: counter hash -> table of normal quantiles (exact integer ops, any torch device)
# ----------------------------------------------------------------------------------------------

_MASK32 = (1 << 32) - 1


def normal_table() -> torch.Tensor:
    """65536 bf16 values: the standard normal quantile at (i + 0.5) / 65536, computed in fp64 on the host."""
    p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
    z = math.sqrt(2.0) * torch.special.erfinv(2.0 * p - 1.0)
    return z.to(torch.bfloat16)


def _mix(x: torch.Tensor) -> torch.Tensor:
    """splitmix64-style finaliser on int64 tensors (two's-complement wrap-around, logical shifts by masking)."""
    x = (x ^ ((x >> 30) & ((1 << 34) - 1))) * (-4658895280553007687)      # 0xBF58476D1CE4E5B9
    x = (x ^ ((x >> 27) & ((1 << 37) - 1))) * (-7723592293110705685)      # 0x94D049BB133111EB
    return x ^ ((x >> 31) & ((1 << 33) - 1))


def hashed_normal(seed: int, index: torch.Tensor, table: torch.Tensor) -> torch.Tensor:
    """bf16 N(0,1)-distributed value for every int64 logical element index (same bits on every device)."""
    x = index * (-7046029254386353131) + int(seed)                         # 0x9E3779B97F4A7C15
    h = _mix(x)
    return table[(h >> 48) & 0xFFFF]


@dataclass
class AttnInputs:
    q: torch.Tensor              # bf16 [B, N, Hq, D]
    k_pool: torch.Tensor         # bf16 [num_pages, Hkv, page_size, D]
    v_pool: torch.Tensor         # bf16 [num_pages, Hkv, page_size, D]
    page_table: torch.Tensor     # int32 [B, max_pages]
    prefix_len: torch.Tensor     # int32 [B]
    num_pages: int
    max_pages: int


def _kv_seed(cfg: WorkloadConfig) -> int:
    return int(seed_streams(cfg)[3].generate_state(1, dtype=np.uint64)[0] >> 1)


def logical_kv(cfg: WorkloadConfig, req: int, pos: torch.Tensor, which: int, table: torch.Tensor,
               seed: Optional[int] = None) -> torch.Tensor:
    """bf16 [len(pos), Hkv, D]: K (which=0) or V (which=1) of request `req` at logical positions `pos`.
    Values depend on (request, position, head, d) only, never on where a page lives physically."""
    seed = _kv_seed(cfg) if seed is None else seed
    dev = pos.device
    h = torch.arange(cfg.Hkv, dtype=torch.int64, device=dev)
    d = torch.arange(cfg.D, dtype=torch.int64, device=dev)
    base = (req * (1 << 20) + pos.to(torch.int64))                          # positions < 2^20
    idx = ((base[:, None, None] * cfg.Hkv + h[None, :, None]) * cfg.D + d[None, None, :]) * 2 + which
    return hashed_normal(seed, idx, table.to(dev))


def make_queries(cfg: WorkloadConfig, device: torch.device | str = "cpu") -> torch.Tensor:
    table = normal_table().to(device)
    n = cfg.B * cfg.N * cfg.Hq * cfg.D
    idx = torch.arange(n, dtype=torch.int64, device=device)
    return hashed_normal(_kv_seed(cfg) ^ 0x5151, idx, table).view(cfg.B, cfg.N, cfg.Hq, cfg.D)


def make_page_table(cfg: WorkloadConfig, ctx_len: np.ndarray) -> Tuple[np.ndarray, int, int]:
    """Physical pages are a seeded random permutation of the pool (allocator churn).  Request i owns the
    pages that cover logical positions 0 .. ctx_len[i] - 1 + N (prefix, root slot and draft slots)."""
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[4]))
    need = (ctx_len - 1 + cfg.N + cfg.page_size - 1) // cfg.page_size
    num_pages = int(need.sum()) + 3                 # a few pages no request owns
    max_pages = int(need.max())
    perm = rng.permutation(num_pages).astype(np.int32)
    table = np.full((cfg.B, max_pages), -1, dtype=np.int32)
    at = 0
    for i in range(cfg.B):
        table[i, :need[i]] = perm[at:at + need[i]]
        at += int(need[i])
    return table, num_pages, max_pages


def make_attention_inputs(cfg: WorkloadConfig, ctx_len: np.ndarray, device: torch.device | str = "cpu",
                          chunk_tokens: int = 1 << 16) -> AttnInputs:
    """Builds the paged pools on `device`.  prefix_len = context length - 1: the root slot's K/V (the last
    context token) is new in this step and sits at logical position prefix_len, draft slot j at prefix_len + j.
    Rows of a request's last page beyond its last slot, and pages nobody owns, are filled too (with values
    keyed to a dummy request id) so that no kernel can pass by reading uninitialised memory."""
    table = normal_table().to(device)
    pt, num_pages, max_pages = make_page_table(cfg, ctx_len)
    pg = cfg.page_size
    k_pool = torch.empty((num_pages, cfg.Hkv, pg, cfg.D), dtype=torch.bfloat16, device=device)
    v_pool = torch.empty_like(k_pool)
    seed = _kv_seed(cfg)
    owned = np.zeros(num_pages, dtype=bool)
    for i in range(cfg.B):
        n_pages = int((ctx_len[i] - 1 + cfg.N + pg - 1) // pg)
        pages = torch.from_numpy(pt[i, :n_pages].astype(np.int64)).to(device)
        owned[pt[i, :n_pages]] = True
        for p0 in range(0, n_pages, max(1, chunk_tokens // pg)):
            p1 = min(n_pages, p0 + max(1, chunk_tokens // pg))
            pos = torch.arange(p0 * pg, p1 * pg, dtype=torch.int64, device=device)
            for which, pool in ((0, k_pool), (1, v_pool)):
                val = logical_kv(cfg, i, pos, which, table, seed)            # [tokens, Hkv, D]
                val = val.view(p1 - p0, pg, cfg.Hkv, cfg.D).permute(0, 2, 1, 3)
                pool[pages[p0:p1]] = val
    free = torch.from_numpy(np.flatnonzero(~owned).astype(np.int64)).to(device)
    if len(free):
        pos = torch.arange(len(free) * pg, dtype=torch.int64, device=device)
        for which, pool in ((0, k_pool), (1, v_pool)):
            val = logical_kv(cfg, cfg.B + 7, pos, which, table, seed)
            pool[free] = val.view(len(free), pg, cfg.Hkv, cfg.D).permute(0, 2, 1, 3)
    q = make_queries(cfg, device)
    return AttnInputs(q=q, k_pool=k_pool, v_pool=v_pool,
                      page_table=torch.from_numpy(pt).to(device),
                      prefix_len=torch.from_numpy((ctx_len - 1).astype(np.int32)).to(device),
                      num_pages=num_pages, max_pages=max_pages)


# ----------------------------------------------------------------------------------------------
# target ids
# ----------------------------------------------------------------------------------------------

def make_targets(cfg: WorkloadConfig, ids: np.ndarray, parent: np.ndarray, num_nodes: np.ndarray,
                 mode: int = 0) -> np.ndarray:
    """Target ids int32[B, N] for a given set of draft trees (any source: they are an input here).

    mode 0 (per slot): target[p] stands for the token the target model emits after slot p.  A slot with
    children agrees with its first (lowest-numbered) child with probability 1 - mismatch, otherwise it is a
    different token; a leaf gets a uniform random token.
    mode 1 (per node): target[j] equals ids[j] with probability 1 - mismatch, otherwise a different token."""
    rng = np.random.Generator(np.random.PCG64(seed_streams(cfg)[5]))
    B, N = ids.shape
    out = rng.integers(0, cfg.vocab, size=(B, N)).astype(np.int32)
    flip = rng.random((B, N)) < cfg.mismatch
    shift = rng.integers(0, cfg.vocab - 1, size=(B, N))
    for i in range(B):
        n = int(num_nodes[i])
        if mode == 1:
            for j in range(n):
                out[i, j] = (ids[i, j] + 1 + shift[i, j]) % cfg.vocab if flip[i, j] else ids[i, j]
            continue
        first_child = np.full(N, -1, dtype=np.int64)
        for j in range(n - 1, 0, -1):
            first_child[parent[i, j]] = j
        for p in range(n):
            c = first_child[p]
            if c >= 0:
                out[i, p] = (ids[i, c] + 1 + shift[i, p]) % cfg.vocab if flip[i, p] else ids[i, c]
    return out


def make_targets_device(cfg: WorkloadConfig, ids: torch.Tensor, parent: torch.Tensor, num_nodes: torch.Tensor,
                        step: int) -> torch.Tensor:
    """Per-slot target ids (mode 0 of `make_targets`) made on the device from device-resident trees, for benchmark
    steps whose trees change from step to step: a slot with children agrees with its lowest-numbered child with
    probability 1 - mismatch, otherwise it is a different token; a leaf gets a uniform random token.  Randomness is
    a counter hash of (step, request, slot).  This stands in for the target model's sampled tokens; it is input
    generation, not part of the method."""
    B, N = ids.shape
    dev = ids.device
    j = torch.arange(N, device=dev, dtype=torch.int64).expand(B, N)
    live = (j >= 1) & (j < num_nodes.to(torch.int64)[:, None])
    first_child = torch.full((B, N), N, dtype=torch.int64, device=dev)
    first_child.scatter_reduce_(1, parent.clamp(min=0).to(torch.int64), torch.where(live, j, torch.full_like(j, N)), "amin",
                                include_self=True)
    has = first_child < N
    child_id = ids.to(torch.int64).gather(1, first_child.clamp(max=N - 1))
    idx = torch.arange(B * N, device=dev, dtype=torch.int64).view(B, N) + (int(step) + 1) * (1 << 24)
    h = _mix(idx * (-7046029254386353131) + (int(seed_streams(cfg)[5].entropy) & 0xFFFF))
    u = ((h >> 40) & 0xFFFFFF).to(torch.float64) / float(1 << 24)
    shift = (h >> 8) & 0x7FFFFFFF
    flip = u < cfg.mismatch
    rnd = shift % cfg.vocab
    wrong = (child_id + 1 + shift % (cfg.vocab - 1)) % cfg.vocab
    out = torch.where(has, torch.where(flip, wrong, child_id), rnd)
    return out.to(torch.int32)
