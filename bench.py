#!/usr/bin/env python
"""Benchmark of the speculate-and-verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload high|low|longtail|wide|tiny] [--impl ours|reference]

A step = one pass of the whole hot path over one batch of live requests: war_draft (suffix match + draft trees)
-> war_verify_attn (tree-masked GQA attention over the paged bf16 KV cache) -> war_accept.  The index build is
set-up and is reported separately.  The metric is verified tokens per second: sum over requests of
(accepted draft tokens + the one token the target model always yields) divided by the step time.

One JSON line is printed by rank 0.  Its headline keys describe the High workload (256 requests; the configuration
the metric is quoted on): `value` has every input resident in HBM; `e2e` repeats the step with the per-step inputs
starting in pinned host memory and the results read back, copies inside the timed region; `roofline` puts the
verify-attention call against the measured HBM copy bandwidth; `cpu_baseline` times the CPU checker (oracle/) on a
bounded sample of the same requests on this machine's host cores and compares what it computes with what the GPU
produced for those requests (`parity_checked`, `parity_ok`).  The default invocation then runs the other four
configurations (`workloads`) and 4 to 64 requests of the High recipe (`load_sweep`), a few steps each, and a run
in which the requests advance between steps (`advancing`: war_commit after every step, so tails, prefix lengths and
trees change as in an engine).  `--workload X` runs one configuration only.

More than one GPU: `python bench.py --gpus N` starts N ranks itself (one process per GPU, torchrun) unless it is
already running under torchrun.  Every rank is a replica with its own requests (weak scaling, no exchange inside a
step); the method's one exchange, the end-of-step all-gather of finished trajectories followed by the same index
append on every rank, is timed as `exchange_ms`.

`--impl reference` times the CPU checker alone (there is no other reference implementation to run).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified tokens/s per speculate+verify step"
UNIT = "tokens/s"
FUSED_MAX_B = 64               # up to this many requests war_verify_attn is one launch, else plan + kernel + combine


def launches_per_step(B: int, kernel: int = 0, score_lengths: int = 1, own_context: bool = False) -> int:
    """Kernels of this library launched by one step: draft, verify attention (1 or 3), accept (+ variants)."""
    return 1 + (1 if (B <= FUSED_MAX_B and kernel == 0) else 3) + 1 + (1 if score_lengths > 1 else 0) + (2 if own_context else 0)


def kv_bytes(cfg, prefix_len: np.ndarray, num_nodes: np.ndarray) -> int:
    """Bytes the verify attention must read once: K and V rows of every prefix position and every tree slot."""
    tokens = int((prefix_len.astype(np.int64) + num_nodes.astype(np.int64))[num_nodes > 0].sum())
    return tokens * cfg.Hkv * cfg.D * 2 * 2


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.gpu = [], None, gpu_index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def mark(self) -> int:
        return len(self.rows)

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, first: int = 0, last=None):
        sm, mx, watts, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[first:last]:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            try:
                watts.append(float(r[2]))
            except Exception:
                pass
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(watts)) if watts else None, "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(cfg, corpus, tails, tail_len, attn, ctx, targets_fn, requests, budget_s=None, keep=False):
    """Runs the CPU checker on the given requests (in order, stopping once budget_s is spent, at least one).
    Returns (tokens verified, seconds, requests done, results): results[i] = what the checker computed for request
    i (trees, attention, acceptance) when `keep` is set."""
    from oracle import accept_oracle, attention_oracle, draft_oracle
    import torch
    scale = 1.0 / float(np.sqrt(cfg.D))
    t0 = time.perf_counter()
    verified, done, results = 0, 0, {}
    pt = attn.page_table.cpu().numpy() if attn is not None else None
    for i in requests:
        ml, ends = draft_oracle.longest_suffix_match(corpus, tails[i], int(tail_len[i]))
        ids, parent, count = draft_oracle.build_draft_tree(corpus, tails[i], ml, ends, cfg.N, cfg.topk)
        n = len(ids)
        full_ids = np.full((1, cfg.N), -1, np.int32); full_par = np.full((1, cfg.N), -1, np.int32)
        full_ids[0, :n] = ids; full_par[0, :n] = parent
        K, V = attention_oracle.gather_request_kv(attn.k_pool, attn.v_pool, pt[i], int(ctx[i]) - 1 + n)
        q = attn.q[i].to("cpu").to(torch.float64).numpy()
        out, lse = attention_oracle.verify_attention_request(q, K, V, int(ctx[i]) - 1, full_par[0], n, scale)
        target = targets_fn(i, full_ids, full_par, n)
        alen, path, bonus = accept_oracle.accept_request(full_ids[0], full_par[0], n, target, 0)
        verified += alen + 1
        done += 1
        if keep:
            results[i] = dict(match_len=ml, n=n, ids=np.asarray(ids), parent=np.asarray(parent), count=np.asarray(count),
                              out=out, lse=lse, accept_len=alen, path=list(path), bonus=bonus)
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    return verified, time.perf_counter() - t0, done, results


def parity_against(results, gpu, N) -> list:
    """Compares the checker's results with the GPU's for the same requests: integers exactly, attention by the rules of
    the parity tests (atol / rtol 1e-2 on the fp32 cast, per-row relative L2 <= 1e-2, lse within 1e-3).  Returns the
    list of mismatches (empty = parity)."""
    bad = []
    for i, r in results.items():
        n = r["n"]
        if int(gpu["match_len"][i]) != r["match_len"] or int(gpu["num_nodes"][i]) != n:
            bad.append((i, "match_len / num_nodes")); continue
        for key in ("ids", "parent", "count"):
            if not np.array_equal(gpu[key][i, :n], r[key]):
                bad.append((i, key))
        path = list(gpu["path"][i, :int(gpu["accept_len"][i])])
        if int(gpu["accept_len"][i]) != r["accept_len"] or path != list(r["path"]) or int(gpu["bonus"][i]) != r["bonus"]:
            bad.append((i, "accept"))
        g, w = gpu["out"][i, :n].astype(np.float64), r["out"]
        if not np.allclose(g.astype(np.float32), w.astype(np.float32), atol=1e-2, rtol=1e-2):
            bad.append((i, "attention atol/rtol"))
        rel = np.sqrt(((g - w) ** 2).sum(-1)) / (np.sqrt((w ** 2).sum(-1)) + 1e-30)
        if rel.max() >= 1e-2:
            bad.append((i, f"attention relative L2 {rel.max():.2e}"))
        if not np.allclose(gpu["lse"][i, :n], r["lse"].astype(np.float32), atol=1e-3, rtol=1e-4):
            bad.append((i, "lse"))
    return bad


def threads_in_use() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        n = 1
    return int(min(n, len(os.sched_getaffinity(0))))


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return (float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy)",
                float(d.get("bf16_tflops_sustained", 0.0)) or 1400.0, "measured (MEASURED_PEAKS.json bf16_tflops_sustained)")
    return 6650.0, "fallback", 1400.0, "fallback"


def roofline_of(cfg, ctx, h_nn, attn_ms, launches: str):
    """Roofline entry of the verify-attention call: algorithmic K/V bytes (or flops) per launch over its CUDA-event
    time, against the measured peak.  `traffic` (DRAM bytes from an ncu capture) is only known where a committed
    profile of a few-GB case of the same recipe gives the read amplification; otherwise null."""
    peak, peak_src, peak_tf, peak_tf_src = peaks()
    kvb = kv_bytes(cfg, ctx - 1, h_nn)
    achieved = kvb / (attn_ms * 1e-3) / 1e9
    G = cfg.Hq // cfg.Hkv
    live = h_nn > 0
    # the same launch seen from the tensor pipe: 4 * rows * D flops per KV token and kv head (QK^T and PV), rows = the
    # (slot, head-of-group) pairs that exist (not the padded MMA tile)
    flops = float(((ctx - 1 + h_nn)[live].astype(np.float64) * (4.0 * G * h_nn[live] * cfg.D)).sum() * cfg.Hkv)
    t_hbm, t_tensor = kvb / (peak * 1e9), flops / (peak_tf * 1e12)
    traffic = None
    amp_path = os.path.join(ROOT, "profiles", f"attn_sm100_kernel_{cfg.name}_traffic.md")
    if os.path.exists(amp_path):
        import re
        with open(amp_path) as f:
            m = re.search(r"^dram_read_amplification\s*=\s*([0-9.]+)", f.read(), flags=re.M)
        traffic = int(kvb * float(m.group(1))) if m else None
    if t_tensor > t_hbm:
        roof = {"bound": "tensor", "achieved": flops / (attn_ms * 1e-3) / 1e12, "peak": peak_tf, "unit": "TFLOP/s",
                "frac": t_tensor / (attn_ms * 1e-3), "traffic": traffic, "flops_per_launch": flops,
                "peak_source": peak_tf_src, "hbm_gbs": achieved}
    else:
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "frac_of_8TBps_nominal": achieved / 8000.0, "peak_source": peak_src,
                "tensor_tflops": flops / (attn_ms * 1e-3) / 1e12}
    kernel = {"name": f"war_verify_attn ({launches})", "bytes_per_launch": kvb, "ms_per_launch": attn_ms}
    return roof, kernel


class Workload:
    """One configuration resident on one GPU: index, requests, KV cache, the step's buffers."""

    def __init__(self, war, W, cfg, dev, args, ix=None, corpus=None):
        import torch
        self.war, self.W, self.cfg, self.dev, self.args = war, W, cfg, dev, args
        self.torch = torch
        self.tok, self.off = corpus if corpus is not None else W.make_corpus(cfg)
        self.tails, self.tl = W.make_request_tails(cfg)
        self.ctx = W.context_lengths(cfg)
        need = (int(((self.ctx - 1 + cfg.N + cfg.page_size - 1) // cfg.page_size).sum()) * cfg.Hkv * cfg.page_size * cfg.D * 2 * 2
                + (0 if ix is not None else (len(self.tok) + cfg.n_traj) * (14 + 44))
                + 3 * cfg.B * cfg.N * cfg.Hq * cfg.D * 2 + (1 << 30))
        free, _total = torch.cuda.mem_get_info(dev)
        if free < need:
            raise MemoryError(f"workload {cfg.name} needs about {need / 2**30:.1f} GiB of device memory, "
                              f"{free / 2**30:.1f} GiB are free on {dev}")
        self.index_stats = {}
        self.owns_index = ix is None
        self.ix = ix if ix is not None else self._build_index()
        self.attn = W.make_attention_inputs(cfg, self.ctx, device=dev)
        self._buffers(cfg.B)

    def _build_index(self):
        torch, war, cfg, dev = self.torch, self.war, self.cfg, self.dev
        tok, off = self.tok, self.off
        d_tok = torch.from_numpy(tok).to(dev)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        ix = war.war_index_build(d_tok, off, cfg.vocab, cfg.P + cfg.N, len(tok) + cfg.n_traj)
        self.index_stats["index_build_s"] = time.perf_counter() - t0
        # the index the steps use is then made the way a rollout would make it: all but the last trajectories first, the
        # rest appended as an RL step's worth of new trajectories (an appended index answers exactly like a fresh build)
        k_new = max(1, cfg.n_traj // 32)
        # one draft call on this first index, so that the first call on the index the steps use (below) measures an empty
        # memo and not the one-time cost of the first launch of a kernel
        _t, _tl = torch.from_numpy(self.tails).to(dev), torch.from_numpy(self.tl).to(dev)
        _z = lambda *sh: torch.zeros(sh, dtype=torch.int32, device=dev)
        war.war_draft(ix, _t, _tl, cfg.N, cfg.topk, 1, _z(cfg.B), _z(cfg.B), _z(cfg.B, cfg.N), _z(cfg.B, cfg.N), None)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        war.war_index_evict(ix, k_new)                         # sliding window: the oldest 1/32 of the trajectories leave
        self.index_stats["index_evict"] = {"trajectories": k_new, "seconds": time.perf_counter() - t0}
        ix.destroy()
        ix = war.war_index_build(d_tok, off[:cfg.n_traj - k_new + 1], cfg.vocab, cfg.P + cfg.N, len(tok) + cfg.n_traj)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        war.war_index_append(ix, d_tok, off[cfg.n_traj - k_new:])
        self.index_stats["index_append"] = {"trajectories": k_new, "tokens": int(off[-1] - off[cfg.n_traj - k_new]),
                                            "seconds": time.perf_counter() - t0}
        self.index_stats["index_tokens"] = int(len(tok))
        # the same amount once more as a stream-ordered update (the oldest trajectories leave first to make room): how
        # long the host is held (enqueue) and how long the stream is busy with it
        for j in range(2):                                     # (the first call grows the allocator's pool; the second is what an engine sees)
            war.war_index_evict(ix, k_new)                     # trajectories [j * k_new, (j + 1) * k_new) leave ... and come back below
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            e0.record()
            war.war_index_append_async(ix, d_tok, off[j * k_new:(j + 1) * k_new + 1])
            e1.record()
            host_s = time.perf_counter() - t0
            torch.cuda.synchronize()
        self.index_stats["index_append_async"] = {"trajectories": k_new, "tokens": int(off[2 * k_new] - off[k_new]), "host_seconds": host_s,
                                                  "stream_seconds": 1e-3 * e0.elapsed_time(e1)}
        return ix

    def _buffers(self, B):
        """(Re)creates the step's buffers for the first B requests of the resident set."""
        torch, war, cfg, dev, args = self.torch, self.war, self.cfg, self.dev, self.args
        N, P_ = cfg.N, self.tails.shape[1]
        self.B = B
        i32 = dict(dtype=torch.int32, device=dev)
        # the step's small integer inputs (tails, their lengths, the target model's tokens) share one allocation
        self.d_in = torch.zeros(B * (P_ + 1 + N), **i32)
        self.d_tails, self.d_tl = self.d_in[:B * P_].view(B, P_), self.d_in[B * P_:B * (P_ + 1)]
        self.d_target = self.d_in[B * (P_ + 1):].view(B, N)
        self.d_tails.copy_(torch.from_numpy(self.tails[:B])); self.d_tl.copy_(torch.from_numpy(self.tl[:B]))
        # the step's small integer results live side by side, so the end-to-end leg reads them back with one copy
        self.d_small = torch.zeros(B * (3 + 3 * N), **i32)
        s = self.d_small
        self.d_nn, self.d_alen, self.d_bonus = s[0:B], s[B:2 * B], s[2 * B:3 * B]
        self.d_ids, self.d_par, self.d_path = (s[3 * B + k * B * N:3 * B + (k + 1) * B * N].view(B, N) for k in range(3))
        self.d_ml, self.d_cnt = torch.zeros(B, **i32), torch.zeros((B, N), **i32)
        a = self.attn
        self.q, self.page_table, self.prefix_len = a.q[:B], a.page_table[:B], a.prefix_len[:B].clone()
        self.d_out = torch.zeros_like(self.q)
        self.d_lse = torch.zeros(self.q.shape[:3], dtype=torch.float32, device=dev)
        self.scale = 1.0 / float(np.sqrt(cfg.D))
        self.params = war.attn_params(self.q, a.k_pool, a.v_pool, self.page_table, self.scale, args.kernel)
        self.ws = war.new_workspace(self.params, dev)
        if args.score_lengths > 1:
            self.d_used = torch.zeros(B, **i32)
            self.draft_ws = torch.empty(war.war_draft_scored_workspace_bytes(B, cfg.P, N, cfg.topk, args.score_lengths),
                                        dtype=torch.uint8, device=dev)
        if args.own_context:
            sub = self.W.scaled(cfg, B=B)
            h_ctx, h_ctx_off = self.W.make_request_contexts(sub, self.ctx[:B])
            self.d_ctx, self.d_ctx_off = torch.from_numpy(h_ctx).to(dev), torch.from_numpy(h_ctx_off).to(dev)
            tree = lambda: [torch.zeros(B, **i32), torch.zeros(B, **i32)] + [torch.zeros((B, N), **i32) for _ in range(3)]
            self.g_tree, self.l_tree = tree(), tree()
            self.d_src = torch.zeros(B, **i32)
            self.local_stream, self.local_done = torch.cuda.Stream(), torch.cuda.Event()
        # targets depend on the trees; the trees are a deterministic function of the inputs, so draft once to make them
        # (on a freshly published index this is also the first draft call: its memo of large-node expansions is empty)
        ev = lambda: torch.cuda.Event(enable_timing=True)
        c0, c1 = ev(), ev()
        torch.cuda.synchronize()
        c0.record(); self.draft(); c1.record()
        torch.cuda.synchronize()
        self.draft_cold_ms = c0.elapsed_time(c1)
        self.h_ids, self.h_par, self.h_nn = self.d_ids.cpu().numpy(), self.d_par.cpu().numpy(), self.d_nn.cpu().numpy()
        self.targets = self.W.make_targets(self.W.scaled(cfg, B=B), self.h_ids, self.h_par, self.h_nn, 0)
        self.d_target.copy_(torch.from_numpy(self.targets))

    # ---- the step ----
    def draft(self):
        torch, war, cfg, args = self.torch, self.war, self.cfg, self.args
        N = cfg.N
        if args.own_context:
            # the two drafts share no data: the own-context scan runs beside the index lookup, then the better tree is kept
            main = torch.cuda.current_stream()
            self.local_stream.wait_stream(main)
            with torch.cuda.stream(self.local_stream):
                war.war_draft_local(self.d_ctx, self.d_ctx_off, self.d_tl, cfg.P, N, cfg.topk, 1, *self.l_tree, args.spec_batch_limit)
                self.local_done.record(self.local_stream)
            war.war_draft(self.ix, self.d_tails, self.d_tl, N, cfg.topk, 1, *self.g_tree, args.spec_batch_limit)
            main.wait_event(self.local_done)
            war.war_draft_pick(self.g_tree, self.l_tree, self.d_src, self.d_ml, self.d_nn, self.d_ids, self.d_par, self.d_cnt)
        elif args.score_lengths > 1:
            war.war_draft_scored(self.ix, self.d_tails, self.d_tl, N, cfg.topk, 1, args.score_lengths, self.draft_ws, self.d_ml,
                                 self.d_used, self.d_nn, self.d_ids, self.d_par, self.d_cnt, args.spec_batch_limit)
        else:
            war.war_draft(self.ix, self.d_tails, self.d_tl, N, cfg.topk, 1, self.d_ml, self.d_nn, self.d_ids, self.d_par, self.d_cnt,
                          args.spec_batch_limit)

    def verify(self, out=None):
        a = self.attn
        self.war.war_verify_attn(self.q, a.k_pool, a.v_pool, self.page_table, self.prefix_len, self.d_nn, self.d_par, self.params,
                                 self.ws, self.d_out if out is None else out, self.d_lse)

    def accept(self):
        self.war.war_accept(self.d_ids, self.d_par, self.d_nn, self.d_target, 0, self.d_alen, self.d_path, self.d_bonus)

    def step(self, attn_events=None):
        self.draft()
        if attn_events is not None:
            attn_events[0].record()
        self.verify()
        if attn_events is not None:
            attn_events[1].record()
        self.accept()

    # ---- measurements ----
    def time_steps(self, steps, warmup, barrier, flush_l2=False, cuda_graph=False, clocks=None):
        """W warm-up steps, then `steps` timed steps between two device-wide synchronisations (CUDA events on the
        launching stream).  Returns a dict of timings in ms."""
        torch = self.torch
        ev = lambda: torch.cuda.Event(enable_timing=True)
        t_warm = time.perf_counter()
        for _ in range(warmup):
            self.step()
        if clocks is not None:                                 # nvidia-smi needs a few hundred ms to start reporting
            while time.perf_counter() - t_warm < 0.6 and not clocks.rows:
                self.step()
                torch.cuda.synchronize()
        barrier()
        attn_ev = [(ev(), ev()) for _ in range(steps)]
        step_ev = [(ev(), ev()) for _ in range(steps)]
        scratch = torch.empty(256 << 20, dtype=torch.uint8, device=self.dev) if flush_l2 else None
        barrier()
        start, stop = ev(), ev()
        graph_ms = None
        if cuda_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                self.step()
            torch.cuda.current_stream().wait_stream(side)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                self.step()
            for _ in range(warmup):
                graph.replay()
            barrier()
            start.record()
            for s in range(steps):
                graph.replay()
            stop.record()
            barrier()
            graph_ms = start.elapsed_time(stop)
            start, stop = ev(), ev()
        first_sample = clocks.mark() if clocks is not None else 0
        start.record()
        for s in range(steps):
            if scratch is not None:
                scratch.fill_(s & 0xFF)
            step_ev[s][0].record()
            self.step(attn_ev[s])
            step_ev[s][1].record()
        stop.record()
        barrier()
        per_step = np.array([a.elapsed_time(b) for a, b in step_ev])
        total_ms = float(per_step.sum()) if flush_l2 else start.elapsed_time(stop)
        res = {"total_ms": graph_ms if graph_ms is not None else total_ms, "eager_ms": total_ms,
               "attn_ms": float(np.mean([a.elapsed_time(b) for a, b in attn_ev])),
               "draft_ms": float(np.mean([step_ev[s][0].elapsed_time(attn_ev[s][0]) for s in range(steps)])),
               "accept_ms": float(np.mean([attn_ev[s][1].elapsed_time(step_ev[s][1]) for s in range(steps)])),
               "per_step": per_step, "first_sample": first_sample}
        del scratch
        return res

    def steps_for(self, seconds: float, at_least: int) -> int:
        """How many steps fill about `seconds` (from three timed ones)."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.step()
        e0.record()
        for _ in range(3):
            self.step()
        e1.record()
        torch.cuda.synchronize()
        per = max(1e-3, e0.elapsed_time(e1) / 3.0)
        return int(max(at_least, min(5000, seconds * 1e3 / per)))

    def counts(self):
        h_alen = self.d_alen.cpu().numpy()
        return int((h_alen.astype(np.int64) + 1).sum()), int(self.h_nn.sum()), float(h_alen.mean())

    def time_e2e(self, steps, barrier):
        """The step with its per-step inputs starting in pinned host memory and its results read back, every copy inside
        the timed region.  Returns (ms for `steps` steps, h2d bytes per step, d2h bytes per step)."""
        torch = self.torch
        pin = lambda t: t.cpu().pin_memory()
        d_out = self.d_out
        overlap_out_ok = d_out.numel() * d_out.element_size() >= (4 << 20)   # small outputs: one stream, one buffer
        h_q, h_in = pin(self.q), pin(self.d_in)
        r_small, r_out = pin(self.d_small), pin(d_out)            # trees, accepted paths and bonus tokens; attention output
        # The host waits every step for the small results (the next step's inputs depend on the accepted tokens); the
        # attention output is a bulk result nobody waits for, so its copy runs on a stream of its own out of one of two
        # output buffers and overlaps the next step.  Every step's copies are still inside the timed region: the region
        # ends with a device-wide synchronize.
        d_outs = [d_out, torch.zeros_like(d_out)] if overlap_out_ok else [d_out, d_out]
        r_outs = [r_out, pin(d_out)] if overlap_out_ok else [r_out, r_out]
        out_stream = torch.cuda.Stream()
        out_copied = [torch.cuda.Event(), torch.cuda.Event()]
        attn_done, small_done = torch.cuda.Event(), torch.cuda.Event()
        h2d = sum(t.numel() * t.element_size() for t in (h_q, h_in))
        d2h = sum(t.numel() * t.element_size() for t in (r_small, r_out))
        # the queries are only needed by the verification: their copy runs on a second stream beside the draft call
        copy_stream = torch.cuda.Stream()
        q_ready = torch.cuda.Event()
        main_stream = torch.cuda.current_stream()
        overlap_q = h_q.numel() * h_q.element_size() >= (4 << 20)   # for a small batch the extra stream costs more than it hides

        def e2e_step(s):
            o, r_o = d_outs[s & 1], r_outs[s & 1]
            self.d_in.copy_(h_in, non_blocking=True)
            if overlap_q:
                copy_stream.wait_stream(main_stream)            # the previous step's readers of q are done
                with torch.cuda.stream(copy_stream):
                    self.q.copy_(h_q, non_blocking=True)
                    q_ready.record(copy_stream)
            else:
                self.q.copy_(h_q, non_blocking=True)
            self.draft()
            if overlap_q:
                main_stream.wait_event(q_ready)
            if overlap_out_ok and s >= 2:
                main_stream.wait_event(out_copied[s & 1])       # this output buffer's previous copy has left the device
            self.verify(o)
            if overlap_out_ok:
                attn_done.record(main_stream)
                with torch.cuda.stream(out_stream):
                    out_stream.wait_event(attn_done)
                    r_o.copy_(o, non_blocking=True)
                    out_copied[s & 1].record(out_stream)
            self.accept()
            r_small.copy_(self.d_small, non_blocking=True)
            if overlap_out_ok:
                small_done.record(main_stream)
                small_done.synchronize()                        # the caller needs the accepted tokens before the next step
            else:
                r_o.copy_(o, non_blocking=True)
                torch.cuda.synchronize()

        for s in range(2):
            e2e_step(s)
        barrier()
        t0 = time.perf_counter()
        for s in range(steps):
            e2e_step(2 + s)
        barrier()
        return 1e3 * (time.perf_counter() - t0), h2d, d2h

    def time_commit(self):
        """war_commit timed on its own, on copies of the request state (it is what a caller runs between two steps, not
        part of the step metric).  Run after everything that needs the cache as it is: it moves K/V rows."""
        torch, war, a = self.torch, self.war, self.attn
        ev = lambda: torch.cuda.Event(enable_timing=True)
        c_pl, c_tails, c_tl = self.prefix_len.clone(), self.d_tails.clone(), self.d_tl.clone()
        war.war_commit(self.d_ids, self.d_alen, self.d_path, self.d_bonus, a.k_pool, a.v_pool, self.page_table, c_pl, c_tails, c_tl)
        c_pl.copy_(self.prefix_len); c_tails.copy_(self.d_tails); c_tl.copy_(self.d_tl)
        c0, c1 = ev(), ev()
        torch.cuda.synchronize()
        c0.record()
        war.war_commit(self.d_ids, self.d_alen, self.d_path, self.d_bonus, a.k_pool, a.v_pool, self.page_table, c_pl, c_tails, c_tl)
        c1.record()
        torch.cuda.synchronize()
        return c0.elapsed_time(c1)

    def time_advancing(self, steps, warmup):
        """Steps between which the requests really advance: war_commit after every step makes the accepted tokens part
        of the context, so the tails, the prefix lengths, the trees and the index memo's hit pattern change from step
        to step as they do in an engine.  The target model's tokens for the new trees are made on the device between
        the verification and the acceptance (outside the timed intervals: they stand in for the model's sampling).
        Contexts are first shortened by the room the advance needs, so that they stay inside the allocated pages.
        Returns {ms_per_step (draft + verify + accept), commit_ms, verified tokens per step}."""
        torch, war, W, cfg, a = self.torch, self.war, self.W, self.cfg, self.attn
        ev = lambda: torch.cuda.Event(enable_timing=True)
        margin = (steps + warmup) * cfg.N
        saved = self.prefix_len.clone(), self.d_tails.clone(), self.d_tl.clone(), self.d_target.clone()
        self.prefix_len.copy_((self.prefix_len - margin).clamp(min=1))
        sub = W.scaled(cfg, B=self.B)
        spans, verified = [], 0
        for s in range(steps + warmup):
            e = [ev() for _ in range(6)]
            e[0].record(); self.draft(); self.verify(); e[1].record()
            self.d_target.copy_(W.make_targets_device(sub, self.d_ids, self.d_par, self.d_nn, s))
            e[2].record(); self.accept(); e[3].record()
            e[4].record()
            war.war_commit(self.d_ids, self.d_alen, self.d_path, self.d_bonus, a.k_pool, a.v_pool, self.page_table, self.prefix_len,
                           self.d_tails, self.d_tl)
            e[5].record()
            if s >= warmup:
                spans.append(e)
        torch.cuda.synchronize()
        status = war.war_device_status()
        step_ms = float(np.mean([x[0].elapsed_time(x[1]) + x[2].elapsed_time(x[3]) for x in spans]))
        commit_ms = float(np.mean([x[4].elapsed_time(x[5]) for x in spans]))
        verified = int((self.d_alen.to(torch.int64) + 1).sum().item())       # of the last step
        for dst, src in zip((self.prefix_len, self.d_tails, self.d_tl, self.d_target), saved):
            dst.copy_(src)
        return {"ms_per_step": step_ms, "commit_ms": commit_ms, "verified_last_step": verified, "device_status": status}

    def gpu_results(self):
        """What the GPU produced in the last step, as host arrays (for the parity check against the checker)."""
        c = lambda t: t.cpu().numpy()
        return dict(match_len=c(self.d_ml), num_nodes=c(self.d_nn), ids=c(self.d_ids), parent=c(self.d_par), count=c(self.d_cnt),
                    accept_len=c(self.d_alen), path=c(self.d_path), bonus=c(self.d_bonus), out=self.d_out.float().cpu().numpy(),
                    lse=c(self.d_lse))

    def close(self):
        if self.owns_index:
            self.ix.destroy()
        self.attn = None
        self.torch.cuda.empty_cache()


def summarize(wl, t, steps, launches):
    """The per-workload entry of the `workloads` / `load_sweep` tables."""
    roof, _ = roofline_of(wl.cfg if wl.B == wl.cfg.B else wl.W.scaled(wl.cfg, B=wl.B), wl.ctx[:wl.B], wl.h_nn, t["attn_ms"], launches)
    verified, slots, _ = wl.counts()
    ms = t["total_ms"] / steps
    return {"requests": wl.B, "ms_per_step": ms, "value": verified / (ms * 1e-3),
            "breakdown_ms": {"draft": t["draft_ms"], "verify_attn": t["attn_ms"], "accept": t["accept_ms"]},
            "bound": roof["bound"], "frac": roof["frac"], "achieved": roof["achieved"], "unit": roof["unit"]}


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=None,
                    help="run one configuration only (high, low, longtail, wide, tiny); default: high as the headline, then "
                         "the others, the load sweep and the advancing run")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", type=int, default=0,
                    help="0 = tensor-core verify attention (one launch up to 64 requests), 1 = plain CUDA-core kernel, "
                         "2 = tensor-core kernel with separate plan / combine launches")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="headline workload only (no other configurations, sweep, advancing run)")
    ap.add_argument("--flush-l2", action="store_true",
                    help="write a 256 MB scratch buffer before every timed step (for workloads whose KV cache fits L2); "
                         "ms_per_step is then the mean of the per-step event intervals, the flush excluded")
    ap.add_argument("--spec-batch-limit", type=int, default=0,
                    help="workload-aware switch of war_draft: above this many running requests the step is a plain decode "
                         "step (root-only trees); 0 = always speculate")
    ap.add_argument("--score-lengths", type=int, default=1,
                    help="draft from the best-scoring of this many suffix lengths (war_draft_scored) instead of from the "
                         "longest match (war_draft); 1 = war_draft, the configuration the metric is quoted on")
    ap.add_argument("--own-context", action="store_true",
                    help="also draft from each request's own context (war_draft_local, on a second stream beside war_draft) "
                         "and verify the better-scoring tree of the two (war_draft_pick)")
    ap.add_argument("--cuda-graph", action="store_true",
                    help="replay the step (draft, verify attention, accept) from one captured CUDA graph, as the paper's engine "
                         "does for both modes; the per-kernel breakdown and the roofline then come from a second, eagerly "
                         "launched pass of the same steps")
    ap.add_argument("--requests", type=int, default=0,
                    help="run the workload's recipe with this many requests instead of its own count (profiling-size cases)")
    ap.add_argument("--advance", action="store_true", help="with --workload: also do the advancing run (war_commit between steps)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    # ---- more than one GPU asked for, not under torchrun yet: start the ranks (one process per GPU) ----
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} asked for, {have} GPU(s) visible")
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import torch
    from paper_2607_17299_b200 import workloads as W
    headline = args.workload or "high"
    cfg = W.CONFIGS[headline]
    if args.requests > 0:
        cfg = W.scaled(cfg, B=args.requests)
    extras = args.workload is None and not args.no_extras and args.requests == 0 and world == 1

    def describe(c, flush=False):
        return {"workload": f"{c.name}: corpus {c.n_traj} trajectories, {c.B} requests, tree <= {c.N} slots, "
                            f"{c.Hq}q/{c.Hkv}kv heads, d={c.D}, page {c.page_size}",
                "requests_per_gpu": c.B, "parallelism": f"replica x{world}" if world > 1 else "single gpu",
                "l2": "inputs (KV cache) far larger than L2, no flush needed" if c.name != "tiny" else
                      ("L2 flushed (256 MB written) before every step" if flush else
                       "KV cache fits L2: value is an L2-resident number (--flush-l2 gives the cold one)")}
    base_config = describe(cfg, args.flush_l2)

    # ------------------------------------------------------------------------------------------
    if args.impl == "reference":
        if rank != 0:
            return
        from oracle import draft_oracle
        tok, off = W.make_corpus(cfg)
        tails, tl = W.make_request_tails(cfg)
        ctx = W.context_lengths(cfg)
        corpus = draft_oracle.Corpus(tok, off)
        per_step = 4
        # KV for a handful of distinct requests, generated once on the host (set-up, untimed); steps cycle through them
        distinct = list(range(min(cfg.B, 16)))
        sub = W.scaled(cfg, B=len(distinct))
        attn = W.make_attention_inputs(sub, ctx[distinct], device="cpu")

        def targets_fn(i, ids, par, n):
            return W.make_targets(W.scaled(cfg, B=1), ids, par, np.array([n]), 0)[0]
        times, verified = [], 0
        for s in range(args.steps + args.warmup):
            reqs = [(s * per_step + k) % len(distinct) for k in range(per_step)]
            v, dt, _, _ = oracle_sample(cfg, corpus, tails, tl, attn, ctx, targets_fn, reqs)
            if s >= args.warmup:
                times.append(dt); verified += v
        total = sum(times)
        value = verified / total
        cores = threads_in_use()
        line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": dict(base_config, sample=f"{per_step} requests per step, cycling through the batch"),
                "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                                 "sample": f"{per_step} requests per step x {args.steps} steps"},
                "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    # ------------------------------------------------------------------------------------------
    from paper_2607_17299_b200 import binding as war
    from paper_2607_17299_b200 import replica
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    try:
        wl = Workload(war, W, cfg, dev, args)
    except MemoryError as e:
        raise SystemExit(f"bench.py: {e}")
    B = cfg.B
    launches = "one launch" if (B <= FUSED_MAX_B and args.kernel == 0) else "plan + attention + combine launches"
    if args.kernel == 1:
        launches = "plan + CUDA-core attention + combine launches"

    clocks = ClockSampler(local_rank)
    clocks.__enter__()
    torch.cuda.synchronize()
    time.sleep(2.0)                                        # the set-up (index build, gigabytes of K/V filled) leaves the board at its
    # power cap: let it recover before the warm-up steps
    t = wl.time_steps(args.steps, args.warmup, barrier, flush_l2=args.flush_l2, cuda_graph=args.cuda_graph, clocks=clocks)
    time.sleep(0.06)                                       # let the sampler see the end of the timed region
    last_sample = clocks.mark()
    status = war.war_device_status()
    verified, slots, accept_len_mean = wl.counts()
    gpu_res = wl.gpu_results() if rank == 0 and not args.no_cpu_baseline and world == 1 else None

    e2e_ms, h2d, d2h = wl.time_e2e(args.steps, barrier)

    # ---- the method's one exchange (end of an RL step): every rank contributes its share of n_traj/32 finished
    # trajectories, all-gathered on the device into each rank's own memory, then the same append on every rank (a
    # sliding window keeps the stored count, so the index stays within its capacity) ----
    # (three rounds, the median reported: the eviction and the append allocate and free their scratch through the
    # driver, and a single round now and then takes ten times as long on the host.  Every round brings back exactly the
    # trajectories that its eviction drops, the oldest ones: after the set-up above the index holds the trajectories in
    # the order 2k .. n-1, 0 .. 2k-1 with k = n_traj/32, so the stored set never changes.)
    k_new = max(world, cfg.n_traj // 32)
    k_setup = max(1, cfg.n_traj // 32)
    share = replica.shard_requests(k_new, rank, world)
    rounds = []
    for rnd in range(3):
        first = 2 * k_setup + rnd * k_new + share.start
        last = first + (share.stop - share.start)
        new_off = wl.off[first:last + 1] - wl.off[first]
        new_tok = torch.from_numpy(wl.tok[wl.off[first]:wl.off[last]]).to(dev)
        barrier()
        x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        x0.record()
        g_tok, g_off = replica.gather_trajectories(new_tok, new_off, dev)
        x1.record()
        torch.cuda.synchronize()
        t1 = time.perf_counter()
        replica_window = cfg.n_traj
        war.war_index_evict(wl.ix, replica.window_eviction(int(war.war_index_info(wl.ix).T), len(g_off) - 1, replica_window))
        t2 = time.perf_counter()
        war.war_index_append(wl.ix, g_tok, g_off)
        torch.cuda.synchronize()
        t3 = time.perf_counter()
        rounds.append((1e3 * (t3 - t0), x0.elapsed_time(x1), 1e3 * (t1 - t0), 1e3 * (t2 - t1), 1e3 * (t3 - t2)))
    rounds.sort()
    exchange_ms, gather_ms = rounds[1][0], rounds[1][1]
    exchange_parts = {"gather_host_ms": rounds[1][2], "evict_ms": rounds[1][3], "append_ms": rounds[1][4],
                      "rounds_ms": [round(r[0], 3) for r in rounds]}

    # ---- the checker on the first requests, timed on the host cores; what it computes is compared with what the GPU
    # produced for the same requests (before anything below moves K/V rows or changes the index) ----
    cpu_baseline = None
    if gpu_res is not None:
        from oracle import draft_oracle
        corpus = draft_oracle.Corpus(wl.tok, wl.off)
        targets = wl.targets
        v, secs, done, results = oracle_sample(cfg, corpus, wl.tails, wl.tl, wl.attn, wl.ctx, lambda i, ids, par, n: targets[i],
                                               list(range(cfg.B)), budget_s=15.0, keep=True)
        bad = parity_against(results, gpu_res, cfg.N)
        cpu_baseline = {"cpu_baseline": {"value": v / secs, "unit": UNIT, "cores": threads_in_use(), "kind": "oracle",
                                         "sample": f"first {done} of {cfg.B} requests, {secs:.1f} s"},
                        "parity_checked": done, "parity_ok": not bad}
        if bad:
            print(json.dumps(cpu_baseline))
            raise SystemExit(f"bench.py: the GPU results differ from the CPU checker: {bad[:8]}")
        del results

    advancing = wl.time_advancing(args.steps, args.warmup) if (extras or args.advance) else None
    commit_ms = wl.time_commit()

    # ---- max over ranks, totals over ranks ----
    total_ms, attn_ms = t["total_ms"], t["attn_ms"]
    agg = torch.tensor([total_ms, e2e_ms, attn_ms, exchange_ms, gather_ms], dtype=torch.float64, device=dev)
    tot = torch.tensor([verified, slots], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(agg, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    total_ms, e2e_ms, attn_ms, exchange_ms, gather_ms = [float(x) for x in agg.tolist()]
    verified_all, slots_all = [float(x) for x in tot.tolist()]
    ms_per_step = total_ms / args.steps

    line = None
    if rank == 0:
        roof, roof_kernel = roofline_of(cfg, wl.ctx, wl.h_nn, attn_ms, launches)
        per_step = t["per_step"]
        line = {
            "metric": METRIC, "value": verified_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(base_config, kernel={0: "tcgen05", 1: "cuda-core", 2: "tcgen05, three launches"}[args.kernel],
                           **({"spec_batch_limit": args.spec_batch_limit} if args.spec_batch_limit else {}),
                           **({"score_lengths": args.score_lengths} if args.score_lengths > 1 else {}),
                           **({"own_context": True, "own_context_share": float(wl.d_src.float().mean().item())}
                              if args.own_context else {}),
                           **({"launch": "one CUDA graph per step", "eager_ms_per_step": t["eager_ms"] / args.steps}
                              if args.cuda_graph else {})),
            "clocks": clocks.summary(t["first_sample"], last_sample),
            "e2e": {"value": verified_all / (e2e_ms / args.steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps},
            "gpu_launches": launches_per_step(B, args.kernel, args.score_lengths, args.own_context) * args.steps,
            "roofline": roof, "roofline_kernel": roof_kernel,
            "breakdown_ms": {"draft": t["draft_ms"], "verify_attn": attn_ms, "accept": t["accept_ms"]},
            "commit_ms": commit_ms,
            "draft_cold_ms": wl.draft_cold_ms,
            "step_ms": {"median": float(np.median(per_step)), "min": float(per_step.min()), "max": float(per_step.max())},
            "slots_verified_per_s": slots_all / (ms_per_step * 1e-3),
            "accept_len_mean": accept_len_mean,
            "exchange_ms": exchange_ms,
            "exchange": {"trajectories": k_new, "tokens": int(g_off[-1]), "all_gather_ms": gather_ms, **exchange_parts,
                         "what": "all-gather of the step's finished trajectories (device to device) + window eviction + "
                                 "war_index_append on every rank"},
            "device_status": status,
        }
        line.update(wl.index_stats)
        if advancing is not None:
            line["advancing"] = advancing
            line["value_advancing"] = advancing["verified_last_step"] / (advancing["ms_per_step"] * 1e-3)
        if cpu_baseline is not None:
            line.update(cpu_baseline)

    # ---- the other configurations, the load sweep: a few steps each (rank 0 of a single-GPU run only) ----
    if extras and rank == 0:
        ix_high, corpus_high = wl.ix, (wl.tok, wl.off)
        wl.owns_index = False
        wl.close()
        sweep = {}
        try:
            sw = Workload(war, W, W.scaled(W.CONFIGS["high"], B=64), dev, args, ix=ix_high, corpus=corpus_high)
            for r in (4, 8, 16, 32, 64):
                sw._buffers(r)
                n_steps = sw.steps_for(0.2, 20)
                tt = sw.time_steps(n_steps, args.warmup, barrier)
                sweep[str(r)] = summarize(sw, tt, n_steps, "one launch" if r <= FUSED_MAX_B else "three launches")
                sweep[str(r)]["steps"] = n_steps
            sw.close()
        except MemoryError as e:
            sweep = {"skipped": str(e)}
        ix_high.destroy()
        line["load_sweep"] = sweep
        table, table_wl = {}, None
        for name, n_steps, flush in (("tiny", 50, False), ("tiny", 50, True), ("low", 20, False), ("longtail", 20, False), ("wide", 5, False)):
            key = name + ("_l2_flushed" if flush else "")
            if flush and table_wl is None:
                continue
            try:
                w2 = table_wl if flush else Workload(war, W, W.CONFIGS[name], dev, args)
            except MemoryError as e:
                table[key] = {"skipped": str(e)}
                continue
            n_steps = w2.steps_for(0.3, n_steps)                   # long enough for the clock sampler to see it
            torch.cuda.synchronize()
            time.sleep(2.0)                                        # the set-up above (filling gigabytes of K/V) and the workloads
            mark0 = clocks.mark()                                  # before it leave the board at its power cap: let it recover
            tt = w2.time_steps(n_steps, args.warmup, barrier, flush_l2=flush)
            entry = summarize(w2, tt, n_steps, "one launch" if w2.B <= FUSED_MAX_B else "three launches")
            entry["config"] = describe(W.CONFIGS[name], flush)
            entry["steps"] = n_steps
            entry["clocks"] = clocks.summary(mark0, clocks.mark())
            if not flush:
                e_ms, _, _ = w2.time_e2e(n_steps, barrier)
                entry["e2e_ms_per_step"] = e_ms / n_steps
            entry["device_status"] = war.war_device_status()
            table[key] = entry
            if name == "tiny" and not flush:
                table_wl = w2                                      # the flushed pass reuses it
            else:
                w2.close()
        line["workloads"] = table
    else:
        wl.close()
    clocks.__exit__(None, None, None)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
