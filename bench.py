#!/usr/bin/env python
"""Benchmark of the speculate-and-verify step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload high|low|longtail|wide|tiny] [--impl ours|reference]

A step = one pass of the whole hot path over one batch of live requests: war_draft (suffix match + draft trees)
-> war_verify_attn (tree-masked GQA attention over the paged bf16 KV cache) -> war_accept.  The index build is
set-up and is reported separately.  The metric is verified tokens per second: sum over requests of
(accepted draft tokens + the one token the target model always yields) divided by the step time.

One JSON line is printed by rank 0.  `value` has every input resident in HBM; `e2e` repeats the step with the
per-step inputs starting in pinned host memory and the results read back, copies inside the timed region;
`roofline` puts the verify-attention call against the measured HBM copy bandwidth; `cpu_baseline` times the CPU
checker (oracle/) on a bounded sample of the same requests on this machine's host cores.

`--impl reference` times that CPU checker alone (there is no other reference implementation to run).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verified tokens/s per speculate+verify step"
UNIT = "tokens/s"
LAUNCHES_PER_STEP = 5          # draft, attention plan, attention, split-KV combine, accept


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

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(cfg, corpus, tails, tail_len, attn, ctx, targets_fn, requests, budget_s=None):
    """Runs the CPU checker on the given requests (in order, stopping once budget_s is spent, at least one).
    Returns (tokens verified, seconds, requests done)."""
    from oracle import accept_oracle, attention_oracle, draft_oracle
    import torch
    scale = 1.0 / float(np.sqrt(cfg.D))
    t0 = time.perf_counter()
    verified, done = 0, 0
    pt = attn.page_table.cpu().numpy() if attn is not None else None
    for i in requests:
        ml, ends = draft_oracle.longest_suffix_match(corpus, tails[i], int(tail_len[i]))
        ids, parent, count = draft_oracle.build_draft_tree(corpus, tails[i], ml, ends, cfg.N, cfg.topk)
        n = len(ids)
        full_ids = np.full((1, cfg.N), -1, np.int32); full_par = np.full((1, cfg.N), -1, np.int32)
        full_ids[0, :n] = ids; full_par[0, :n] = parent
        K, V = attention_oracle.gather_request_kv(attn.k_pool, attn.v_pool, pt[i], int(ctx[i]) - 1 + n)
        q = attn.q[i].to("cpu").to(torch.float64).numpy()
        attention_oracle.verify_attention_request(q, K, V, int(ctx[i]) - 1, full_par[0], n, scale)
        target = targets_fn(i, full_ids, full_par, n)
        alen, _, _ = accept_oracle.accept_request(full_ids[0], full_par[0], n, target, 0)
        verified += alen + 1
        done += 1
        if budget_s is not None and time.perf_counter() - t0 > budget_s:
            break
    return verified, time.perf_counter() - t0, done


def threads_in_use() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        n = 1
    return int(min(n, len(os.sched_getaffinity(0))))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="high")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", type=int, default=0, help="0 = tensor-core verify attention, 1 = plain CUDA-core kernel")
    ap.add_argument("--no-cpu-baseline", action="store_true")
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
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    import torch
    from paper_2607_17299_b200 import workloads as W
    cfg = W.CONFIGS[args.workload]
    if args.requests > 0:
        cfg = W.scaled(cfg, B=args.requests)
    base_config = {"workload": f"{cfg.name}: corpus {cfg.n_traj} trajectories, {cfg.B} requests, tree <= {cfg.N} slots, "
                               f"{cfg.Hq}q/{cfg.Hkv}kv heads, d={cfg.D}, page {cfg.page_size}",
                   "requests_per_gpu": cfg.B, "parallelism": f"replica x{world}" if world > 1 else "single gpu",
                   "l2": "inputs (KV cache) far larger than L2, no flush needed" if cfg.name != "tiny" else
                         ("L2 flushed (256 MB written) before every step" if args.flush_l2 else
                          "KV cache fits L2: value is an L2-resident number (--flush-l2 gives the cold one)")}

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
            v, dt, _ = oracle_sample(cfg, corpus, tails, tl, attn, ctx, targets_fn, reqs)
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
    import torch.distributed as dist
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- set-up: corpus, index, requests, KV cache (all seeded, synthetic) ----
    tok, off = W.make_corpus(cfg)
    tails, tl = W.make_request_tails(cfg)
    make_tails = (tails, tl)
    ctx = W.context_lengths(cfg)
    # the GPUs are shared: make sure the workload fits in what is free before allocating anything large
    need = (int(((ctx - 1 + cfg.N + cfg.page_size - 1) // cfg.page_size).sum()) * cfg.Hkv * cfg.page_size * cfg.D * 2 * 2   # K and V pools
            + (len(tok) + cfg.n_traj) * (14 + 44)                                                                        # index + build scratch
            + 3 * cfg.B * cfg.N * cfg.Hq * cfg.D * 2 + (1 << 30))                                                        # q, out, workspace, slack
    free, _total = torch.cuda.mem_get_info(dev)
    if free < need:
        raise SystemExit(f"bench.py: workload {cfg.name} needs about {need / 2**30:.1f} GiB of device memory, "
                         f"{free / 2**30:.1f} GiB are free on cuda:{local_rank}")
    d_tok = torch.from_numpy(tok).to(dev)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ix = war.war_index_build(d_tok, off, cfg.vocab, cfg.P + cfg.N, len(tok) + cfg.n_traj)
    index_build_s = time.perf_counter() - t0
    # the index the steps use is then made the way a rollout would make it: all but the last trajectories first, the
    # rest appended as an RL step's worth of new trajectories (an appended index answers exactly like a fresh build)
    k_new = max(1, cfg.n_traj // 32)
    # one draft call on this first index, so that the first call on the index the steps use (below) measures an empty
    # memo and not the one-time cost of the first launch of a kernel
    _t, _tl = torch.from_numpy(make_tails[0]).to(dev), torch.from_numpy(make_tails[1]).to(dev)
    _z = lambda *sh: torch.zeros(sh, dtype=torch.int32, device=dev)
    war.war_draft(ix, _t, _tl, cfg.N, cfg.topk, 1, _z(cfg.B), _z(cfg.B), _z(cfg.B, cfg.N), _z(cfg.B, cfg.N), None)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    war.war_index_evict(ix, k_new)                         # sliding window: the oldest 1/32 of the trajectories leave
    index_evict_s = time.perf_counter() - t0
    ix.destroy()
    ix = war.war_index_build(d_tok, off[:cfg.n_traj - k_new + 1], cfg.vocab, cfg.P + cfg.N, len(tok) + cfg.n_traj)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    war.war_index_append(ix, d_tok, off[cfg.n_traj - k_new:])
    index_append_s = time.perf_counter() - t0
    index_append_tokens = int(off[-1] - off[cfg.n_traj - k_new])
    del d_tok
    attn = W.make_attention_inputs(cfg, ctx, device=dev)
    B, N = cfg.B, cfg.N
    i32 = dict(dtype=torch.int32, device=dev)
    # the step's small integer inputs (tails, their lengths, the target model's tokens) share one allocation as well
    P_ = tails.shape[1]
    d_in = torch.zeros(B * (P_ + 1 + N), **i32)
    d_tails, d_tl, d_target = d_in[:B * P_].view(B, P_), d_in[B * P_:B * (P_ + 1)], d_in[B * (P_ + 1):].view(B, N)
    d_tails.copy_(torch.from_numpy(tails)); d_tl.copy_(torch.from_numpy(tl))
    # the step's small integer results live side by side in one allocation, so the end-to-end leg reads them back with one copy
    d_small = torch.zeros(B * (3 + 3 * N), **i32)
    d_nn, d_alen, d_bonus = d_small[0:B], d_small[B:2 * B], d_small[2 * B:3 * B]
    d_ids, d_par, d_path = (d_small[3 * B + k * B * N:3 * B + (k + 1) * B * N].view(B, N) for k in range(3))
    d_ml, d_cnt = torch.zeros(B, **i32), torch.zeros((B, N), **i32)
    d_out = torch.zeros_like(attn.q)
    d_lse = torch.zeros(attn.q.shape[:3], dtype=torch.float32, device=dev)
    scale = 1.0 / float(np.sqrt(cfg.D))
    params = war.attn_params(attn.q, attn.k_pool, attn.v_pool, attn.page_table, scale, args.kernel)
    ws = war.new_workspace(params, dev)

    # targets depend on the trees; the trees are a deterministic function of the inputs, so draft once to make them
    # (this is also the first draft call on the freshly published index: its memo of large-node expansions is empty)
    if args.score_lengths > 1:
        d_used = torch.zeros(cfg.B, dtype=torch.int32, device=dev)
        draft_ws = torch.empty(war.war_draft_scored_workspace_bytes(cfg.B, cfg.P, N, cfg.topk, args.score_lengths),
                               dtype=torch.uint8, device=dev)

    if args.own_context:
        h_ctx, h_ctx_off = W.make_request_contexts(cfg, ctx)
        d_ctx, d_ctx_off = torch.from_numpy(h_ctx).to(dev), torch.from_numpy(h_ctx_off).to(dev)
        i32 = dict(dtype=torch.int32, device=dev)
        g_tree = [torch.zeros(cfg.B, **i32), torch.zeros(cfg.B, **i32)] + [torch.zeros((cfg.B, N), **i32) for _ in range(3)]
        l_tree = [torch.zeros(cfg.B, **i32), torch.zeros(cfg.B, **i32)] + [torch.zeros((cfg.B, N), **i32) for _ in range(3)]
        d_src = torch.zeros(cfg.B, **i32)
        local_stream = torch.cuda.Stream()
        local_done = torch.cuda.Event()

    def draft():
        if args.own_context:
            # the two drafts share no data: the own-context scan runs beside the index lookup, then the better tree is kept
            main = torch.cuda.current_stream()
            local_stream.wait_stream(main)
            with torch.cuda.stream(local_stream):
                war.war_draft_local(d_ctx, d_ctx_off, d_tl, cfg.P, N, cfg.topk, 1, *l_tree, args.spec_batch_limit)
                local_done.record(local_stream)
            war.war_draft(ix, d_tails, d_tl, N, cfg.topk, 1, *g_tree, args.spec_batch_limit)
            main.wait_event(local_done)
            war.war_draft_pick(g_tree, l_tree, d_src, d_ml, d_nn, d_ids, d_par, d_cnt)
        elif args.score_lengths > 1:
            war.war_draft_scored(ix, d_tails, d_tl, N, cfg.topk, 1, args.score_lengths, draft_ws, d_ml, d_used, d_nn, d_ids,
                                 d_par, d_cnt, args.spec_batch_limit)
        else:
            war.war_draft(ix, d_tails, d_tl, N, cfg.topk, 1, d_ml, d_nn, d_ids, d_par, d_cnt, args.spec_batch_limit)

    ev = lambda: torch.cuda.Event(enable_timing=True)
    cold0, cold1 = ev(), ev()
    torch.cuda.synchronize()
    cold0.record()
    draft()
    cold1.record()
    torch.cuda.synchronize()
    draft_cold_ms = cold0.elapsed_time(cold1)
    h_ids, h_par, h_nn = d_ids.cpu().numpy(), d_par.cpu().numpy(), d_nn.cpu().numpy()
    targets = W.make_targets(cfg, h_ids, h_par, h_nn, 0)
    d_target.copy_(torch.from_numpy(targets))

    def step(attn_events=None):
        draft()
        if attn_events is not None:
            attn_events[0].record()
        war.war_verify_attn(attn.q, attn.k_pool, attn.v_pool, attn.page_table, attn.prefix_len, d_nn, d_par, params, ws,
                            d_out, d_lse)
        if attn_events is not None:
            attn_events[1].record()
        war.war_accept(d_ids, d_par, d_nn, d_target, 0, d_alen, d_path, d_bonus)

    # nvidia-smi needs a few hundred ms to start reporting, so the sampler runs from the warm-up through the timed
    # region (and is given a moment to produce its first lines while the GPU is already under load)
    clocks = ClockSampler(local_rank)
    clocks.__enter__()
    t_warm = time.perf_counter()
    for _ in range(args.warmup):
        step()
    while time.perf_counter() - t_warm < 0.6 and not clocks.rows:
        step()
        torch.cuda.synchronize()
    barrier()
    attn_ev = [(ev(), ev()) for _ in range(args.steps)]
    step_ev = [(ev(), ev()) for _ in range(args.steps)]
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if args.flush_l2 else None
    barrier()
    start, stop = ev(), ev()
    graph_ms = None
    if args.cuda_graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        for _ in range(args.warmup):
            graph.replay()
        barrier()
        start.record()
        for s in range(args.steps):
            graph.replay()
        stop.record()
        barrier()
        graph_ms = start.elapsed_time(stop)
        start, stop = ev(), ev()
    start.record()
    for s in range(args.steps):
        if scratch is not None:
            scratch.fill_(s & 0xFF)
        step_ev[s][0].record()
        step(attn_ev[s])
        step_ev[s][1].record()
    stop.record()
    barrier()
    per_step = np.array([a.elapsed_time(b) for a, b in step_ev])
    total_ms = float(per_step.sum()) if args.flush_l2 else start.elapsed_time(stop)
    eager_ms = total_ms
    if graph_ms is not None:
        total_ms = graph_ms
    time.sleep(0.06)                                       # let the sampler see the end of the timed region
    clocks.__exit__(None, None, None)
    attn_ms = float(np.mean([a.elapsed_time(b) for a, b in attn_ev]))
    draft_ms = float(np.mean([step_ev[s][0].elapsed_time(attn_ev[s][0]) for s in range(args.steps)]))
    accept_ms = float(np.mean([attn_ev[s][1].elapsed_time(step_ev[s][1]) for s in range(args.steps)]))
    status = war.war_device_status()
    h_alen = d_alen.cpu().numpy()
    verified = int((h_alen.astype(np.int64) + 1).sum())
    slots = int(h_nn.sum())

    # ---- end to end: per-step inputs start in pinned host memory, results are read back ----
    pin = lambda t: t.cpu().pin_memory()
    overlap_out_ok = d_out.numel() * d_out.element_size() >= (4 << 20)   # small outputs: one stream, one buffer
    h_q, h_in = pin(attn.q), pin(d_in)
    r_small, r_out = pin(d_small), pin(d_out)                 # trees, accepted paths and bonus tokens; attention output
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
        d_in.copy_(h_in, non_blocking=True)
        if overlap_q:
            copy_stream.wait_stream(main_stream)            # the previous step's readers of q are done
            with torch.cuda.stream(copy_stream):
                attn.q.copy_(h_q, non_blocking=True)
                q_ready.record(copy_stream)
        else:
            attn.q.copy_(h_q, non_blocking=True)
        draft()
        if overlap_q:
            main_stream.wait_event(q_ready)
        if overlap_out_ok and s >= 2:
            main_stream.wait_event(out_copied[s & 1])       # this output buffer's previous copy has left the device
        war.war_verify_attn(attn.q, attn.k_pool, attn.v_pool, attn.page_table, attn.prefix_len, d_nn, d_par, params, ws,
                            o, d_lse)
        if overlap_out_ok:
            attn_done.record(main_stream)
            with torch.cuda.stream(out_stream):
                out_stream.wait_event(attn_done)
                r_o.copy_(o, non_blocking=True)
                out_copied[s & 1].record(out_stream)
        war.war_accept(d_ids, d_par, d_nn, d_target, 0, d_alen, d_path, d_bonus)
        r_small.copy_(d_small, non_blocking=True)
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
    for s in range(args.steps):
        e2e_step(2 + s)
    barrier()
    e2e_ms = 1e3 * (time.perf_counter() - t0)

    # ---- commit (the accepted tokens become context), timed on its own: it is what a caller runs between two
    # steps, not part of the step metric.  Run last: it moves K/V rows of the resident cache.
    c_pl, c_tails, c_tl = attn.prefix_len.clone(), d_tails.clone(), d_tl.clone()
    war.war_commit(d_ids, d_alen, d_path, d_bonus, attn.k_pool, attn.v_pool, attn.page_table, c_pl, c_tails, c_tl)
    c_pl.copy_(attn.prefix_len); c_tails.copy_(d_tails); c_tl.copy_(d_tl)
    c0, c1 = ev(), ev()
    torch.cuda.synchronize()
    c0.record()
    war.war_commit(d_ids, d_alen, d_path, d_bonus, attn.k_pool, attn.v_pool, attn.page_table, c_pl, c_tails, c_tl)
    c1.record()
    torch.cuda.synchronize()
    commit_ms = c0.elapsed_time(c1)

    # ---- max over ranks, totals over ranks ----
    agg = torch.tensor([total_ms, e2e_ms, attn_ms], dtype=torch.float64, device=dev)
    tot = torch.tensor([verified, slots], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(agg, op=dist.ReduceOp.MAX)
        dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    total_ms, e2e_ms, attn_ms = [float(x) for x in agg.tolist()]
    verified_all, slots_all = [float(x) for x in tot.tolist()]
    ms_per_step = total_ms / args.steps

    if rank == 0:
        peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
        if os.path.exists(peaks_path):
            with open(peaks_path) as f:
                peak, peak_src = float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, copy)"
        else:
            peak, peak_src = 6650.0, "fallback"
        kvb = kv_bytes(cfg, ctx - 1, h_nn)
        achieved = kvb / (attn_ms * 1e-3) / 1e9
        # the same launch seen from the tensor pipe: 4 * rows * D flops per KV token and kv head (QK^T and PV), rows = the
        # (slot, head-of-group) pairs that exist (not the padded MMA tile)
        G = cfg.Hq // cfg.Hkv
        live = h_nn > 0
        flops = float(((ctx - 1 + h_nn)[live].astype(np.float64) * (4.0 * G * h_nn[live] * cfg.D)).sum() * cfg.Hkv)
        peak_tf = None
        if os.path.exists(peaks_path):
            with open(peaks_path) as f:
                peak_tf = float(json.load(f).get("bf16_tflops_sustained", 0.0)) or None
        peak_tf = peak_tf or 1400.0
        t_hbm, t_tensor = kvb / (peak * 1e9), flops / (peak_tf * 1e12)
        tensor_bound = t_tensor > t_hbm
        # DRAM bytes per launch of the attention kernel from the committed ncu summary of this workload, if there is one
        traffic = None
        traffic_path = os.path.join(ROOT, "profiles", f"attn_sm100_kernel_{cfg.name}_traffic.md")
        if os.path.exists(traffic_path) and args.requests == 0:
            import re
            with open(traffic_path) as f:
                m = re.search(r"^dram_bytes_per_launch\s*=\s*(\d+)", f.read(), flags=re.M)
            traffic = int(m.group(1)) if m else None
        line = {
            "metric": METRIC, "value": verified_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(base_config, kernel="tcgen05" if args.kernel == 0 else "cuda-core",
                           **({"spec_batch_limit": args.spec_batch_limit} if args.spec_batch_limit else {}),
                           **({"score_lengths": args.score_lengths} if args.score_lengths > 1 else {}),
                           **({"own_context": True, "own_context_share": float(d_src.float().mean().item())}
                              if args.own_context else {}),
                           **({"launch": "one CUDA graph per step", "eager_ms_per_step": eager_ms / args.steps}
                              if args.cuda_graph else {})),
            "clocks": clocks.summary(),
            "e2e": {"value": verified_all / (e2e_ms / args.steps * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps},
            "gpu_launches": (LAUNCHES_PER_STEP + (args.score_lengths > 1) + 2 * args.own_context) * args.steps,
            "roofline": ({"bound": "tensor", "achieved": flops / (attn_ms * 1e-3) / 1e12, "peak": peak_tf, "unit": "TFLOP/s",
                          "frac": t_tensor / (attn_ms * 1e-3), "traffic": traffic, "flops_per_launch": flops,
                          "peak_source": "measured (MEASURED_PEAKS.json bf16_tflops_sustained)" if os.path.exists(peaks_path) else "fallback",
                          "hbm_gbs": achieved} if tensor_bound else
                         {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                          "traffic": traffic, "frac_of_8TBps_nominal": achieved / 8000.0, "peak_source": peak_src,
                          "tensor_tflops": flops / (attn_ms * 1e-3) / 1e12}),
            "roofline_kernel": {"name": "war_verify_attn (plan + attention + combine launches)", "bytes_per_launch": kvb,
                                "ms_per_launch": attn_ms},
            "breakdown_ms": {"draft": draft_ms, "verify_attn": attn_ms, "accept": accept_ms},
            "commit_ms": commit_ms,
            "draft_cold_ms": draft_cold_ms,
            "step_ms": {"median": float(np.median(per_step)), "min": float(per_step.min()), "max": float(per_step.max())},
            "slots_verified_per_s": slots_all / (ms_per_step * 1e-3),
            "accept_len_mean": float(h_alen.mean()), "index_build_s": index_build_s, "index_tokens": int(len(tok)),
            "index_append": {"trajectories": k_new, "tokens": index_append_tokens, "seconds": index_append_s},
            "index_evict": {"trajectories": k_new, "seconds": index_evict_s},
            "device_status": status,
        }
        if not args.no_cpu_baseline and world == 1:
            from oracle import draft_oracle
            corpus = draft_oracle.Corpus(tok, off)
            def targets_fn(i, ids, par, n):
                return targets[i]
            v, secs, done = oracle_sample(cfg, corpus, tails, tl, attn, ctx, targets_fn, list(range(cfg.B)), budget_s=15.0)
            line["cpu_baseline"] = {"value": v / secs, "unit": UNIT, "cores": threads_in_use(), "kind": "oracle",
                                    "sample": f"first {done} of {cfg.B} requests, {secs:.1f} s"}
        print(json.dumps(line))
    ix.destroy()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
