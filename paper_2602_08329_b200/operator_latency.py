"""Attention-operator latency of the library on the shapes of the paper's efficiency study.

    python -m paper_2602_08329_b200.operator_latency            # Table-3 shapes
    python -m paper_2602_08329_b200.operator_latency --graph    # the same, blocks of s steps replayed from CUDA graphs
    python -m paper_2602_08329_b200.operator_latency --configs  # the benchmark's C2..C5 shapes
    python -m paper_2602_08329_b200.operator_latency --configs --group-sets   # one set per KV head (variant)
    python -m paper_2602_08329_b200.operator_latency --configs --summary  # JSON: time, bytes, roofline per layer-step
    python -m paper_2602_08329_b200.operator_latency --gated              # cosine-gated schedule vs fixed at equal rho-hat

The paper (Sec. 5.4, Table 3) times one attention layer of LLaMA-2-7B-Chat (32 MHA heads,
head_dim 128) in decode at batch 8 / 16 and 1k-4k cached tokens, token sparsity 1/8, block
size s = 8 / 16, against a dense FlashAttention-2 call, on an A100.  This script times the same
shapes here: the in-library dense flash-decode kernel, a sharing step, a retrieval step, and the
amortised per-step latency for s = 8 and 16.  Budgets follow Sec. 5.3.2 scaled to the length
(C_sink 16, C_local 64, k = N/8 - 80).  Data are synthetic (`workloads.py`).

Each figure is the median of per-step CUDA-event times over independent cache copies visited
round-robin (so that no step finds its rows in L2).  Prints a markdown table.
"""
from __future__ import annotations

import argparse
import statistics

import torch

from . import binding as P
from . import workloads as W

PAPER_TABLE3_MS = {  # (batch, seqlen): (Flash, CPE-8, CPE-16) in ms on an A100 (Table 3)
    (8, 1024): (0.230, 0.092, 0.078), (8, 2048): (0.830, 0.144, 0.095), (8, 4096): (1.630, 0.506, 0.469),
    (16, 1024): (0.440, 0.089, 0.075), (16, 2048): (1.630, 0.196, 0.165), (16, 4096): (3.230, 0.904, 0.821),
}


def table3_workload(batch: int, n: int, s: int = 8) -> W.Workload:
    """The Table-3 shape (batch, n cached tokens) with the budgets of Sec. 5.3.2 scaled to the
    length: C_sink 16, C_local 64, k = n/8 - 80 (432 at 4k); one MHA layer of 32 heads."""
    return W.Workload(f"table3_b{batch}_{n}", layers=1, batch=batch, q_heads=32, kv_heads=32, context=n,
                      steps=4, top_k=n // 8 - 80, window=64, sinks=16, refresh=s, heavy_hitters=16,
                      decay_span=min(512, n // 8), seed=100 + batch + n)


def time_workload(w: W.Workload, dev, copies: int = 4, reps: int = 6, group_sets: bool = False):
    """Median device time (us) of a dense step, a retrieval step and a sharing step."""
    w = w.scaled(layers=copies, steps=max(w.refresh, 2) + 1)
    table = None
    if w.page_size:
        table, pool = W.make_page_table(w)
        kv = []
        for _, k, v in W.make_layer_kv(w, dev):       # page one copy at a time to bound memory
            kv.append((W.to_paged(w, k, table, pool), W.to_paged(w, v, table, pool)))
            del k, v
        table = table.to(dev)
    else:
        kv = [(k, v) for _, k, v in W.make_layer_kv(w, dev)]
    q = W.make_queries(w, dev)
    B, Hq = w.batch, w.q_heads
    kps = W.top_k_per_seq(w)
    max_k = max(w.top_k, int(w.k_frac * w.context))
    ctx = P.Context(copies, B, Hq, w.kv_heads, w.capacity, max_k, w.window, w.sinks, max_dilate_r=w.dilate_r,
                    page_size=w.page_size, flags=CTX_FLAGS)
    sched = P.make_schedule(w.top_k, w.window, w.sinks, refresh_interval=w.refresh, dilate_r=w.dilate_r,
                            top_k_per_seq=None if kps is None else kps.to(dev),
                            flags=P.PRHS_GROUP_SETS if group_sets else 0)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    t0, t1 = W.seq_lens_at(w, 0).to(dev), W.seq_lens_at(w, 1).to(dev)
    views0 = [P.make_view(kv[l][0], kv[l][1], t0, page_table=table, max_seq_len=w.capacity) for l in range(copies)]
    views1 = [P.make_view(kv[l][0], kv[l][1], t1, page_table=table, max_seq_len=w.capacity) for l in range(copies)]
    stream = torch.cuda.current_stream()

    def timed(fn):
        ts = []
        for r in range(reps):
            evs = []
            for l in range(copies):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                fn(l)
                b.record(stream)
                evs.append((a, b))
            torch.cuda.synchronize()
            if r > 0:
                ts += [a.elapsed_time(b) * 1e3 for a, b in evs]
        return statistics.median(ts)

    dense = timed(lambda l: ctx.dense_decode_attn(q[l, 0], views0[l], B, out))
    refresh = timed(lambda l: ctx.decode_step(l, 0, sched, q[l, 0], views0[l], B, out))
    shared = timed(lambda l: ctx.decode_step(l, 1, sched, q[l, 1], views1[l], B, out))
    idx, cnt = ctx.get_index_set(B)
    # Per-kernel times of a retrieval step: event pairs recorded inside the library.
    ctx.profile_begin()
    for _ in range(2):
        for l in range(copies):
            ctx.decode_step(l, 0, sched, q[l, 0], views0[l], B, out)
    kern = {name: ms * 1e3 / n for name, (ms, n) in ctx.profile_end().items() if n}
    ctx.close()
    # Bytes a sharing step must move: every listed row once per query head (logical), and once
    # per KV head for the union over the heads of a group (unique).
    G = Hq // w.kv_heads
    cap = idx.shape[-1]
    valid = torch.arange(cap, device=idx.device)[None, None, :] < cnt[:, :, None]
    logical = int(cnt.sum()) * 512
    mark = torch.zeros(B * w.kv_heads, w.capacity + 1, dtype=torch.bool, device=idx.device)
    unit = (torch.arange(B, device=idx.device)[:, None] * w.kv_heads
            + torch.arange(Hq, device=idx.device)[None, :] // G)[:, :, None].expand_as(idx)
    mark[unit[valid].long(), idx[valid].long()] = True
    unique = int(mark.sum()) * 512
    key_bytes = int(t0.sum()) * w.kv_heads * 256
    return {"dense_us": dense, "refresh_us": refresh, "shared_us": shared,
            "set_size": float(cnt.float().mean()), "kernels": kern, "logical_bytes": logical,
            "unique_bytes": unique, "key_bytes": key_bytes}


def time_blocks(w: W.Workload, dev, s: int, copies: int = 4, reps: int = 6, group_sets: bool = False):
    """Per-step device time (us) of a whole block of s decode steps (one retrieval, s - 1 sharing
    steps) and of s dense steps, each block replayed from a CUDA graph: what a decode loop pays
    once the per-launch host work is out of the way.  Blocks of independent cache copies are
    replayed in turn."""
    w = w.scaled(layers=copies, steps=s)
    table = None
    if w.page_size:
        table, pool = W.make_page_table(w)
        kv = []
        for _, k, v in W.make_layer_kv(w, dev):       # page one copy at a time to bound memory
            kv.append((W.to_paged(w, k, table, pool), W.to_paged(w, v, table, pool)))
            del k, v
        table = table.to(dev)
    else:
        kv = [(k, v) for _, k, v in W.make_layer_kv(w, dev)]
    q = W.make_queries(w, dev)
    B, Hq = w.batch, w.q_heads
    kps = W.top_k_per_seq(w)
    max_k = max(w.top_k, int(w.k_frac * w.context))
    ctx = P.Context(copies, B, Hq, w.kv_heads, w.capacity, max_k, w.window, w.sinks, max_dilate_r=w.dilate_r,
                    page_size=w.page_size, flags=CTX_FLAGS)
    sched = P.make_schedule(w.top_k, w.window, w.sinks, refresh_interval=s, dilate_r=w.dilate_r,
                            top_k_per_seq=None if kps is None else kps.to(dev),
                            flags=P.PRHS_GROUP_SETS if group_sets else 0)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    lens = [W.seq_lens_at(w, n).to(dev) for n in range(s)]
    views = [[P.make_view(kv[l][0], kv[l][1], lens[n], page_table=table, max_seq_len=w.capacity) for n in range(s)]
             for l in range(copies)]
    side = torch.cuda.Stream()
    graphs = {"sparse": [], "dense": []}
    with torch.cuda.stream(side):
        for l in range(copies):
            for kind in ("sparse", "dense"):
                def block(stream):
                    for n in range(s):
                        if kind == "sparse":
                            ctx.decode_step(l, n, sched, q[l, n], views[l][n], B, out, stream=stream)
                        else:
                            ctx.dense_decode_attn(q[l, n], views[l][n], B, out, stream=stream)
                block(side)
                side.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
                    block(torch.cuda.current_stream())
                graphs[kind].append(g)
    torch.cuda.synchronize()
    res = {}
    stream = torch.cuda.current_stream()
    for kind in ("sparse", "dense"):
        ts = []
        for r in range(reps):
            for g in graphs[kind]:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                g.replay()
                b.record(stream)
                torch.cuda.synchronize()
                if r > 0:
                    ts.append(a.elapsed_time(b) * 1e3 / s)
        res[kind] = statistics.median(ts)
    assert ctx.check() == 0
    ctx.close()
    return res


CTX_FLAGS = 0      # PRHS_CFG_* flags every context of this module is created with (--ctx-flags)


def _make_caches(w: W.Workload, dev):
    """(kv list per layer, page table on the device or None): the workload's caches, paged if it asks."""
    if w.page_size:
        table, pool = W.make_page_table(w)
        kv = []
        for _, k, v in W.make_layer_kv(w, dev):       # page one layer at a time to bound memory
            kv.append((W.to_paged(w, k, table, pool), W.to_paged(w, v, table, pool)))
            del k, v
        return kv, table.to(dev)
    return [(k, v) for _, k, v in W.make_layer_kv(w, dev)], None


def _set_bytes(idx, cnt, w: W.Workload):
    """(logical, unique) bytes a step must gather for the lists (idx, cnt): every listed row once per
    query head, and once per KV head for the union over the heads of a group; 512 B per row (K + V)."""
    B, Hq, cap = idx.shape
    G = Hq // w.kv_heads
    valid = torch.arange(cap)[None, None, :] < cnt[:, :, None]
    mark = torch.zeros(B * w.kv_heads, w.capacity + 1, dtype=torch.bool)
    unit = (torch.arange(B)[:, None] * w.kv_heads + torch.arange(Hq)[None, :] // G)[:, :, None].expand_as(idx)
    mark[unit[valid].long(), idx[valid].long()] = True
    return int(cnt.sum()) * 512, int(mark.sum()) * 512


def config_summary(w: W.Workload, dev, reps: int = 7, copies: int = 4, group_sets: bool = False,
                   hbm_peak_gbs: float | None = None) -> dict:
    """One configuration of the benchmark, timed as its schedule runs it.

    A block is one retrieval period: s decode steps of every layer of ONE layer group (the
    configuration's G_L layers, each with its own cache; the first layer retrieves on the
    block's first step, every other layer-step shares), or, for a single-layer configuration,
    s decode steps of `copies` independent copies of the layer (each retrieves once).  Either
    way consecutive layer-steps touch different caches, so no step finds its rows in L2.  The
    block is captured into a CUDA graph once and replayed `reps` times (median); the dense
    baseline likewise.  Bytes are the algorithmic bytes of the path: K once per retrieval and
    the gathered K/V rows of every layer-step, logical (per query head) and unique (per KV head).
    """
    s = w.refresh
    grouped = w.layer_group > 1
    NL = w.layer_group if grouped else copies
    ws = w.scaled(layers=NL, steps=s + 1)
    kv, table = _make_caches(ws, dev)
    q = W.make_queries(ws, dev)
    B, Hq = ws.batch, ws.q_heads
    kps = W.top_k_per_seq(ws)
    max_k = max(ws.top_k, int(ws.k_frac * ws.context))
    ctx = P.Context(NL, B, Hq, ws.kv_heads, ws.capacity, max_k, ws.window, ws.sinks, max_dilate_r=ws.dilate_r,
                    page_size=ws.page_size, min_layer_group=ws.layer_group, flags=CTX_FLAGS)
    sched = P.make_schedule(ws.top_k, ws.window, ws.sinks, refresh_interval=s, layer_group=ws.layer_group,
                            dilate_r=ws.dilate_r, top_k_per_seq=None if kps is None else kps.to(dev),
                            flags=P.PRHS_GROUP_SETS if group_sets else 0)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    lens = [W.seq_lens_at(ws, n).to(dev) for n in range(s)]
    views = [[P.make_view(kv[l][0], kv[l][1], lens[n], page_table=table, max_seq_len=ws.capacity)
              for n in range(s)] for l in range(NL)]
    order = [(l, n) for n in range(s) for l in range(NL)]

    def block(kind, stream=None):
        for l, n in order:
            if kind == "sparse":
                ctx.decode_step(l, n, sched, q[l, n], views[l][n], B, out, stream=stream)
            else:
                ctx.dense_decode_attn(q[l, n], views[l][n], B, out, stream=stream)

    # ---- bytes and per-step times from one directly launched block (an event pair per layer-step)
    stream = torch.cuda.current_stream()
    block("sparse")
    torch.cuda.synchronize()
    step_us, sizes, key_bytes = {}, {}, 0
    evs = []
    ctx.profile_begin(16 * len(order))
    for l, n in order:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        ctx.decode_step(l, n, sched, q[l, n], views[l][n], B, out)
        b.record(stream)
        evs.append((a, b))
    prof = ctx.profile_end()
    torch.cuda.synchronize()
    retr = [(l, n) for l, n in order if n == 0 and (l % ws.layer_group == 0)]
    times = {ln: a.elapsed_time(b) * 1e3 for ln, (a, b) in zip(order, evs)}
    share = [ln for ln in order if ln not in retr]
    step_us["retrieval"] = statistics.median(times[ln] for ln in retr)
    step_us["sharing"] = statistics.median(times[ln] for ln in share) if share else None
    kernels = {name: ms * 1e3 / cnt for name, (ms, cnt) in prof.items() if cnt}
    # set sizes: the retrieving call (undilated set) and a sharing call (dilated set)
    ctx.decode_step(0, 0, sched, q[0, 0], views[0][0], B, out)
    idx_s, cnt_s = ctx.get_index_set(B)
    sizes["retrieval"] = _set_bytes(idx_s, cnt_s, ws)
    sizes["sharing"] = (0, 0)
    if share:
        l, n = (1, 0) if grouped else (0, 1)      # a follower layer, or the layer's next step
        ctx.decode_step(l, n, sched, q[l, n], views[l][n], B, out)
        idx_s, cnt_s = ctx.get_index_set(B)
        sizes["sharing"] = _set_bytes(idx_s, cnt_s, ws)
    key_bytes = int(lens[0].sum()) * ws.kv_heads * 256
    n_retr, n_steps = len(retr), len(order)
    per_step = {kind: (n_retr * (key_bytes + sizes["retrieval"][i]) + (n_steps - n_retr) * sizes["sharing"][i]) / n_steps
                for i, kind in enumerate(("logical", "unique"))}
    dense_bytes = int(lens[0].sum()) * ws.kv_heads * 512

    # ---- whole blocks replayed from CUDA graphs
    side = torch.cuda.Stream()
    graphs = {}
    with torch.cuda.stream(side):
        for kind in ("sparse", "dense"):
            block(kind, side)
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
                block(kind, torch.cuda.current_stream())
            graphs[kind] = g
    torch.cuda.synchronize()
    us = {}
    for kind in ("sparse", "dense"):
        graphs[kind].replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            graphs[kind].replay()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3 / n_steps)
        us[kind] = (statistics.median(ts), min(ts), max(ts))
    flags = ctx.check()
    ctx.close()
    del kv, views, graphs
    torch.cuda.empty_cache()
    res = {
        "workload": ws.name, "batch": B, "q_heads": Hq, "kv_heads": ws.kv_heads, "context": ws.context,
        "refresh_interval": s, "layer_group": ws.layer_group, "paged": bool(ws.page_size),
        "caches": f"{NL} layers of one layer group" if grouped else f"{NL} independent copies of the layer",
        "layer_steps_per_retrieval": n_steps // n_retr,
        "us_per_layer_step": us["sparse"][0], "us_per_layer_step_min_max": list(us["sparse"][1:]),
        "dense_us_per_layer_step": us["dense"][0], "dense_over_sparse": us["dense"][0] / us["sparse"][0],
        "retrieval_step_us": step_us["retrieval"], "sharing_step_us": step_us["sharing"],
        "kernel_avg_us_per_launch": {k: round(v, 1) for k, v in kernels.items()},
        "key_bytes_per_retrieval": key_bytes,
        "gather_bytes_logical": {"retrieval_step": sizes["retrieval"][0], "sharing_step": sizes["sharing"][0]},
        "gather_bytes_unique": {"retrieval_step": sizes["retrieval"][1], "sharing_step": sizes["sharing"][1]},
        "bytes_per_layer_step_logical": per_step["logical"], "bytes_per_layer_step_unique": per_step["unique"],
        "dense_bytes_per_layer_step": dense_bytes, "dense_gbs": dense_bytes / us["dense"][0] / 1e3,
        "mean_set_size_sharing": float(cnt_s.float().mean()),
        "select_fallback": bool(flags & P.PRHS_FLAG_SELECT_FALLBACK),
    }
    for kind in ("logical", "unique"):
        gbs = per_step[kind] / us["sparse"][0] / 1e3
        res[f"achieved_gbs_{kind}"] = gbs
        res[f"frac_of_8tbs_{kind}"] = gbs / 8000.0
        if hbm_peak_gbs:
            res[f"frac_of_measured_peak_{kind}"] = gbs / hbm_peak_gbs
    return res


def gated_summary(w: W.Workload, dev, tau: float = 0.8, sigma: float = 0.7, s: int = 16, blocks: int = 2,
                  copies: int = 2, reps: int = 5) -> dict:
    """The cosine-gated schedule (Eq. 9) timed against the fixed schedule at the same retrieval ratio.

    `copies` independent caches of the (single-layer) workload decode `blocks` blocks of `s` steps
    each, round-robin, with sim_threshold = tau and a query drift sigma large enough that a share
    of the heads fails the similarity test and retrieves inside the block.  The whole run is
    captured into a CUDA graph and replayed (the decisions depend only on the queries, so every
    replay takes the same ones); rho-hat is the fraction of (step, head) pairs that retrieved.  The
    fixed schedule is then timed the same way with the refresh interval nearest to 1 / rho-hat.
    """
    T = blocks * s
    ws = w.scaled(layers=copies, steps=T, layer_group=1, sigma=sigma, refresh=s)
    kv, table = _make_caches(ws, dev)
    q = W.make_queries(ws, dev)
    B, Hq = ws.batch, ws.q_heads
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    lens = [W.seq_lens_at(ws, n).to(dev) for n in range(T)]
    views = [[P.make_view(kv[l][0], kv[l][1], lens[n], page_table=table, max_seq_len=ws.capacity)
              for n in range(T)] for l in range(copies)]
    order = [(l, n) for n in range(T) for l in range(copies)]
    stream = torch.cuda.current_stream()

    def run(sim_threshold, refresh):
        ctx = P.Context(copies, B, Hq, ws.kv_heads, ws.capacity, ws.top_k, ws.window, ws.sinks,
                        max_dilate_r=ws.dilate_r, page_size=ws.page_size,
                        max_block_sets=refresh if sim_threshold is not None else 1, flags=CTX_FLAGS)
        sched = P.make_schedule(ws.top_k, ws.window, ws.sinks, refresh_interval=refresh, dilate_r=ws.dilate_r,
                                sim_threshold=-1.0 if sim_threshold is None else sim_threshold)
        retrieved = 0
        for l, n in order:                       # direct pass: warms up and counts the retrievals
            ctx.decode_step(l, n, sched, q[l, n], views[l][n], B, out)
            if sim_threshold is not None:
                need, _ = ctx.get_gate(l, B)
                retrieved += int(need.sum())
            elif n % refresh == 0:
                retrieved += B * Hq
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side, capture_error_mode="thread_local"):
                for l, n in order:
                    ctx.decode_step(l, n, sched, q[l, n], views[l][n], B, out, stream=torch.cuda.current_stream())
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            g.replay()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) * 1e3 / len(order))
        assert ctx.check() & ~P.PRHS_FLAG_SELECT_FALLBACK == 0
        ctx.close()
        return statistics.median(ts), retrieved / (len(order) * B * Hq)

    gated_us, rho = run(tau, s)
    s_eq = max(1, round(1.0 / max(rho, 1e-6)))
    while T % s_eq:                              # whole blocks of the fixed schedule in the same run
        s_eq -= 1
    fixed_us, rho_fixed = run(None, s_eq)
    del kv, views
    torch.cuda.empty_cache()
    return {"workload": ws.name, "batch": B, "tau": tau, "sigma": sigma, "block": s, "steps": T, "caches": copies,
            "rho_hat": rho, "gated_us_per_step": gated_us,
            "fixed_refresh_interval": s_eq, "fixed_rho_hat": rho_fixed, "fixed_us_per_step": fixed_us,
            "gated_over_fixed": gated_us / fixed_us}


def configs_summary(dev, group_sets=False, only=None, batch=0):
    import json
    for w in (W.C2_LLAMA2_7B, W.C3_MISTRAL, W.C4_LLAMA3_128K, W.C5_SERVING):
        if only and w.name != only:
            continue
        if batch:
            w = w.scaled(batch=batch)
        print(json.dumps(config_summary(w, dev, group_sets=group_sets)), flush=True)


def table3(dev, graph=False):
    if graph:
        print("| BS | seqlen | k | dense us / step | s=8 us / step | s=16 us / step | dense / s=8 | dense / s=16 "
              "| paper Flash / CPE-8 / CPE-16 ms (A100), ratios |")
        print("|---|---|---|---|---|---|---|---|---|")
        for batch in (8, 16):
            for n in (1024, 2048, 4096):
                w = table3_workload(batch, n)
                k = w.top_k
                r8, r16 = time_blocks(w, dev, 8), time_blocks(w, dev, 16)
                pf, p8, p16 = PAPER_TABLE3_MS[(batch, n)]
                print(f"| {batch} | {n} | {k} | {r16['dense']:.1f} | {r8['sparse']:.1f} | {r16['sparse']:.1f} | "
                      f"{r8['dense'] / r8['sparse']:.2f}x | {r16['dense'] / r16['sparse']:.2f}x | "
                      f"{pf} / {p8} / {p16}, {pf / p8:.1f}x / {pf / p16:.1f}x |")
        return
    print("| BS | seqlen | k | dense us | retrieval step us | sharing step us | amortised s=8 us | amortised s=16 us "
          "| dense / s=16 | paper Flash / CPE-8 / CPE-16 ms (A100) |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for batch in (8, 16):
        for n in (1024, 2048, 4096):
            w = table3_workload(batch, n)
            k = w.top_k
            r = time_workload(w, dev)
            am = {s: (r["refresh_us"] + (s - 1) * r["shared_us"]) / s for s in (8, 16)}
            pf, p8, p16 = PAPER_TABLE3_MS[(batch, n)]
            print(f"| {batch} | {n} | {k} | {r['dense_us']:.1f} | {r['refresh_us']:.1f} | {r['shared_us']:.1f} | "
                  f"{am[8]:.1f} | {am[16]:.1f} | {r['dense_us'] / am[16]:.2f}x | {pf} / {p8} / {p16} |")


def configs_graph(dev, group_sets=False, only=None, batch=0):
    print("| config | steps per retrieval (s x G_L) | dense us / step | sparse us / step | dense / sparse |")
    print("|---|---|---|---|---|")
    for w in (W.C2_LLAMA2_7B, W.C3_MISTRAL, W.C4_LLAMA3_128K, W.C5_SERVING):
        if only and w.name != only:
            continue
        if batch:
            w = w.scaled(batch=batch)
        period = w.refresh * w.layer_group
        # a follower layer's step costs what a sharing step costs: one block of `period` steps
        r = time_blocks(w.scaled(layer_group=1), dev, period, copies=4 if w.context < 50000 else 2,
                        group_sets=group_sets)
        print(f"| {w.name} | {period} | {r['dense']:.1f} | {r['sparse']:.1f} | {r['dense'] / r['sparse']:.2f}x |",
              flush=True)
        torch.cuda.empty_cache()


def configs(dev, group_sets=False, only=None, batch=0):
    print("| config | dense us | retrieval step us | sharing step us | amortised (config's s, G_L) us | "
          "mean set size | dense / amortised | sharing step GB/s logical / unique | retrieval step kernels us |")
    print("|---|---|---|---|---|---|---|---|---|")
    for w in (W.C2_LLAMA2_7B, W.C3_MISTRAL, W.C4_LLAMA3_128K, W.C5_SERVING):
        if only and w.name != only:
            continue
        if batch:
            w = w.scaled(batch=batch)
        r = time_workload(w.scaled(layer_group=1), dev, copies=4 if w.context < 50000 else 2, group_sets=group_sets)
        period = w.refresh * w.layer_group      # layer-steps per retrieval
        am = (r["refresh_us"] + (period - 1) * r["shared_us"]) / period
        gbs = [r[k] / (r["shared_us"] * 1e3) for k in ("logical_bytes", "unique_bytes")]
        kern = ", ".join(f"{k} {v:.1f}" for k, v in r["kernels"].items())
        print(f"| {w.name} | {r['dense_us']:.1f} | {r['refresh_us']:.1f} | {r['shared_us']:.1f} | {am:.1f} | "
              f"{r['set_size']:.0f} | {r['dense_us'] / am:.2f}x | {gbs[0]:.0f} / {gbs[1]:.0f} | {kern} "
              f"(K stream {r['key_bytes'] / 1e6:.0f} MB) |")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", action="store_true", help="time the benchmark's C2..C5 shapes instead")
    ap.add_argument("--graph", action="store_true",
                    help="whole blocks of steps (one retrieval and the sharing steps that follow) replayed from "
                         "CUDA graphs: time per step")
    ap.add_argument("--summary", action="store_true",
                    help="with --configs: one JSON line per configuration, timed as its own schedule runs it (layer "
                         "groups included): time, bytes and roofline fractions per layer-step")
    ap.add_argument("--gated", action="store_true",
                    help="the cosine-gated schedule (tau 0.8) on the c2 shape against the fixed schedule at the same "
                         "retrieval ratio: one JSON line per query drift sigma")
    ap.add_argument("--sigmas", default="0.6,0.7,0.75", help="with --gated: query drifts to time")
    ap.add_argument("--only", default=None, help="with --configs: time this configuration alone (its name)")
    ap.add_argument("--batch", type=int, default=0, help="with --configs: override the batch size (profiler captures)")
    ap.add_argument("--ctx-flags", type=int, default=0,
                    help="PRHS_CFG_* flags for every context (4: mma.sync scoring, 8: tcgen05 group attention, ...)")
    ap.add_argument("--group-sets", action="store_true",
                    help="with --configs: the labelled variant with one index set per KV head (not in the paper)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    global CTX_FLAGS
    CTX_FLAGS = args.ctx_flags
    if args.gated:
        import json
        w = W.CONFIGS[args.only] if args.only else W.C2_LLAMA2_7B
        if args.batch:
            w = w.scaled(batch=args.batch)
        for sg in args.sigmas.split(","):
            print(json.dumps(gated_summary(w, dev, sigma=float(sg))), flush=True)
    elif args.configs and args.summary:
        configs_summary(dev, args.group_sets, args.only, args.batch)
    elif args.configs:
        (configs_graph if args.graph else configs)(dev, args.group_sets, args.only, args.batch)
    else:
        table3(dev, args.graph)


if __name__ == "__main__":
    main()
