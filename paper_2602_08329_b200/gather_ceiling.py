"""How fast can the rows of a sharing step be gathered at all?

    python -m paper_2602_08329_b200.gather_ceiling [--config c2_llama2_7b_layer] [--batch B]

Runs one retrieval step and one sharing step of a benchmark configuration, materialises the
sharing step's index lists, and times, on those lists: the gathered attention itself (fused list
and explicit list), and the bare row gather of `prhs_gather_probe` in its four variants (plain
loads, cp.async ring, per-row bulk copies, TMA gather4).  Every figure is the median of per-launch CUDA-event times
over independent cache copies visited in turn (no launch finds its rows in L2).  Prints a markdown
table: what the attention kernel could gain from a different copy mechanism, and what no mechanism
can give it.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics

import torch

from . import binding as P
from . import workloads as W

VARIANTS = ["plain 16-byte loads into registers", "cp.async 16-byte copies, shared-memory ring",
            "cp.async.bulk, one 256-byte copy per row", "TMA tile::gather4, four rows per instruction"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="c2_llama2_7b_layer")
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--copies", type=int, default=3)
    ap.add_argument("--reps", type=int, default=7)
    args = ap.parse_args()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    w = W.CONFIGS[args.config]
    if w.page_size:
        raise SystemExit("the probe reads contiguous caches")
    if args.batch:
        w = w.scaled(batch=args.batch)
    L = args.copies
    w = w.scaled(layers=L, steps=2, layer_group=1)
    kv = [(k, v) for _, k, v in W.make_layer_kv(w, dev)]
    q = W.make_queries(w, dev)
    B, Hq = w.batch, w.q_heads
    ctx = P.Context(L, B, Hq, w.kv_heads, w.capacity, w.top_k, w.window, w.sinks, max_dilate_r=w.dilate_r)
    sched = P.make_schedule(w.top_k, w.window, w.sinks, refresh_interval=w.refresh, dilate_r=w.dilate_r)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    t0, t1 = W.seq_lens_at(w, 0).to(dev), W.seq_lens_at(w, 1).to(dev)
    v0 = [P.make_view(kv[l][0], kv[l][1], t0, max_seq_len=w.capacity) for l in range(L)]
    v1 = [P.make_view(kv[l][0], kv[l][1], t1, max_seq_len=w.capacity) for l in range(L)]
    cap = ctx.index_capacity
    lists = []
    for l in range(L):
        ctx.decode_step(l, 0, sched, q[l, 0], v0[l], B, out)
        idx = torch.empty(B, Hq, cap, dtype=torch.int32, device=dev)
        cnt = torch.empty(B, Hq, dtype=torch.int32, device=dev)
        ctx.build_index_set(l, 1, sched, v1[l], B, idx, cnt)
        lists.append((idx, cnt))
    rows = int(lists[0][1].sum())
    nbytes = rows * 512
    stream = torch.cuda.current_stream()

    def timed(fn, rounds=4):
        """Median time per launch: each sample brackets `rounds` passes over the cache copies with one
        pair of events (the event clock ticks in steps of about 2 us: a single launch is too short to
        time on its own), launches back to back, every launch on another copy than the one before."""
        ts = []
        for r in range(args.reps + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(rounds):
                for l in range(L):
                    fn(l)
            b.record(stream)
            torch.cuda.synchronize()
            if r > 0:
                ts.append(a.elapsed_time(b) * 1e3 / (rounds * L))
        return statistics.median(ts)

    res = [("gathered attention, list built in the kernel (a sharing step)",
            timed(lambda l: ctx.decode_step(l, 1, sched, q[l, 1], v1[l], B, out)))]
    res.append(("gathered attention, explicit lists",
                timed(lambda l: ctx.sparse_decode_attn(q[l, 1], v1[l], lists[l][0], lists[l][1], B, out))))
    for variant, name in enumerate(VARIANTS):
        res.append((f"bare gather: {name}", timed(lambda l: ctx.gather_probe(variant, v1[l], lists[l][0], lists[l][1], B))))
    # the same attention with its rows brought in by TMA row gathers (a context flag)
    ctx_t = P.Context(L, B, Hq, w.kv_heads, w.capacity, w.top_k, w.window, w.sinks, max_dilate_r=w.dilate_r,
                      flags=P.PRHS_CFG_TMA_GATHER)
    res.insert(2, ("gathered attention, explicit lists, rows by TMA gather4 (PRHS_CFG_TMA_GATHER)",
                   timed(lambda l: ctx_t.sparse_decode_attn(q[l, 1], v1[l], lists[l][0], lists[l][1], B, out))))
    assert ctx_t.check() == 0
    ctx_t.close()
    flags = ctx.check()
    peak = None
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    if os.path.exists(path):
        peak = float(json.load(open(path))["hbm_gbs"])
    print(f"{w.name}: batch {B}, {Hq} heads, {rows} listed rows ({rows / (B * Hq):.0f} per unit), "
          f"{nbytes / 1e6:.1f} MB per launch, {L} cache copies in turn; device flags {flags}")
    print("| what | us | GB/s |" + (" of measured copy peak |" if peak else ""))
    print("|---|---|---|" + ("---|" if peak else ""))
    for name, us in res:
        gbs = nbytes / us / 1e3
        print(f"| {name} | {us:.1f} | {gbs:.0f} |" + (f" {gbs / peak:.2f} |" if peak else ""))
    ctx.close()


if __name__ == "__main__":
    main()
