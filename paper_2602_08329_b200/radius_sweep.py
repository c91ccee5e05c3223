"""Block size x dilation radius sweep of the dropped-mass diagnostic on the 128K configuration.

    python -m paper_2602_08329_b200.radius_sweep [--q-scale 3] [--halo 0.7] [--batch 4]

For every cell s in {1, 2, 4, 8} x r in {0, 1, 2} the library decodes the configuration's T
steps and reports, over all (sequence, head, step):

  delta      dropped mass of the set in use (Sec. 3.2: 1 - sum of the full softmax over the set)
  delta*     dropped mass of the same step's own top-k set (the per-step oracle selector)
  beta       delta - delta*: what sharing costs on top of selecting afresh (Sec. 3.3)
  coverage   |S*_n  intersect  M_n| / k: how much of the step's own top-k the shared middle set
             still holds (the overlap the paper plots against query distance, Sec. 4.1)
  |C|        mean size of the index set
  us         amortised device time per step (CUDA events, diagnostic off)

delta* and S*_n come from a second library context that retrieves on every step (s = 1); at
s = 1 the anchor attends over its undilated set, so that row is the sanity row: beta = 0,
coverage = 1 for every r.  Data are synthetic (`workloads.py`); the position-clustered variant
(`--halo`) gives every heavy hitter weaker copies on its neighbours, which is the structure the
neighbour dilation of Eq. 10 is built for -- on i.i.d. keys a larger radius only grows the set.
Prints a markdown table.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as P
from . import workloads as W


def run_cell(w: W.Workload, dev, k, v, q, s: int, r: int):
    B, Hq = w.batch, w.q_heads
    mk = lambda: P.Context(1, B, Hq, w.kv_heads, w.capacity, w.top_k, w.window, w.sinks, max_dilate_r=max(r, 1))
    ctx, probe = mk(), mk()
    sched = P.make_schedule(w.top_k, w.window, w.sinks, refresh_interval=s, dilate_r=r, flags=P.PRHS_WANT_DELTA)
    sched_t = P.make_schedule(w.top_k, w.window, w.sinks, refresh_interval=s, dilate_r=r)
    sched_1 = P.make_schedule(w.top_k, w.window, w.sinks, refresh_interval=1, dilate_r=r, flags=P.PRHS_WANT_DELTA)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=dev)
    delta = torch.empty(B, Hq, dtype=torch.float32, device=dev)
    delta1 = torch.empty_like(delta)
    star = torch.empty(B, Hq, w.top_k, dtype=torch.int32, device=dev)
    nstar = torch.empty(B, Hq, dtype=torch.int32, device=dev)
    mark = torch.zeros(B * Hq, w.capacity + 1, dtype=torch.bool, device=dev)
    rows = torch.arange(B * Hq, device=dev)[:, None]
    acc = {"delta": [], "delta1": [], "cov": [], "size": []}
    lens = [W.seq_lens_at(w, n).to(dev) for n in range(w.steps)]
    views = [P.make_view(k, v, t, max_seq_len=w.capacity) for t in lens]
    for n in range(w.steps):
        ctx.decode_step(0, n, sched, q[0, n], views[n], B, out, out_delta=delta)
        idx, cnt = ctx.get_index_set(B)
        probe.decode_step(0, n, sched_1, q[0, n], views[n], B, out, out_delta=delta1)
        s_star, n_star, _, _ = probe.get_shared_set(0, B)
        idx, cnt = idx.to(dev).view(B * Hq, -1).long(), cnt.to(dev).view(-1)
        s_star, n_star = s_star.to(dev).view(B * Hq, -1).long(), n_star.to(dev).view(-1)
        valid = torch.arange(idx.shape[1], device=dev)[None, :] < cnt[:, None]
        mark.zero_()
        mark[rows.expand_as(idx)[valid], idx[valid]] = True
        sv = torch.arange(s_star.shape[1], device=dev)[None, :] < n_star[:, None]
        hit = (mark[rows.expand_as(s_star), s_star.clamp_min(0)] & sv).sum(1)
        acc["cov"].append(hit.float() / n_star.clamp_min(1).float())
        acc["delta"].append(delta.flatten().clone())
        acc["delta1"].append(delta1.flatten().clone())
        acc["size"].append(cnt.float())
    assert ctx.check() == 0 and probe.check() == 0
    probe.close()
    # timing: the same schedule without the diagnostic, three passes, the last two timed
    stream = torch.cuda.current_stream()
    times = []
    for rep in range(3):
        evs = []
        for n in range(w.steps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            ctx.decode_step(0, n, sched_t, q[0, n], views[n], B, out)
            b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
        if rep:
            times.append(sum(a.elapsed_time(b) for a, b in evs) * 1e3 / w.steps)
    ctx.close()
    cat = {name: torch.cat(x) for name, x in acc.items()}
    return {"delta_mean": float(cat["delta"].mean()), "delta_max": float(cat["delta"].max()),
            "delta1_mean": float(cat["delta1"].mean()),
            "beta_mean": float((cat["delta"] - cat["delta1"]).mean()),
            "beta_max": float((cat["delta"] - cat["delta1"]).max()),
            "cov_mean": float(cat["cov"].mean()), "cov_min": float(cat["cov"].min()),
            "size": float(cat["size"].mean()), "us": min(times)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--q-scale", type=float, default=3.0, help="query scale (1 = flat synthetic attention)")
    ap.add_argument("--halo", type=float, default=0.7, help="neighbour weight of the clustered variant (0 = i.i.d.)")
    ap.add_argument("--batch", type=int, default=W.C4_LLAMA3_128K.batch)
    ap.add_argument("--sigma", type=float, default=W.C4_LLAMA3_128K.sigma, help="query drift per step")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    w = W.C4_LLAMA3_128K.scaled(q_scale=args.q_scale, halo=args.halo, batch=args.batch, sigma=args.sigma)
    k, v = W.make_kv(w, dev)
    q = W.make_queries(w, dev)
    print(f"{w.name}: batch {w.batch}, {w.q_heads}/{w.kv_heads} heads, N {w.context}, k {w.top_k}, W {w.window}, "
          f"S0 {w.sinks}, T {w.steps}, m k/3, q_scale {w.q_scale}, halo {w.halo}, sigma {w.sigma}\n")
    print("| s | r | delta mean | delta max | delta* mean | beta mean | beta max | coverage mean | coverage min "
          "| mean set size | us / step |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    for s in (1, 2, 4, 8):
        for r in (0, 1, 2):
            c = run_cell(w, dev, k, v, q, s, r)
            print(f"| {s} | {r} | {c['delta_mean']:.4f} | {c['delta_max']:.4f} | {c['delta1_mean']:.4f} | "
                  f"{c['beta_mean']:.4f} | {c['beta_max']:.4f} | {c['cov_mean']:.4f} | {c['cov_min']:.4f} | "
                  f"{c['size']:.0f} | {c['us']:.1f} |", flush=True)


if __name__ == "__main__":
    main()
