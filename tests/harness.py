"""Shared helpers for the GPU parity tests: run the CUDA path through the C ABI and the CPU
oracle on the same seeded tensors, and compare with the tolerances the benchmark fixes.

Tolerances (bf16 inputs, fp32 accumulation on the GPU, float64 in the oracle):
  index sets      bit-exact, except positions whose oracle logit lies within 1e-3 relative
                  of the k-th (or, for dilation extras, the m-th) largest logit
  attention y     max-abs 2e-2 between the kernel's bf16 output and the oracle's float64 value,
                  the oracle evaluated on the GPU's own index set.  (The oracle's value is not
                  rounded to bf16 first: with both sides rounded, a value near a rounding tie at
                  |y| >= 4, where one bf16 step is 2^-5 = 0.031, can land one whole step apart
                  although each side is within half a step of the exact result.)
  delta           1e-4 absolute
  logits          1e-4 absolute + 1e-5 relative (fp32 accumulation order)
  order inside S* two winners may appear in either order only if their oracle logits differ by
                  no more than twice the logit tolerance (each side's fp32 logit is within one
                  tolerance of the exact value); the order fixes the top-m of Eq. 10
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import prhs_oracle as O
from paper_2602_08329_b200 import binding as P
from paper_2602_08329_b200 import workloads as W

Y_TOL = 2e-2
DELTA_TOL = 1e-4
TIE_REL = 1e-3
LOGIT_ATOL, LOGIT_RTOL = 1e-4, 1e-5
SIM_TOL = 1e-4          # a cosine similarity this close to tau may fall either way (fp32 vs float64)


def np32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


def tie_band(a_ref: float) -> float:
    return TIE_REL * max(abs(a_ref), 1e-3)


def order_band(a_ref: float) -> float:
    """How far apart two oracle logits may lie for the kernel to rank them the other way round."""
    return 2.0 * (LOGIT_ATOL + LOGIT_RTOL * abs(a_ref))


def check_topk_legal(a32: np.ndarray, got_desc: np.ndarray, want_desc: np.ndarray, where=""):
    """`got_desc` must equal the oracle's S* except for near-ties with the k-th logit (membership:
    the 1e-3 relative band), and be in the oracle's order except between logits that the fp32
    accumulation order cannot tell apart (order: twice the logit tolerance)."""
    assert len(got_desc) == len(want_desc), f"{where}: |S*| {len(got_desc)} != {len(want_desc)}"
    if len(want_desc) == 0:
        return
    assert len(set(got_desc.tolist())) == len(got_desc), f"{where}: duplicate winners"
    a_k = float(a32[want_desc[-1]])
    diff = np.setxor1d(got_desc, want_desc)
    for i in diff:
        assert abs(float(a32[i]) - a_k) <= tie_band(a_k), \
            f"{where}: position {i} logit {a32[i]} differs from the oracle set beyond the tie band of {a_k}"
    # descending order (ties by lower position), up to what the logit tolerance allows
    ag = a32[got_desc].astype(np.float64)
    bands = 2.0 * (LOGIT_ATOL + LOGIT_RTOL * np.abs(ag[:-1]))
    assert np.all(np.diff(ag) <= bands), f"{where}: S* not in descending-logit order"
    if len(diff) == 0:
        same = got_desc == want_desc
        for j in np.nonzero(~same)[0]:
            assert abs(float(a32[got_desc[j]]) - float(a32[want_desc[j]])) <= order_band(a32[want_desc[j]]), \
                f"{where}: order differs at rank {j} beyond what the logit tolerance allows"


def make_ctx(w: W.Workload, **over):
    kw = dict(num_layers=w.layers, max_batch=w.batch, num_q_heads=w.q_heads, num_kv_heads=w.kv_heads,
              max_context=w.capacity, max_k=max(w.top_k, int(w.k_frac * w.context)),
              max_window=w.window, max_sinks=w.sinks, max_dilate_r=max(w.dilate_r, 1), max_dilate_m=-1,
              page_size=w.page_size, min_layer_group=w.layer_group,
              max_block_sets=w.refresh if w.sim_threshold is not None else 1)
    kw.update(over)
    return P.Context(**kw)


def make_sched(w: W.Workload, device, flags=0, **over):
    kps = W.top_k_per_seq(w)
    kps_dev = kps.to(device) if kps is not None else None
    kw = dict(top_k=w.top_k, window=w.window, sinks=w.sinks, refresh_interval=w.refresh,
              layer_group=w.layer_group, dilate_r=w.dilate_r, dilate_m=-1, top_k_per_seq=kps_dev,
              flags=flags, psaw_phi=w.psaw_phi, psaw_alpha=w.psaw_alpha,
              psaw_layer_start=w.psaw_layer_start,
              sim_threshold=-1.0 if w.sim_threshold is None else w.sim_threshold)
    kw.update(over)
    return P.make_schedule(**kw)


def oracle_sched(w: W.Workload, **over) -> O.Schedule:
    kps = W.top_k_per_seq(w)
    kw = dict(top_k=w.top_k, window=w.window, sinks=w.sinks, refresh_interval=w.refresh,
              layer_group=w.layer_group, dilate_r=w.dilate_r, dilate_m=-1,
              top_k_per_seq=None if kps is None else kps.numpy(),
              # the C ABI carries phi and alpha as fp32: give the oracle the same values
              psaw_phi=float(np.float32(w.psaw_phi)), psaw_alpha=float(np.float32(w.psaw_alpha)),
              psaw_layer_start=w.psaw_layer_start, num_layers=w.layers,
              sim_threshold=None if w.sim_threshold is None else float(np.float32(w.sim_threshold)))
    kw.update(over)
    return O.Schedule(**kw)


class HostKV:
    """Lazy host copies of single (layer, b, kvh) cache slices as float32 numpy arrays."""

    def __init__(self):
        self.cache = {}

    def get(self, tag, tensor, b, kvh):
        key = (tag, b, kvh)
        if key not in self.cache:
            self.cache[key] = np32(tensor[b, kvh])
        return self.cache[key]


class _HostSlices:
    """K[b, kvh] / V[b, kvh] for the oracle, copied from the device one slice at a time."""

    def __init__(self, host, tag, tensor):
        self.host, self.tag, self.tensor = host, tag, tensor

    def __getitem__(self, key):
        b, kvh = key
        return self.host.get(self.tag, self.tensor, b, kvh)


def run_schedule_parity(w: W.Workload, device, units, layers=None, steps=None, want_delta=True,
                        paged=False, check_scores=True, group_sets=False, dilate_anchor=False, dilate_m=-1,
                        ctx_over=None):
    """Drive prhs_decode_step over the workload's schedule and compare sampled (b, h) units.

    The oracle follows the same schedule.  Where the GPU retrieved, its S* is first checked
    for legality against the oracle's own top-k (near-ties at the k-th logit only) and then
    handed to the oracle as an override, so that every later comparison in the block
    (dilation, shared sets, attention, delta) is exact.
    `ctx_over` overrides sizes of the context (a context larger than the workload).
    `dilate_anchor` makes the retrieving call attend over the dilated set too; `dilate_m` fixes the
    number of dilated winners instead of k/3.  `group_sets` runs the labelled variant with one set per KV head (ranking by the group's
    maximum logit) on both sides.
    Returns a dict of summary statistics.
    """
    layers = list(range(w.layers)) if layers is None else layers
    steps = w.steps if steps is None else steps
    ctx = make_ctx(w, max_dilate_m=dilate_m, **(ctx_over or {}))
    flags = ((P.PRHS_WANT_DELTA if want_delta else 0) | (P.PRHS_GROUP_SETS if group_sets else 0) |
             (P.PRHS_DILATE_ANCHOR if dilate_anchor else 0))
    sched = make_sched(w, device, flags=flags, dilate_m=dilate_m)
    osched = oracle_sched(w, group_sets=group_sets, dilate_anchor=dilate_anchor, dilate_m=dilate_m)
    orc = O.PrhsOracle(osched, w.q_heads, w.kv_heads)
    q_all = W.make_queries(w, device)
    kv = {l: (k, v) for l, k, v in W.make_layer_kv(w, device, layers=layers)}
    table = pool = None
    paged_kv = {}
    if paged:
        table, pool = W.make_page_table(w)
        for l in layers:
            paged_kv[l] = (W.to_paged(w, kv[l][0], table, pool), W.to_paged(w, kv[l][1], table, pool))
        table_dev = table.to(device)
    host = HostKV()
    B, Hq = w.batch, w.q_heads
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device=device)
    dlt = torch.empty(B, Hq, dtype=torch.float32, device=device)
    stats = dict(select_fallback=False, max_y_err=0.0, max_delta_err=0.0, near_tie_sets=0, checked=0,
                 deltas=[], set_sizes=[], retrievals=0)
    gq = w.q_heads // w.kv_heads
    for n in range(steps):
        t_host = W.seq_lens_at(w, n)
        t_dev = t_host.to(device)
        for l in layers:
            k_l, v_l = kv[l]
            if paged:
                view = P.make_view(paged_kv[l][0], paged_kv[l][1], t_dev, page_table=table_dev,
                                   max_seq_len=w.capacity)
            else:
                view = P.make_view(k_l, v_l, t_dev, max_seq_len=w.capacity)
            q = q_all[l, n].contiguous()
            ctx.decode_step(l, n, sched, q, view, B, out, dlt if want_delta else None)
            idx, cnt = ctx.get_index_set(B)
            dev_flags = ctx.check()
            assert dev_flags & ~P.PRHS_FLAG_SELECT_FALLBACK == 0
            stats["select_fallback"] = stats["select_fallback"] or bool(dev_flags & P.PRHS_FLAG_SELECT_FALLBACK)
            y_gpu, d_gpu = np32(out), np32(dlt)
            gated = w.sim_threshold is not None
            leader = l % w.layer_group == 0
            qh = np32(q)
            Ks, Vs = _HostSlices(host, ("k", l), k_l), _HostSlices(host, ("v", l), v_l)
            # which units retrieved: the fixed schedule, or the cosine gate's decision on the device
            over_ref = {}
            if gated and leader:
                need, gref = ctx.get_gate(l, B)
                retr = {u: bool(need[u[0], u[1]]) for u in units}
                pos = n % w.refresh
                if pos > 0:
                    tau = osched.sim_threshold
                    for (b, h) in units:
                        blk = orc.blocks[(l // w.layer_group, b, h)]
                        want_ref, sims = O.gate_decision(qh[b, h], blk.queries, tau)
                        got_ref = int(gref[b, h])
                        where = f"layer {l} step {n} unit ({b},{h})"
                        assert -1 <= got_ref < pos and (got_ref < 0) == retr[(b, h)], where
                        if got_ref != want_ref:       # only similarities within rounding of tau may differ
                            assert all(sims[j] <= tau + SIM_TOL for j in range(got_ref + 1, pos)), where
                            assert got_ref < 0 or sims[got_ref] > tau - SIM_TOL, where
                            stats["near_tie_sets"] += 1
                        over_ref[(b, h)] = got_ref
            elif gated:
                retr = {u: False for u in units}
            else:
                retr = {u: orc.is_retrieval(l, n) for u in units}
            retrieve = any(retr.values())
            if retrieve:
                s_star, n_star, s_hat, n_hat = ctx.get_shared_set(l, B)
                scores = ctx.get_scores(B) if check_scores else None
            over_s = {}
            if retrieve:
                for (b, h) in units:
                    if not retr[(b, h)]:
                        continue
                    t = int(t_host[b])
                    where = f"layer {l} step {n} unit ({b},{h})"
                    hs = h - h % gq if group_sets else h        # whose rows hold the set and the logits
                    if group_sets:
                        a = O.group_logits([O.dense_scores(qh[b, hs + j], Ks[b, h // gq], t) for j in range(gq)])
                    else:
                        a = O.dense_scores(qh[b, h], Ks[b, h // gq], t)
                    a32 = O.rank_logits(a)
                    want = O.topk_middle(a, t, w.sinks, w.window, osched.k_for(b), osched.psaw_for(l, t))
                    got = s_star[b, h, : int(n_star[b, h])].numpy().astype(np.int64)
                    before = len(np.setxor1d(got, want))
                    check_topk_legal(a32, got, want, where)
                    stats["near_tie_sets"] += int(before > 0)
                    if check_scores:
                        sg = scores[b, hs, :t].numpy()
                        assert np.allclose(sg, a32, atol=LOGIT_ATOL, rtol=LOGIT_RTOL), f"{where}: logits differ"
                    over_s[(b, hs)] = got         # legal: the oracle adopts it
            ref = orc.decode_step(l, n, qh, Ks, Vs, t_host.numpy(), units=units, want_delta=want_delta,
                                  override_s_star=over_s, override_ref=over_ref)
            for (b, h) in units:
                t = int(t_host[b])
                where = f"layer {l} step {n} unit ({b},{h})"
                assert ref["retrieved"][(b, h)] == retr[(b, h)], where
                if retr[(b, h)]:
                    got_hat = s_hat[b, h, : int(n_hat[b, h])].numpy().astype(np.int64)
                    assert np.array_equal(got_hat, ref["s_hat"][(b, h)]), f"{where}: dilated set differs"
                    stats["retrievals"] += 1
                C_want = ref["set"][(b, h)]
                C_got = idx[b, h, : int(cnt[b, h])].numpy().astype(np.int64)
                assert np.array_equal(C_got, C_want), f"{where}: index set differs"
                err = float(np.max(np.abs(y_gpu[b, h] - ref["y"][(b, h)])))
                assert err <= Y_TOL, f"{where}: attention max-abs error {err}"
                stats["max_y_err"] = max(stats["max_y_err"], err)
                stats["set_sizes"].append(len(C_want))
                if want_delta:
                    d_ref = ref["delta"][(b, h)]
                    derr = abs(float(d_gpu[b, h]) - d_ref)
                    assert derr <= DELTA_TOL, f"{where}: delta {d_gpu[b, h]} vs {d_ref}"
                    stats["max_delta_err"] = max(stats["max_delta_err"], derr)
                    stats["deltas"].append(d_ref)
                stats["checked"] += 1
    ctx.close()
    return stats
