"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle.

Small cases compare every element; the benchmark's full-size configurations compare sampled
(sequence, head) units that the oracle computes one by one, in the launch configuration the
benchmark times.  Tolerances are stated in tests/harness.py.

The selection kernel's CTA width follows the number of (sequence, head) units, so the
full-size tests are chosen to cover every width at the batch the configuration really uses:
  1024 threads (at most one unit per SM)   test_c4_long_context_sampled (4 x 32 = 128 units),
                                           test_c3_stack_slice_sampled (batch 4)
  512 threads                              test_c2_full_size_sampled (8 x 32 = 256 units),
                                           test_c5_full_batch_sampled (64 x 32 = 2048 units, a
                                           multi-wave grid of every kernel)
  256 threads (two to four units per SM)   test_c3_full_batch_sampled (16 x 32 = 512 units),
                                           test_table3_operator_shapes[16-4096-16]
Retrieval scoring runs the tcgen05 kernel (TMA-staged) everywhere except in the
test_score_mma_sync_* tests (PRHS_CFG_MMA_SYNC_SCORE: mma.sync consumer warps behind the same TMA
ring) and the test_score_ring_* tests (PRHS_CFG_NO_TMA: the cp.async ring kernel).
"""
import math

import numpy as np
import pytest
import torch

from oracle import prhs_oracle as O
from paper_2602_08329_b200 import binding as P
from paper_2602_08329_b200 import workloads as W
from tests import harness as H

pytestmark = pytest.mark.gpu


def all_units(w):
    return [(b, h) for b in range(w.batch) for h in range(w.q_heads)]


def small(name="small", **kw):
    base = dict(layers=1, batch=2, q_heads=4, kv_heads=2, context=1500, steps=4, top_k=48, window=16,
                sinks=4, refresh=2, heavy_hitters=8, decay_span=64, seed=11)
    base.update(kw)
    return W.Workload(name, **base)


# ------------------------------------------------------------------ stage by stage
@pytest.mark.parametrize("gq", [1, 2, 4, 8])
def test_sparse_attention_over_given_sets(cuda_device, gq):
    w = small(q_heads=8, kv_heads=8 // gq, context=3000, seed=20 + gq)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = torch.tensor([2999, 1234], dtype=torch.int32)
    g = np.random.default_rng(gq)
    cap = 700
    idx = torch.full((w.batch, w.q_heads, cap), -7, dtype=torch.int32)
    cnt = torch.zeros(w.batch, w.q_heads, dtype=torch.int32)
    sets = {}
    sizes = [0, 1, 15, 16, 17, 255, 256, 257, 511, 640, 700, 33, 300, 64, 129, 5]
    for b in range(w.batch):
        for h in range(w.q_heads):
            n = min(sizes[(b * w.q_heads + h) % len(sizes)], int(t_host[b]))
            C = np.sort(g.permutation(int(t_host[b]))[:n])
            sets[(b, h)] = C
            idx[b, h, :n] = torch.from_numpy(C.astype(np.int32))
            cnt[b, h] = n
    ctx = H.make_ctx(w)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    lse = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
    dlt = torch.empty_like(lse)
    ctx.sparse_decode_attn(q, view, idx.to(cuda_device), cnt.to(cuda_device), w.batch, out, lse)
    ctx.delta(q, view, idx.to(cuda_device), cnt.to(cuda_device), w.batch, dlt)
    assert ctx.check() == 0
    y, ls, dl, qh = H.np32(out), H.np32(lse), H.np32(dlt), H.np32(q)
    for (b, h), C in sets.items():
        kvh = h // gq
        Kh, Vh = H.np32(k[b, kvh]), H.np32(v[b, kvh])
        y_ref, lse_ref = O.attn_over_set(qh[b, h], Kh, Vh, C)
        assert np.max(np.abs(y[b, h] - y_ref)) <= H.Y_TOL
        if len(C) == 0:
            assert ls[b, h] == -math.inf and np.all(y[b, h] == 0) and dl[b, h] == 1.0
            continue
        assert abs(ls[b, h] - lse_ref) <= 1e-4
        a = O.dense_scores(qh[b, h], Kh, int(t_host[b]))
        assert abs(dl[b, h] - O.delta_from_lse(lse_ref, O.logsumexp(a))) <= H.DELTA_TOL
    ctx.close()


@pytest.mark.parametrize("gq", [1, 4, 8, 16])
def test_dense_baseline_matches_oracle(cuda_device, gq):
    w = small(q_heads=max(4, gq), kv_heads=max(4, gq) // gq, context=5000, seed=30 + gq)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 1].contiguous()
    t_host = torch.tensor([5003, 777], dtype=torch.int32)
    ctx = H.make_ctx(w)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    lse = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
    ctx.dense_decode_attn(q, view, w.batch, out, lse)
    assert ctx.check() == 0
    y, ls, qh = H.np32(out), H.np32(lse), H.np32(q)
    for b, h in all_units(w):
        y_ref, lse_ref = O.dense_attention(qh[b, h], H.np32(k[b, h // gq]), H.np32(v[b, h // gq]), int(t_host[b]))
        assert np.max(np.abs(y[b, h] - y_ref)) <= H.Y_TOL
        assert abs(ls[b, h] - lse_ref) <= 1e-4
    ctx.close()


@pytest.mark.parametrize("gq,context", [(1, 1500), (2, 2500), (4, 4100), (8, 700)])
def test_score_topk_and_dilation(cuda_device, gq, context):
    w = small(q_heads=8, kv_heads=8 // gq, context=context, top_k=96, seed=40 + gq)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = torch.tensor([context + 1, context // 2 + 3], dtype=torch.int32)
    ctx = H.make_ctx(w)
    sched = H.make_sched(w, cuda_device)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    oi = torch.empty(w.batch, w.q_heads, w.top_k, dtype=torch.int32, device=cuda_device)
    oc = torch.empty(w.batch, w.q_heads, dtype=torch.int32, device=cuda_device)
    ol = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
    ctx.score_topk(0, 0, q, view, sched, w.batch, oi, oc, ol)
    assert ctx.check() == 0
    scores = ctx.get_scores(w.batch)
    s_star, n_star, s_hat, n_hat = ctx.get_shared_set(0, w.batch)
    assert torch.equal(s_star[:, :, : w.top_k], oi.cpu()) and torch.equal(n_star, oc.cpu())
    qh, lf = H.np32(q), H.np32(ol)
    for b, h in all_units(w):
        t = int(t_host[b])
        Kh = H.np32(k[b, h // gq])
        a = O.dense_scores(qh[b, h], Kh, t)
        a32 = O.rank_logits(a)
        assert np.allclose(scores[b, h, :t].numpy(), a32, atol=1e-4, rtol=1e-5)
        assert abs(lf[b, h] - O.logsumexp(a)) <= 1e-4
        want = O.topk_middle(a, t, w.sinks, w.window, w.top_k)
        got = s_star[b, h, : int(n_star[b, h])].numpy().astype(np.int64)
        H.check_topk_legal(a32, got, want, f"unit ({b},{h})")
        assert np.all(s_star[b, h, int(n_star[b, h]):].numpy() == -1)
        hat = s_hat[b, h, : int(n_hat[b, h])].numpy().astype(np.int64)
        assert np.array_equal(hat, O.dilate(got, w.top_k // 3, 1, t))
    ctx.close()


def test_identical_keys_take_the_tie_path(cuda_device):
    # all logits equal: S* must be the k lowest middle positions, in position order
    w = small(batch=1, q_heads=2, kv_heads=1, context=3000, top_k=100)
    k, v = W.make_kv(w, cuda_device)
    k[:] = k[:, :, :1, :]
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = torch.tensor([2900], dtype=torch.int32)
    ctx = H.make_ctx(w)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    ctx.score_topk(0, 0, q, view, H.make_sched(w, cuda_device), 1)
    assert ctx.check() == P.PRHS_FLAG_SELECT_FALLBACK      # all-equal logits: the generic path ran
    s_star, n_star, s_hat, n_hat = ctx.get_shared_set(0, 1)
    for h in range(2):
        assert int(n_star[0, h]) == 100
        assert np.array_equal(s_star[0, h, :100].numpy(), np.arange(4, 104))
        assert np.array_equal(s_hat[0, h, : int(n_hat[0, h])].numpy(), np.arange(3, 104))
    ctx.close()


def test_partial_ties_at_the_threshold(cuda_device):
    # duplicated key rows straddle the k-th place: the lower positions must win
    w = small(batch=1, q_heads=1, kv_heads=1, context=2000, top_k=10, heavy_hitters=0)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t = 2001
    a = O.dense_scores(H.np32(q)[0, 0], H.np32(k[0, 0]), t)
    order = O.topk_middle(a, t, 4, 16, 12)
    src = int(order[9])                                    # the 10th best key ...
    dup = [p for p in (100, 900, 1500) if p not in set(order.tolist())]
    for p in dup:
        k[0, 0, p] = k[0, 0, src]                          # ... now appears several times
    ctx = H.make_ctx(w)
    view = P.make_view(k, v, torch.tensor([t], dtype=torch.int32, device=cuda_device), max_seq_len=w.capacity)
    ctx.score_topk(0, 0, q, view, H.make_sched(w, cuda_device), 1)
    s_star, n_star, _, _ = ctx.get_shared_set(0, 1)
    a = O.dense_scores(H.np32(q)[0, 0], H.np32(k[0, 0]), t)
    want = O.topk_middle(a, t, 4, 16, 10)
    assert np.array_equal(s_star[0, 0, :10].numpy(), want)
    assert int(want[-1]) == min(dup + [src])
    ctx.close()


def test_degenerate_lengths(cuda_device):
    # t <= S0 + W (empty middle), t == 1, k larger than the middle range
    w = small(batch=4, q_heads=2, kv_heads=2, context=300, top_k=64, window=16, sinks=4, steps=1)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = torch.tensor([1, 20, 50, 301], dtype=torch.int32)
    ctx = H.make_ctx(w)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    out = torch.empty(4, 2, 128, dtype=torch.bfloat16, device=cuda_device)
    dlt = torch.empty(4, 2, dtype=torch.float32, device=cuda_device)
    sched = H.make_sched(w, cuda_device, flags=P.PRHS_WANT_DELTA, refresh_interval=1)
    ctx.decode_step(0, 0, sched, q, view, 4, out, dlt)
    assert ctx.check() == 0
    idx, cnt = ctx.get_index_set(4)
    qh, y, d = H.np32(q), H.np32(out), H.np32(dlt)
    for b, h in all_units(w):
        t = int(t_host[b])
        Kh, Vh = H.np32(k[b, h]), H.np32(v[b, h])
        a = O.dense_scores(qh[b, h], Kh, t)
        C = O.build_set(t, 4, 16, O.topk_middle(a, t, 4, 16, 64))
        assert np.array_equal(idx[b, h, : int(cnt[b, h])].numpy(), C)
        if t <= 4 + 16 + 64:
            assert len(C) == t and abs(d[b, h]) <= H.DELTA_TOL      # nothing dropped
        y_ref, _ = O.attn_over_set(qh[b, h], Kh, Vh, C)
        assert np.max(np.abs(y[b, h] - y_ref)) <= H.Y_TOL
    ctx.close()


def test_full_budget_equals_dense(cuda_device):
    w = small(batch=1, q_heads=4, kv_heads=2, context=900, top_k=1024, steps=1)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_dev = torch.tensor([901], dtype=torch.int32, device=cuda_device)
    ctx = H.make_ctx(w)
    view = P.make_view(k, v, t_dev, max_seq_len=w.capacity)
    out = torch.empty(1, 4, 128, dtype=torch.bfloat16, device=cuda_device)
    dense = torch.empty_like(out)
    dlt = torch.empty(1, 4, dtype=torch.float32, device=cuda_device)
    ctx.decode_step(0, 0, H.make_sched(w, cuda_device, flags=P.PRHS_WANT_DELTA), q, view, 1, out, dlt)
    ctx.dense_decode_attn(q, view, 1, dense)
    _, cnt = ctx.get_index_set(1)
    assert torch.all(cnt == 901)
    assert torch.max(torch.abs(out.float() - dense.float())) <= 1e-2
    assert torch.max(torch.abs(dlt)) <= H.DELTA_TOL
    ctx.close()


def test_bad_index_is_flagged_not_faulted(cuda_device):
    w = small(batch=1, q_heads=1, kv_heads=1, context=500)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_dev = torch.tensor([400], dtype=torch.int32, device=cuda_device)
    idx = torch.tensor([[[0, 5, 400, -3, 399, 10 ** 6]]], dtype=torch.int32, device=cuda_device)
    cnt = torch.tensor([[6]], dtype=torch.int32, device=cuda_device)
    ctx = H.make_ctx(w)
    out = torch.empty(1, 1, 128, dtype=torch.bfloat16, device=cuda_device)
    ctx.sparse_decode_attn(q, P.make_view(k, v, t_dev), idx, cnt, 1, out)
    with pytest.raises(P.PrhsError) as e:
        ctx.check()
    assert e.value.status == 7
    assert ctx.check() == 0                                  # the flag word was cleared
    y_ref, _ = O.attn_over_set(H.np32(q)[0, 0], H.np32(k[0, 0]), H.np32(v[0, 0]), np.array([0, 5, 399]))
    assert np.max(np.abs(H.np32(out)[0, 0] - y_ref)) <= H.Y_TOL
    ctx.close()


@pytest.mark.parametrize("flags,group_sets", [(0, False), (P.PRHS_CFG_MMA_SYNC_SCORE, False), (P.PRHS_CFG_NO_TMA, False),
                                              (P.PRHS_CFG_TMA_GATHER, False), (0, True),
                                              (P.PRHS_CFG_GROUP_TCGEN05, True)])
def test_bad_page_id_is_flagged_not_dereferenced(cuda_device, flags, group_sets):
    # page ids outside the pool in one sequence's table: every kernel that looks pages up (the three
    # scoring kernels, the gathered attention kernels, the dense baseline) checks the id before it
    # forms an address, skips the page and records the anomaly; the other sequence is untouched
    w = small(batch=2, q_heads=8, kv_heads=2, context=1500, top_k=64, page_size=16, seed=61)
    table, pool = W.make_page_table(w)
    k, v = W.make_kv(w, cuda_device)
    kp, vp = W.to_paged(w, k, table, pool), W.to_paged(w, v, table, pool)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_dev = W.seq_lens_at(w, 0).to(cuda_device)
    bad = table.clone()
    bad[1, 5] = pool + 3
    bad[1, 9] = -1
    sched = H.make_sched(w, cuda_device, flags=P.PRHS_GROUP_SETS if group_sets else 0)
    outs = []
    for tab in (table, bad):
        ctx = H.make_ctx(w, flags=flags)
        view = P.make_view(kp, vp, t_dev, page_table=tab.to(cuda_device), max_seq_len=w.capacity)
        out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
        dense = torch.empty_like(out)
        ctx.decode_step(0, 0, sched, q, view, w.batch, out)
        ctx.dense_decode_attn(q, view, w.batch, dense)
        if tab is table:
            assert ctx.check() == 0
        else:
            with pytest.raises(P.PrhsError) as e:
                ctx.check()
            assert e.value.status == 7 and int(str(e.value).split("0x")[1], 16) & P.PRHS_FLAG_BAD_PAGE
            assert ctx.check() == 0
        outs.append((out.cpu(), dense.cpu()))
        ctx.close()
    assert torch.equal(outs[0][0][0], outs[1][0][0]) and torch.equal(outs[0][1][0], outs[1][1][0])
    assert torch.isfinite(outs[1][1][1].float()).all()


def test_results_are_deterministic(cuda_device):
    w = small(context=2500)
    outs = []
    for _ in range(2):
        torch.cuda.empty_cache()
        k, v = W.make_kv(w, cuda_device)
        q = W.make_queries(w, cuda_device)
        ctx = H.make_ctx(w)
        sched = H.make_sched(w, cuda_device)
        out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
        res = []
        for n in range(w.steps):
            view = P.make_view(k, v, W.seq_lens_at(w, n).to(cuda_device), max_seq_len=w.capacity)
            ctx.decode_step(0, n, sched, q[0, n].contiguous(), view, w.batch, out)
            idx, cnt = ctx.get_index_set(w.batch)
            res.append((out.clone().cpu(), idx.clone(), cnt.clone()))
        outs.append(res)
        ctx.close()
    for a, b in zip(*outs):
        assert torch.equal(a[2], b[2])
        for bb in range(w.batch):
            for h in range(w.q_heads):
                c = int(a[2][bb, h])
                assert torch.equal(a[1][bb, h, :c], b[1][bb, h, :c])
        assert torch.equal(a[0], b[0])


# ------------------------------------------------------------- schedules end to end
def test_schedule_small_every_unit(cuda_device):
    w = small(steps=6, refresh=3, context=2200)
    st = H.run_schedule_parity(w, cuda_device, all_units(w))
    assert st["checked"] == 6 * w.batch * w.q_heads


def test_schedule_cross_layer_groups(cuda_device):
    w = small(layers=4, layer_group=2, steps=4, refresh=2, q_heads=4, kv_heads=1, context=1800, seed=12)
    st = H.run_schedule_parity(w, cuda_device, all_units(w))
    assert st["checked"] == 4 * 4 * w.batch * w.q_heads


@pytest.mark.parametrize("phi,alpha,ls", [(0.7, 1.0, 3), (0.5, 2.0, 1), (0.9, 0.5, 4)])
def test_schedule_with_sliding_window(cuda_device, phi, alpha, ls):
    # progressive sliding attention window on the upper layers, with cross-layer groups:
    # followers clip the leader's shared set by their own, larger window start
    w = small(layers=4, layer_group=2, steps=4, refresh=2, q_heads=4, kv_heads=2, context=2600, seed=14,
              psaw_layer_start=ls, psaw_phi=phi, psaw_alpha=alpha)
    st = H.run_schedule_parity(w, cuda_device, all_units(w))
    assert st["checked"] == 4 * 4 * w.batch * w.q_heads
    assert min(st["set_sizes"]) < max(st["set_sizes"])         # deeper layers attend over fewer rows


@pytest.mark.parametrize("tau,sigma", [(0.8, 0.7), (0.95, 0.3), (-0.5, 1.5), (0.999, 0.05)])
def test_schedule_with_cosine_gate(cuda_device, tau, sigma):
    # per-head sharing decisions on the device: some heads retrieve, others share, inside one
    # launch; followers (second layer of each group) follow their leader's decision
    w = small(layers=4, layer_group=2, steps=9, refresh=4, q_heads=8, kv_heads=2, context=2300, seed=15,
              sigma=sigma, sim_threshold=tau)
    st = H.run_schedule_parity(w, cuda_device, all_units(w))
    assert st["checked"] == 4 * 9 * w.batch * w.q_heads
    leaders_heads = 2 * w.batch * w.q_heads
    assert st["retrievals"] >= 3 * leaders_heads          # steps 0, 4 and 8 always retrieve
    if (tau, sigma) == (0.8, 0.7):
        assert 3 * leaders_heads < st["retrievals"] < 9 * leaders_heads    # a real mix


@pytest.mark.parametrize("tau,sigma,paged", [(0.8, 0.7, False), (0.9, 0.45, True), (0.8, 0.3, False), (0.99, 1.5, False)])
def test_cosine_gate_two_branches(cuda_device, tau, sigma, paged):
    # without the diagnostic a gated step runs as two branches: the attention of the heads that
    # share on a second stream, beside the scoring and selection of the heads that retrieve, whose
    # attention follows (Fig. 6); a real mix, nearly all sharing, all retrieving
    w = small(layers=4, layer_group=2, steps=9, refresh=4, batch=3, q_heads=8, kv_heads=2, context=2500, seed=27,
              min_context=600 if paged else 0, page_size=16 if paged else 0, sigma=sigma, sim_threshold=tau)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, want_delta=False)
    assert st["checked"] == 4 * 9 * w.batch * w.q_heads
    leaders_heads = 2 * w.batch * w.q_heads
    if sigma == 0.7:
        assert 3 * leaders_heads < st["retrievals"] < 9 * leaders_heads
    if sigma == 1.5:
        assert st["retrievals"] == 9 * leaders_heads           # no query is that similar: every head retrieves every step


def test_cosine_gate_two_branches_in_a_cuda_graph(cuda_device):
    # the forked branch is captured with the step and joins it: replays equal the direct calls
    w = small(steps=8, refresh=4, batch=3, q_heads=8, kv_heads=2, context=2400, seed=28, sigma=0.7, sim_threshold=0.8)
    k, v = W.make_kv(w, cuda_device)
    q_all = W.make_queries(w, cuda_device)[0]
    sched = H.make_sched(w, cuda_device)
    views = [P.make_view(k, v, W.seq_lens_at(w, n).to(cuda_device), max_seq_len=w.capacity) for n in range(w.steps)]
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    ctx = H.make_ctx(w)
    direct, needs = [], []
    for n in range(w.steps):
        ctx.decode_step(0, n, sched, q_all[n], views[n], w.batch, out)
        direct.append(out.clone())
        needs.append(ctx.get_gate(0, w.batch)[0].clone())
    assert ctx.check() == 0
    assert 0 < int(torch.stack(needs)[1:4].sum()) < 3 * w.batch * w.q_heads          # a mix inside the block
    side = torch.cuda.Stream()
    outs = [torch.empty_like(out) for _ in range(w.steps)]
    with torch.cuda.stream(side):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for n in range(w.steps):
                ctx.decode_step(0, n, sched, q_all[n], views[n], w.batch, outs[n], stream=torch.cuda.current_stream())
    torch.cuda.synchronize()
    for _ in range(2):
        for o in outs:
            o.zero_()
        g.replay()
        torch.cuda.synchronize()
        for n in range(w.steps):
            assert torch.equal(outs[n], direct[n]), f"step {n}"
    assert ctx.check() == 0
    ctx.close()


def test_cosine_gate_gqa_paged_with_window(cuda_device):
    w = small(layers=2, layer_group=1, steps=6, refresh=3, batch=3, q_heads=8, kv_heads=1, context=2100,
              min_context=500, page_size=16, top_k=0, k_frac=0.03, seed=16, sigma=0.6, sim_threshold=0.85,
              psaw_layer_start=1, psaw_phi=0.8)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=True)
    assert st["checked"] == 2 * 6 * w.batch * w.q_heads


def test_schedule_paged_and_ragged(cuda_device):
    w = small(layers=2, layer_group=2, steps=4, refresh=2, batch=5, q_heads=8, kv_heads=2,
              context=3000, min_context=300, page_size=16, top_k=0, k_frac=0.03, seed=13)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=True)
    assert st["checked"] == 2 * 4 * w.batch * w.q_heads


def test_paged_identity_equals_contiguous(cuda_device):
    w = small(batch=2, q_heads=4, kv_heads=2, context=1000, page_size=16, steps=2)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_dev = W.seq_lens_at(w, 0).to(cuda_device)
    table, pool = W.make_page_table(w)
    kp, vp = W.to_paged(w, k, table, pool), W.to_paged(w, v, table, pool)
    outs = []
    for paged in (False, True):
        ctx = H.make_ctx(w, page_size=16 if paged else 0)
        view = (P.make_view(kp, vp, t_dev, page_table=table.to(cuda_device), max_seq_len=w.capacity)
                if paged else P.make_view(k, v, t_dev, max_seq_len=w.capacity))
        out = torch.empty(2, 4, 128, dtype=torch.bfloat16, device=cuda_device)
        ctx.decode_step(0, 0, H.make_sched(w, cuda_device), q, view, 2, out)
        idx, cnt = ctx.get_index_set(2)
        dense = torch.empty_like(out)
        ctx.dense_decode_attn(q, view, 2, dense)
        outs.append((out.cpu(), idx, cnt, dense.cpu()))
        assert ctx.check() == 0
        ctx.close()
    assert torch.equal(outs[0][2], outs[1][2]) and torch.equal(outs[0][0], outs[1][0])
    assert torch.equal(outs[0][3], outs[1][3])                 # the dense baseline through pages


def test_c1_tiny_exactly_as_specified(cuda_device):
    st = H.run_schedule_parity(W.C1_TINY, cuda_device, all_units(W.C1_TINY))
    assert st["checked"] == 4 * 8
    assert max(st["set_sizes"]) <= 4 + 256 + 2 * 85 + 64


# --------------------------------------------------- full-size configurations, sampled units
def test_c2_full_size_sampled(cuda_device):
    w = W.C2_LLAMA2_7B.scaled(steps=8)
    units = [(0, 0), (3, 17), (7, 31), (5, 8)]
    st = H.run_schedule_parity(w, cuda_device, units)
    assert st["checked"] == 8 * len(units)
    assert not st["select_fallback"]          # the sampled-threshold path handled every unit


def test_c4_long_context_sampled(cuda_device):
    # 128K context: the selection works from global memory (candidates exceed shared memory)
    w = W.C4_LLAMA3_128K.scaled(steps=5)
    units = [(0, 0), (1, 13), (3, 31)]
    st = H.run_schedule_parity(w, cuda_device, units, check_scores=True)
    assert st["checked"] == 5 * len(units)


def test_c3_stack_slice_sampled(cuda_device):
    # the Mistral-shaped stack at full per-layer size, first two layer groups
    w = W.C3_MISTRAL.scaled(layers=8, steps=5, batch=4)
    units = [(0, 0), (2, 21), (3, 31)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1, 3, 4, 7])
    assert st["checked"] == 5 * 5 * len(units)


def test_c3_top_layers_with_sliding_window_sampled(cuda_device):
    # layers 25..32 of a 32-layer stack prune with the paper's defaults (phi 0.7, alpha 1, l_s 24)
    w = W.C3_MISTRAL.scaled(steps=5, batch=2, psaw_layer_start=24)
    units = [(0, 3), (1, 30)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[24, 25, 27, 28, 31])
    assert st["checked"] == 5 * 5 * len(units)


def test_c5_serving_mix_sampled(cuda_device):
    # ragged paged serving mix at reduced batch and layers (full per-sequence sizes)
    w = W.C5_SERVING.scaled(layers=4, steps=5, batch=6)
    units = [(0, 0), (2, 9), (5, 31), (3, 16)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1, 3], paged=True)
    assert st["checked"] == 5 * 3 * len(units)


def test_c3_full_batch_sampled(cuda_device):
    # the Mistral-shaped stack at its real batch of 16 (512 selection units: the 256-thread
    # launch of the selection kernel), two layer groups, leaders and followers
    w = W.C3_MISTRAL.scaled(layers=8, steps=6)
    units = [(0, 0), (5, 9), (11, 22), (15, 31)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1, 3, 4, 7])
    assert st["checked"] == 6 * 5 * len(units)
    assert not st["select_fallback"]


def test_c5_full_batch_sampled(cuda_device):
    # the serving mix at its real batch of 64 ragged, paged sequences (2048 selection units,
    # k_b = floor(0.03 N_b)): the leader and one follower of a layer group
    w = W.C5_SERVING.scaled(layers=4, steps=5)
    units = [(0, 0), (17, 9), (40, 31), (63, 16), (29, 4)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1], paged=True)
    assert st["checked"] == 5 * 2 * len(units)
    assert not st["select_fallback"]


# ----------------------------------------- the paper's operator-benchmark shapes (Sec. 5.4, Table 3)
@pytest.mark.parametrize("batch,n,s", [(16, 4096, 16), (8, 1024, 8)])
def test_table3_operator_shapes(cuda_device, batch, n, s):
    # budgets of Sec. 5.3.2 (C_sink 16, C_local 64, k = n/8 - 80 = 432 at 4k), blocks of s steps:
    # one whole block and the start of the next
    from paper_2602_08329_b200 import operator_latency as OL
    w = OL.table3_workload(batch, n, s).scaled(steps=s + 2)
    assert (w.sinks, w.window) == (16, 64) and w.top_k == (432 if n == 4096 else 48)
    g = np.random.default_rng(batch + n)
    units = sorted({(int(g.integers(batch)), int(g.integers(32))) for _ in range(20)})
    st = H.run_schedule_parity(w, cuda_device, units)
    assert st["checked"] == (s + 2) * len(units)
    assert st["retrievals"] == 2 * len(units) and not st["select_fallback"]
    assert max(st["set_sizes"]) <= 16 + w.top_k + 2 * (w.top_k // 3) + 64


# --------------------------------------------------- retrieval scoring without the TMA kernels
@pytest.mark.parametrize("paged", [False, True])
def test_score_ring_small_every_unit(cuda_device, paged):
    # PRHS_CFG_NO_TMA: the key stream goes through the cp.async ring kernel (what the library
    # falls back to by itself when the driver offers no tensor-map encoder)
    w = small(layers=2, layer_group=2, steps=4, refresh=2, batch=3, q_heads=8, kv_heads=2, context=2700,
              min_context=400 if paged else 0, page_size=16 if paged else 0, seed=17)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, ctx_over=dict(flags=P.PRHS_CFG_NO_TMA))
    assert st["checked"] == 2 * 4 * w.batch * w.q_heads


def test_score_ring_c2_sampled(cuda_device):
    w = W.C2_LLAMA2_7B.scaled(steps=5)
    units = [(0, 0), (6, 30), (2, 11)]
    st = H.run_schedule_parity(w, cuda_device, units, ctx_over=dict(flags=P.PRHS_CFG_NO_TMA))
    assert st["checked"] == 5 * len(units) and not st["select_fallback"]


def test_score_kernels_logits_agree(cuda_device):
    # the three scoring kernels (tcgen05, mma.sync behind TMA, mma.sync behind cp.async) on the same
    # inputs: same logits (each within the tolerance of the oracle, so within twice that of each
    # other) and the same log-sum-exp
    w = small(batch=2, q_heads=8, kv_heads=2, context=5000, top_k=64, seed=18)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    view = P.make_view(k, v, W.seq_lens_at(w, 0).to(cuda_device), max_seq_len=w.capacity)
    res = []
    for flags in (0, P.PRHS_CFG_MMA_SYNC_SCORE, P.PRHS_CFG_NO_TMA):
        ctx = H.make_ctx(w, flags=flags)
        lse = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
        ctx.score_topk(0, 0, q, view, H.make_sched(w, cuda_device), w.batch, out_lse_full=lse)
        assert ctx.check() == 0
        res.append((ctx.get_scores(w.batch)[:, :, : w.context + 1], lse.cpu()))
        ctx.close()
    for other in res[1:]:
        assert torch.allclose(res[0][0], other[0], atol=2 * H.LOGIT_ATOL, rtol=2 * H.LOGIT_RTOL)
        assert torch.allclose(res[0][1], other[1], atol=1e-4)


# ------------------------------------------------ retrieval scoring on the tcgen05 tensor cores
def test_score_tcgen05_logits_against_oracle(cuda_device):
    # the default scoring kernel (tcgen05) on the smallest useful case: several 128-key tiles and a
    # ragged last one per split, grouped-query heads (4 per KV head), logits and log-sum-exp element
    # by element
    w = small(batch=2, q_heads=8, kv_heads=2, context=5000, top_k=64, seed=41)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = W.seq_lens_at(w, 0)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    ctx = H.make_ctx(w)
    lse = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
    ctx.score_topk(0, 0, q, view, H.make_sched(w, cuda_device), w.batch, out_lse_full=lse)
    assert ctx.check() == 0
    scores = ctx.get_scores(w.batch)
    kn, qn = k.float().cpu().numpy().astype(np.float64), q.float().cpu().numpy().astype(np.float64)
    gq = w.q_heads // w.kv_heads
    for b in range(w.batch):
        t = int(t_host[b])
        for h in range(w.q_heads):
            ref = O.dense_scores(qn[b, h], kn[b, h // gq], t)
            got = scores[b, h, :t].numpy().astype(np.float64)
            assert np.allclose(got, ref, atol=H.LOGIT_ATOL, rtol=H.LOGIT_RTOL), (b, h, np.abs(got - ref).max())
            assert abs(float(lse[b, h]) - O.logsumexp(ref)) < 1e-4
    ctx.close()


@pytest.mark.parametrize("paged", [False, True])
def test_score_tcgen05_small_every_unit(cuda_device, paged):
    w = small(layers=2, layer_group=2, steps=4, refresh=2, batch=3, q_heads=8, kv_heads=2, context=2700,
              min_context=400 if paged else 0, page_size=16 if paged else 0, seed=42)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged)
    assert st["checked"] == 2 * 4 * w.batch * w.q_heads


def test_score_tcgen05_group_of_sixteen_and_single_head(cuda_device):
    # the widest group the MMA tile holds (16 heads on its 16 columns) and multi-head attention
    # (one live column)
    for q_heads, kv_heads in ((16, 1), (4, 4)):
        w = small(batch=2, q_heads=q_heads, kv_heads=kv_heads, context=1500, steps=3, refresh=2, seed=43)
        st = H.run_schedule_parity(w, cuda_device, all_units(w))
        assert st["checked"] == 3 * w.batch * w.q_heads


# ------------------------------------- retrieval scoring with mma.sync consumer warps (an option)
@pytest.mark.parametrize("paged", [False, True])
def test_score_mma_sync_small_every_unit(cuda_device, paged):
    # PRHS_CFG_MMA_SYNC_SCORE: the TMA-staged kernel whose eight consumer warps run m16n8k16 MMAs
    w = small(layers=2, layer_group=2, steps=4, refresh=2, batch=3, q_heads=8, kv_heads=2, context=2700,
              min_context=400 if paged else 0, page_size=16 if paged else 0, seed=44)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged,
                               ctx_over=dict(flags=P.PRHS_CFG_MMA_SYNC_SCORE))
    assert st["checked"] == 2 * 4 * w.batch * w.q_heads


def test_score_mma_sync_c2_sampled(cuda_device):
    w = W.C2_LLAMA2_7B.scaled(steps=5)
    units = [(0, 0), (7, 31), (3, 12)]
    st = H.run_schedule_parity(w, cuda_device, units, ctx_over=dict(flags=P.PRHS_CFG_MMA_SYNC_SCORE))
    assert st["checked"] == 5 * len(units) and not st["select_fallback"]


def test_score_mma_sync_c5_sampled(cuda_device):
    # paged, ragged, grouped queries at a reduced batch
    w = W.C5_SERVING.scaled(layers=4, steps=2, batch=6)
    units = [(0, 0), (5, 31), (2, 9), (3, 16)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1], paged=True,
                               ctx_over=dict(flags=P.PRHS_CFG_MMA_SYNC_SCORE))
    assert st["checked"] == 2 * 2 * len(units)


# ------------------------------------------ gathered attention with rows by TMA gather (an option)
@pytest.mark.parametrize("paged", [False, True])
def test_tma_gather_attention_small_every_unit(cuda_device, paged):
    # PRHS_CFG_TMA_GATHER: the same attention with tile::gather4 copies instead of cp.async (off by
    # default, it measured slower); ragged tails, empty middle sets, out-of-tensor filler rows
    w = small(layers=2, layer_group=2, steps=4, refresh=2, batch=3, q_heads=8, kv_heads=2, context=2900,
              min_context=200 if paged else 0, page_size=16 if paged else 0, seed=31, psaw_layer_start=2)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged,
                               ctx_over=dict(flags=P.PRHS_CFG_TMA_GATHER))
    assert st["checked"] == 2 * 4 * w.batch * w.q_heads


def test_tma_gather_attention_given_sets_and_bad_index(cuda_device):
    w = small(q_heads=8, kv_heads=4, context=3000, seed=32)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = torch.tensor([2999, 1234], dtype=torch.int32)
    g = np.random.default_rng(32)
    cap = 700
    idx = torch.full((w.batch, w.q_heads, cap), -7, dtype=torch.int32)
    cnt = torch.zeros(w.batch, w.q_heads, dtype=torch.int32)
    sets = {}
    sizes = [0, 1, 15, 16, 17, 255, 256, 257, 511, 640, 700, 33, 300, 64, 129, 5]
    for b, h in all_units(w):
        n = min(sizes[(b * w.q_heads + h) % len(sizes)], int(t_host[b]))
        C = np.sort(g.permutation(int(t_host[b]))[:n])
        sets[(b, h)] = C
        idx[b, h, :n] = torch.from_numpy(C.astype(np.int32))
        cnt[b, h] = n
    ctx = H.make_ctx(w, flags=P.PRHS_CFG_TMA_GATHER)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    lse = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
    ctx.sparse_decode_attn(q, view, idx.to(cuda_device), cnt.to(cuda_device), w.batch, out, lse)
    assert ctx.check() == 0
    y, ls, qh = H.np32(out), H.np32(lse), H.np32(q)
    for (b, h), C in sets.items():
        y_ref, lse_ref = O.attn_over_set(qh[b, h], H.np32(k[b, h // 2]), H.np32(v[b, h // 2]), C)
        assert np.max(np.abs(y[b, h] - y_ref)) <= H.Y_TOL
        assert (ls[b, h] == -math.inf) if len(C) == 0 else abs(ls[b, h] - lse_ref) <= 1e-4
    bad = idx.clone()
    bad[1, 2, 1] = 10 ** 6                                  # skipped (a zero-filled row, masked) and flagged
    ctx.sparse_decode_attn(q, view, bad.to(cuda_device), cnt.to(cuda_device), w.batch, out, lse)
    with pytest.raises(P.PrhsError) as e:
        ctx.check()
    assert e.value.status == 7
    C = np.delete(sets[(1, 2)], 1)
    y_ref, _ = O.attn_over_set(qh[1, 2], H.np32(k[1, 1]), H.np32(v[1, 1]), C)
    assert np.max(np.abs(H.np32(out)[1, 2] - y_ref)) <= H.Y_TOL
    ctx.close()


# ----------------------------------------------------------- measurement support: the gather probe
def test_gather_probe_variants_run_clean(cuda_device):
    # the bare row gather behind `python -m paper_2602_08329_b200.gather_ceiling`: every copy
    # mechanism over real index lists (ragged tails, an empty list), no anomaly; then a list
    # with an out-of-range entry, which is replaced and flagged, not read
    w = small(batch=3, q_heads=8, kv_heads=2, context=4000, seed=29)
    k, v = W.make_kv(w, cuda_device)
    t_dev = W.seq_lens_at(w, 0).to(cuda_device)
    view = P.make_view(k, v, t_dev, max_seq_len=w.capacity)
    g = np.random.default_rng(29)
    cap = 900
    idx = torch.zeros(w.batch, w.q_heads, cap, dtype=torch.int32)
    cnt = torch.zeros(w.batch, w.q_heads, dtype=torch.int32)
    for b, h in all_units(w):
        n = 0 if (b, h) == (1, 1) else int(g.integers(1, cap + 1))
        idx[b, h, :n] = torch.from_numpy(np.sort(g.permutation(4000)[:n]).astype(np.int32))
        cnt[b, h] = n
    idx, cnt = idx.to(cuda_device), cnt.to(cuda_device)
    ctx = H.make_ctx(w)
    for variant in range(4):
        ctx.gather_probe(variant, view, idx, cnt, w.batch)
        assert ctx.check() == 0, variant
    bad = idx.clone()
    bad[2, 3, 0] = 10 ** 6
    for variant in range(4):
        ctx.gather_probe(variant, view, bad, cnt, w.batch)
        with pytest.raises(P.PrhsError) as e:
            ctx.check()
        assert e.value.status == 7, variant
    with pytest.raises(P.PrhsError):
        ctx.gather_probe(4, view, idx, cnt, w.batch)
    ctx.close()


# ------------------------------------------------------------------- host-buffer entry point
@pytest.mark.parametrize("pinned", [True, False])
def test_decode_step_host_buffers(cuda_device, pinned):
    # pinned buffers are read and written by the kernels directly, pageable ones are copied
    pin = (lambda x: x.pin_memory()) if pinned else (lambda x: x)
    w = small(steps=3, refresh=2, context=1200)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)
    k2, v2 = k.clone(), v.clone()
    ctx_a, ctx_b = H.make_ctx(w), H.make_ctx(w)
    ctx_cs = [H.make_ctx(w)]
    sched = H.make_sched(w, cuda_device)
    out_a = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    t_dev = torch.zeros(w.batch, dtype=torch.int32, device=cuda_device)
    for n in range(w.steps):
        t_host = W.seq_lens_at(w, n)
        ctx_a.decode_step(0, n, sched, q[0, n].contiguous(), P.make_view(k, v, t_host.to(cuda_device)),
                          w.batch, out_a)
        # the host entry point appends the new token's rows itself: blank them first
        pos = (t_host - 1).long()
        bi = torch.arange(w.batch)
        new_k, new_v = k[bi, :, pos].cpu().contiguous(), v[bi, :, pos].cpu().contiguous()
        k2[bi, :, pos] = 0
        v2[bi, :, pos] = 0
        host_out = pin(torch.zeros(w.batch, w.q_heads, 128, dtype=torch.bfloat16))
        ctx_b.decode_step_host(0, n, sched, pin(q[0, n].cpu().contiguous()), pin(new_k), pin(new_v),
                               pin(t_host.contiguous()), P.make_view(k2, v2, t_dev), w.batch, host_out)
        assert torch.equal(t_dev.cpu(), t_host)
        if pinned:      # the variant that does not synchronise: valid once the stream has caught up
            k3, v3, t3 = k2.clone(), v2.clone(), torch.zeros_like(t_dev)
            k3[bi, :, pos] = 0
            out_async = pin(torch.zeros(w.batch, w.q_heads, 128, dtype=torch.bfloat16))
            held = (pin(q[0, n].cpu().contiguous()), pin(new_k), pin(new_v), pin(t_host.contiguous()))
            ctx_cs[0].decode_step_host(0, n, sched, *held, P.make_view(k3, v3, t3), w.batch, out_async,
                                       sync=False)
            torch.cuda.synchronize()        # the host buffers are held until here
            assert torch.equal(out_async, host_out) and torch.equal(k3, k)
        assert torch.equal(host_out, out_a.cpu())
    assert torch.equal(k2, k) and torch.equal(v2, v)
    ctx_a.close(); ctx_b.close(); ctx_cs[0].close()


# ------------------------------------------------------------------------- host validation
def test_host_side_errors(cuda_device):
    w = small()
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_dev = W.seq_lens_at(w, 0).to(cuda_device)
    view = P.make_view(k, v, t_dev)
    ctx = H.make_ctx(w)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)

    def status(fn):
        with pytest.raises(P.PrhsError) as e:
            fn()
        return e.value.status

    good = H.make_sched(w, cuda_device)
    assert status(lambda: ctx.decode_step(0, 1, good, q, view, w.batch, out)) == 5       # no anchor yet
    assert status(lambda: ctx.decode_step(0, 0, good, q, view, w.batch + 1, out)) == 6   # batch
    assert status(lambda: ctx.decode_step(0, 0, H.make_sched(w, cuda_device, top_k=w.top_k + 1), q, view,
                                          w.batch, out)) == 6
    assert status(lambda: ctx.decode_step(0, 0, H.make_sched(w, cuda_device, refresh_interval=0), q, view,
                                          w.batch, out)) == 1
    assert status(lambda: ctx.decode_step(5, 0, good, q, view, w.batch, out)) == 1       # layer range
    assert status(lambda: ctx.decode_step(0, 0, good, None, view, w.batch, out)) == 1    # NULL q
    with pytest.raises(P.PrhsError) as e:
        P.Context(1, 1, 4, 2, 1000, 16, 16, 4, head_dim=64)
    assert e.value.status == 2
    ctx.decode_step(0, 0, good, q, view, w.batch, out)                                   # still usable
    assert ctx.check() == 0
    ctx.close()


def test_host_entry_point_rejects_rows_beyond_the_cache(cuda_device):
    """A context dimensioned for longer sequences than the cache holds: the host-buffer entry
    point must refuse a length whose new row would land outside the cache, before it writes
    anything (the cache and the device lengths stay as they were)."""
    w = small(steps=2)
    k, v = W.make_kv(w, cuda_device)
    k0, v0 = k.clone(), v.clone()
    ctx = H.make_ctx(w, max_context=w.capacity + 4000)
    sched = H.make_sched(w, cuda_device)
    t_dev = torch.full((w.batch,), 7, dtype=torch.int32, device=cuda_device)
    g = torch.Generator().manual_seed(5)
    hq = torch.randn(w.batch, w.q_heads, 128, generator=g).to(torch.bfloat16).pin_memory()
    hk = torch.randn(w.batch, w.kv_heads, 128, generator=g).to(torch.bfloat16).pin_memory()
    hout = torch.zeros(w.batch, w.q_heads, 128, dtype=torch.bfloat16).pin_memory()

    def status(t_list, view, **kw):
        ht = torch.tensor(t_list, dtype=torch.int32).pin_memory()
        with pytest.raises(P.PrhsError) as e:
            ctx.decode_step_host(0, 0, kw.get("sched", sched), hq, hk, hk, ht, view, w.batch, hout)
        return e.value.status

    full = P.make_view(k, v, t_dev)                                # max_seq_len 0: the context's maximum
    assert status([w.capacity + 1, 10], full) == 6                 # beyond the (b, kvh) slice (strides)
    assert status([10, w.capacity + 3999], full) == 6
    short = P.make_view(k, v, t_dev, max_seq_len=1000)
    assert status([1001, 10], short) == 6                          # beyond the capacity the view declares
    assert status([0, 10], full) == 1
    assert status([10, 10], full, sched=H.make_sched(w, cuda_device, top_k=w.top_k + 1)) == 6   # bad schedule
    torch.cuda.synchronize()
    assert torch.equal(k, k0) and torch.equal(v, v0) and bool((t_dev == 7).all())   # nothing was written
    ht = torch.tensor([w.capacity, 1000], dtype=torch.int32).pin_memory()           # the largest legal length
    ctx.decode_step_host(0, 0, sched, hq, hk, hk, ht, full, w.batch, hout)
    assert ctx.check() == 0 and torch.equal(t_dev.cpu(), ht)
    ctx.close()


def test_default_dilation_count_must_fit_the_context(cuda_device):
    # m = floor(k / 3) by default: a context created for fewer dilated winners refuses the schedule
    # instead of truncating the dilated set
    w = small()
    ctx = H.make_ctx(w, max_dilate_m=3)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    view = P.make_view(k, v, W.seq_lens_at(w, 0).to(cuda_device))
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    with pytest.raises(P.PrhsError) as e:
        ctx.decode_step(0, 0, H.make_sched(w, cuda_device), q, view, w.batch, out)      # 48 / 3 = 16 > 3
    assert e.value.status == 6
    ctx.decode_step(0, 0, H.make_sched(w, cuda_device, dilate_m=3), q, view, w.batch, out)
    assert ctx.check() == 0
    ctx.close()


@pytest.mark.gpu
def test_radius_sweep_cells_small():
    """The sweep script's cell on a small shape: the s = 1 row is the per-step oracle selector
    (beta 0, coverage 1, whatever r), and sharing can only lose coverage."""
    from paper_2602_08329_b200 import radius_sweep as RS
    dev = torch.device("cuda:0")
    w = W.C1_TINY.scaled(steps=8, halo=0.7, q_scale=3.0, sigma=0.3, heavy_hitters=32)
    k, v = W.make_kv(w, dev)
    q = W.make_queries(w, dev)
    c1 = RS.run_cell(w, dev, k, v, q, 1, 2)
    assert c1["beta_max"] == 0.0 and c1["cov_min"] == 1.0
    assert c1["size"] <= w.sinks + w.top_k + w.window
    c4 = RS.run_cell(w, dev, k, v, q, 4, 1)
    assert c4["cov_mean"] <= 1.0 and c4["size"] > c1["size"]
    assert abs(c4["delta1_mean"] - c1["delta_mean"]) < 1e-5      # delta* does not depend on the cell
    c40 = RS.run_cell(w, dev, k, v, q, 4, 0)
    assert c40["beta_mean"] >= -1e-5        # without dilation a shared set never beats the step's own top-k
    assert c40["cov_mean"] <= c4["cov_mean"] + 1e-9


# ------------------------------------------------ labelled variant: one index set per KV head
@pytest.mark.gpu
@pytest.mark.parametrize("hq,hkv,paged", [(8, 2, False), (16, 1, False), (12, 4, True), (4, 4, False)])
def test_group_sets_schedule(cuda_device, hq, hkv, paged):
    # group-shared sets (ranking by the group's maximum logit), cross-layer groups and a
    # sliding window on the top layers; the (4, 4) case has one head per KV head, where the
    # variant is the method itself
    w = small(layers=4, layer_group=2, steps=5, refresh=2, q_heads=hq, kv_heads=hkv, context=2400, seed=41,
              psaw_layer_start=3, page_size=16 if paged else 0)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, group_sets=True)
    assert st["checked"] == 4 * 5 * w.batch * w.q_heads
    assert not st["select_fallback"]


@pytest.mark.gpu
def test_group_sets_rejects_cosine_gate(cuda_device):
    w = small(q_heads=8, kv_heads=2, sim_threshold=0.8)
    ctx = H.make_ctx(w)
    sched = H.make_sched(w, cuda_device, flags=P.PRHS_GROUP_SETS)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    view = P.make_view(k, v, W.seq_lens_at(w, 0).to(cuda_device), max_seq_len=w.capacity)
    with pytest.raises(P.PrhsError) as e:
        ctx.decode_step(0, 0, sched, q[0, 0].contiguous(), view, w.batch, out)
    assert e.value.status == 2       # PRHS_ERR_UNSUPPORTED
    ctx.close()


@pytest.mark.gpu
def test_group_sets_c3_slice_sampled(cuda_device):
    # the Mistral-shaped stack at full per-layer size with group-shared sets
    w = W.C3_MISTRAL.scaled(layers=8, steps=5, batch=4)
    units = [(0, 0), (0, 3), (2, 21), (3, 31)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1, 3, 4], group_sets=True)
    assert st["checked"] == 4 * 5 * len(units)


# ------------------------- the group-shared variant's attention on the tcgen05 tensor cores
@pytest.mark.gpu
def test_group_sets_tcgen05_one_small_case(cuda_device):
    # PRHS_CFG_GROUP_TCGEN05, smallest useful case: lists of a few 128-row tiles with a ragged last
    # one, four heads per KV head, retrieval and sharing steps
    w = small(layers=1, steps=3, refresh=2, batch=2, q_heads=8, kv_heads=2, context=2400, top_k=300, seed=51)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), group_sets=True,
                               ctx_over=dict(flags=P.PRHS_CFG_GROUP_TCGEN05))
    assert st["checked"] == 3 * w.batch * w.q_heads


@pytest.mark.gpu
@pytest.mark.parametrize("hq,hkv,paged", [(8, 2, False), (16, 1, False), (12, 4, True), (4, 4, False)])
def test_group_sets_tcgen05_schedule(cuda_device, hq, hkv, paged):
    w = small(layers=4, layer_group=2, steps=5, refresh=2, q_heads=hq, kv_heads=hkv, context=2400, seed=52,
              psaw_layer_start=3, page_size=16 if paged else 0)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, group_sets=True,
                               ctx_over=dict(flags=P.PRHS_CFG_GROUP_TCGEN05))
    assert st["checked"] == 4 * 5 * w.batch * w.q_heads


@pytest.mark.gpu
@pytest.mark.parametrize("paged", [False, True])
def test_group_sets_tcgen05_more_units_than_sms(cuda_device, paged):
    # more (sequence, KV head) units than the GPU has SMs: the library launches the kernel in its second
    # shape (one softmax group and one loader set per CTA, two CTAs per SM)
    w = small(layers=1, steps=3, refresh=2, batch=24, q_heads=16, kv_heads=8, context=900, top_k=200,
              min_context=300, page_size=16 if paged else 0, seed=53)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, group_sets=True,
                               ctx_over=dict(flags=P.PRHS_CFG_GROUP_TCGEN05))
    assert st["checked"] == 3 * w.batch * w.q_heads


@pytest.mark.gpu
def test_group_sets_tcgen05_full_shapes_sampled(cuda_device):
    # the Mistral-shaped stack, the 128K shape (several splits per unit: partials and the merge) and the
    # ragged paged serving mix
    over = dict(flags=P.PRHS_CFG_GROUP_TCGEN05)
    w = W.C3_MISTRAL.scaled(layers=8, steps=5, batch=4)
    st = H.run_schedule_parity(w, cuda_device, [(0, 0), (0, 3), (2, 21), (3, 31)], layers=[0, 1, 3, 4],
                               group_sets=True, ctx_over=over)
    assert st["checked"] == 4 * 5 * 4
    w = W.C4_LLAMA3_128K.scaled(steps=5)
    st = H.run_schedule_parity(w, cuda_device, [(0, 0), (1, 13), (3, 31)], group_sets=True, ctx_over=over)
    assert st["checked"] == 5 * 3 and not st["select_fallback"]
    w = W.C5_SERVING.scaled(layers=4, steps=5, batch=6)
    st = H.run_schedule_parity(w, cuda_device, [(0, 0), (2, 9), (5, 31), (3, 16)], layers=[0, 1, 3], paged=True,
                               group_sets=True, ctx_over=over)
    assert st["checked"] == 5 * 3 * 4


# ------------------------------------------- selection kernel: the rarely taken configurations
@pytest.mark.gpu
@pytest.mark.parametrize("case", ["large_k_bitonic", "one_bitmap", "k_above_candidates", "list_everything"])
def test_selection_shared_memory_layouts(cuda_device, case):
    """The selection kernel sizes its shared memory from the context's maxima and switches
    layout with them: a budget so large that the list cannot hold a second sort buffer (the
    in-place bitonic sort takes over), a context so long that only one position bitmap fits
    (two sweeps), k above the middle range (everything is a winner), and a range short enough
    to list every candidate without sampling."""
    if case == "large_k_bitonic":
        w, over = small(context=30000, top_k=5000, batch=1, q_heads=2, kv_heads=2, seed=61), {}
    elif case == "one_bitmap":
        w, over = small(context=20000, top_k=300, batch=1, q_heads=2, kv_heads=1, seed=62), dict(max_context=1_000_000)
    elif case == "k_above_candidates":
        w, over = small(context=900, top_k=2000, batch=2, seed=63), {}
    else:
        w, over = small(context=3000, top_k=64, batch=2, seed=64), {}
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = W.seq_lens_at(w, 0)
    ctx = H.make_ctx(w, **over)
    sched = H.make_sched(w, cuda_device)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    ctx.score_topk(0, 0, q, view, sched, w.batch)
    assert ctx.check() == 0                         # in particular: no fallback to the generic path
    s_star, n_star, s_hat, n_hat = ctx.get_shared_set(0, w.batch)
    qh = H.np32(q)
    gq = w.q_heads // w.kv_heads
    for b, h in all_units(w):
        t = int(t_host[b])
        a = O.dense_scores(qh[b, h], H.np32(k[b, h // gq]), t)
        want = O.topk_middle(a, t, w.sinks, w.window, w.top_k)
        got = s_star[b, h, : int(n_star[b, h])].numpy().astype(np.int64)
        H.check_topk_legal(O.rank_logits(a), got, want, f"{case} unit ({b},{h})")
        hat = s_hat[b, h, : int(n_hat[b, h])].numpy().astype(np.int64)
        assert np.array_equal(hat, O.dilate(got, w.top_k // 3, 1, t))
    # and a whole step over that set
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    ctx.decode_step(0, 0, sched, q, view, w.batch, out)
    idx, cnt = ctx.get_index_set(w.batch)
    assert ctx.check() == 0
    for b, h in all_units(w)[:2]:
        C = idx[b, h, : int(cnt[b, h])].numpy().astype(np.int64)
        y, _ = O.attn_over_set(qh[b, h], H.np32(k[b, h // gq]), H.np32(v[b, h // gq]), C)
        assert np.max(np.abs(H.np32(out)[b, h] - y)) <= H.Y_TOL
    ctx.close()


# ------------------------------------------------------------------ failure path, without a fault
@pytest.mark.gpu
def test_bounded_wait_gives_up_and_context_survives(cuda_device):
    """A wait on a barrier that nothing completes runs out of its budget, the kernel reports
    it through the flag word, and the same context then decodes as if nothing had happened."""
    w = small(steps=2, context=1800)
    ctx = H.make_ctx(w)
    assert ctx.selftest_wait(500_000) == 1
    with pytest.raises(P.PrhsError) as e:
        ctx.check()
    assert e.value.status == 7                                # PRHS_ERR_DEVICE_FLAG
    assert ctx.check() == 0                                   # reported once, then cleared
    with pytest.raises(P.PrhsError):
        ctx.selftest_wait(10**12)                             # budgets are capped
    # the same context decodes, bit for bit like a fresh one
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    sched = H.make_sched(w, cuda_device)
    view = P.make_view(k, v, W.seq_lens_at(w, 0).to(cuda_device), max_seq_len=w.capacity)
    outs = []
    for c in (ctx, H.make_ctx(w)):
        out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
        c.decode_step(0, 0, sched, q, view, w.batch, out)
        assert c.check() == 0
        outs.append(out.cpu())
        c.close()
    assert torch.equal(outs[0], outs[1])
    st = H.run_schedule_parity(w, cuda_device, all_units(w))
    assert st["checked"] == 2 * w.batch * w.q_heads


@pytest.mark.gpu
def test_contexts_of_different_sizes_side_by_side(cuda_device):
    """A large context, then a small one, then the large one is used: kernel attributes set at
    creation must not depend on which context was created last."""
    big = small(context=30000, top_k=5000, batch=1, q_heads=2, kv_heads=2, seed=71)
    little = small(context=1500, seed=72)
    ctx_big, ctx_little = H.make_ctx(big), H.make_ctx(little)
    for w, ctx in ((big, ctx_big), (little, ctx_little), (big, ctx_big)):
        k, v = W.make_kv(w, cuda_device)
        q = W.make_queries(w, cuda_device)[0, 0].contiguous()
        view = P.make_view(k, v, W.seq_lens_at(w, 0).to(cuda_device), max_seq_len=w.capacity)
        out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
        ctx.decode_step(0, 0, H.make_sched(w, cuda_device), q, view, w.batch, out)
        assert ctx.check() == 0
        idx, cnt = ctx.get_index_set(w.batch)
        C = idx[0, 0, : int(cnt[0, 0])].numpy().astype(np.int64)
        y, _ = O.attn_over_set(H.np32(q)[0, 0], H.np32(k[0, 0]), H.np32(v[0, 0]), C)
        assert np.max(np.abs(H.np32(out)[0, 0] - y)) <= H.Y_TOL
    ctx_big.close(); ctx_little.close()


@pytest.mark.gpu
def test_non_finite_keys_stay_contained(cuda_device):
    """NaN / Inf inputs are outside the method's definition; the library must still return, keep
    every index in range, and leave the heads of other KV heads exactly as they are."""
    w = small(context=6000, batch=2, q_heads=4, kv_heads=2, steps=2, seed=81)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)
    k_bad = k.clone()
    k_bad[0, 0, 100] = float("nan")
    k_bad[0, 0, 2000:2010] = float("inf")
    k_bad[0, 0, 3000] = float("-inf")
    outs = []
    for keys in (k, k_bad):
        ctx = H.make_ctx(w)
        sched = H.make_sched(w, cuda_device)
        res = []
        for n in range(w.steps):
            view = P.make_view(keys, v, W.seq_lens_at(w, n).to(cuda_device), max_seq_len=w.capacity)
            out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
            ctx.decode_step(0, n, sched, q[0, n].contiguous(), view, w.batch, out)
            idx, cnt = ctx.get_index_set(w.batch)
            assert ctx.check() & ~P.PRHS_FLAG_SELECT_FALLBACK == 0
            t = W.seq_lens_at(w, n)
            for b in range(w.batch):
                for h in range(w.q_heads):
                    c = idx[b, h, : int(cnt[b, h])]
                    assert int(cnt[b, h]) <= ctx.index_capacity and bool((c >= 0).all()) and bool((c < int(t[b])).all())
            res.append(out.cpu())
        outs.append(res)
        ctx.close()
    gq = w.q_heads // w.kv_heads
    for a, b_ in zip(*outs):
        assert torch.equal(a[1], b_[1])                 # the other sequence
        assert torch.equal(a[0, gq:], b_[0, gq:])       # the other KV head of the same sequence


# ------------------------------------------------------------ seeded random schedules end to end
def _random_workload(seed):
    g = np.random.default_rng(seed)
    hkv = int(g.choice([1, 2, 4]))
    gq = int(g.choice([1, 2, 4, 8]))
    layer_group = int(g.choice([1, 2]))
    refresh = int(g.choice([1, 2, 3, 4]))
    context = int(g.integers(300, 5000))
    paged = bool(g.integers(0, 2))
    ragged = bool(g.integers(0, 2))
    kw = dict(layers=2 * layer_group, layer_group=layer_group, batch=int(g.integers(1, 4)), q_heads=hkv * gq,
              kv_heads=hkv, context=context, steps=int(g.integers(2, 6)), refresh=refresh,
              top_k=int(g.choice([0, 1, 7, 64, 200, 700])), window=int(g.choice([0, 1, 16, 100, 600])),
              sinks=int(g.choice([0, 1, 4, 33])), dilate_r=int(g.choice([0, 1, 2])),
              heavy_hitters=int(g.choice([0, 8])), decay_span=int(g.choice([0, 64])), seed=1000 + seed,
              halo=float(g.choice([0.0, 0.7])), q_scale=float(g.choice([1.0, 3.0])),
              page_size=16 if paged else 0, min_context=max(40, context // 3) if ragged else 0,
              psaw_layer_start=int(g.choice([0, 0, 1, 2])))
    if kw["heavy_hitters"] and context - kw["window"] - kw["decay_span"] - kw["sinks"] < 16:
        kw["heavy_hitters"] = 0
    return small(f"random{seed}", **kw), paged, bool(g.integers(0, 2)) and gq > 1


@pytest.mark.gpu
@pytest.mark.parametrize("seed", list(range(14)))
def test_random_schedules(cuda_device, seed):
    """Seeded random shapes and budgets (zero and oversized budgets, windows longer than the
    context, one or several layer groups, paged and ragged caches, sliding windows, group-shared
    sets): every unit of every (layer, step) against the oracle."""
    w, paged, group_sets = _random_workload(seed)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, group_sets=group_sets)
    assert st["checked"] == w.layers * w.steps * w.batch * w.q_heads


@pytest.mark.gpu
@pytest.mark.parametrize("seed", list(range(100, 112)))
def test_random_schedules_kernel_options(cuda_device, seed):
    """The same random shapes through the optional kernels, in turn: scoring with mma.sync behind the TMA
    ring, scoring behind the cp.async ring, the TMA row-gather attention, and the group-shared variant's
    attention on tcgen05."""
    w, paged, group_sets = _random_workload(seed)
    flags = [P.PRHS_CFG_MMA_SYNC_SCORE, P.PRHS_CFG_NO_TMA, P.PRHS_CFG_TMA_GATHER, P.PRHS_CFG_GROUP_TCGEN05][seed % 4]
    if flags == P.PRHS_CFG_GROUP_TCGEN05:
        group_sets = True
        if w.q_heads == w.kv_heads:
            w = w.scaled(q_heads=2 * w.q_heads)
    elif flags == P.PRHS_CFG_TMA_GATHER:
        group_sets = False
    st = H.run_schedule_parity(w, cuda_device, all_units(w), paged=paged, group_sets=group_sets,
                               ctx_over=dict(flags=flags))
    assert st["checked"] == w.layers * w.steps * w.batch * w.q_heads


@pytest.mark.gpu
def test_group_sets_stage_calls(cuda_device):
    """The stage-by-stage entry points with group-shared sets: prhs_score_topk hands every head
    of a group the group's S* (ranked by the group maximum), prhs_build_index_set the group's
    set, and the explicit-list attention over it equals the fused step."""
    w = small(q_heads=8, kv_heads=2, context=3000, top_k=96, seed=91)
    gq = 4
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_host = W.seq_lens_at(w, 0)
    ctx = H.make_ctx(w)
    sched = H.make_sched(w, cuda_device, flags=P.PRHS_GROUP_SETS)
    view = P.make_view(k, v, t_host.to(cuda_device), max_seq_len=w.capacity)
    oi = torch.empty(w.batch, w.q_heads, w.top_k, dtype=torch.int32, device=cuda_device)
    oc = torch.empty(w.batch, w.q_heads, dtype=torch.int32, device=cuda_device)
    ol = torch.empty(w.batch, w.q_heads, dtype=torch.float32, device=cuda_device)
    ctx.score_topk(0, 0, q, view, sched, w.batch, oi, oc, ol)
    assert ctx.check() == 0
    qh = H.np32(q)
    for b in range(w.batch):
        t = int(t_host[b])
        for kvh in range(w.kv_heads):
            heads = [O.dense_scores(qh[b, kvh * gq + j], H.np32(k[b, kvh]), t) for j in range(gq)]
            ag = O.group_logits(heads)
            want = O.topk_middle(ag, t, w.sinks, w.window, w.top_k)
            for j in range(gq):
                h = kvh * gq + j
                got = oi[b, h, : int(oc[b, h])].cpu().numpy().astype(np.int64)
                H.check_topk_legal(ag, got, want, f"unit ({b},{h})")
                assert torch.equal(oi[b, h], oi[b, kvh * gq])
                assert abs(float(ol[b, h]) - O.logsumexp(heads[j])) <= 1e-4      # log-sum-exp stays per head
    cap = ctx.index_capacity
    idx = torch.empty(w.batch, w.q_heads, cap, dtype=torch.int32, device=cuda_device)
    cnt = torch.empty(w.batch, w.q_heads, dtype=torch.int32, device=cuda_device)
    ctx.build_index_set(0, 0, sched, view, w.batch, idx, cnt)
    out_a = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    out_b = torch.empty_like(out_a)
    ctx.sparse_decode_attn(q, view, idx, cnt, w.batch, out_a)
    ctx.decode_step(0, 0, sched, q, view, w.batch, out_b)
    assert ctx.check() == 0
    for b in range(w.batch):
        for h in range(w.q_heads):
            assert int(cnt[b, h]) == int(cnt[b, h - h % gq])
            assert torch.equal(idx[b, h, : int(cnt[b, h])], idx[b, h - h % gq, : int(cnt[b, h])])
    assert float((out_a.float() - out_b.float()).abs().max()) <= 2e-2     # different kernels, same set
    ctx.close()


@pytest.mark.gpu
def test_decode_step_in_a_cuda_graph(cuda_device):
    """prhs_decode_step only enqueues work (no allocation, no synchronisation), so a step can be
    captured into a CUDA graph and replayed: lengths and queries live in device buffers that the
    caller updates between replays.  A retrieval step and a sharing step are captured once and
    replayed over two blocks; results equal the direct calls bit for bit."""
    w = small(steps=8, refresh=4, context=2600, seed=95)
    k, v = W.make_kv(w, cuda_device)
    q_all = W.make_queries(w, cuda_device)[0]
    sched = H.make_sched(w, cuda_device)
    direct = []
    ctx = H.make_ctx(w)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    for n in range(w.steps):
        view = P.make_view(k, v, W.seq_lens_at(w, n).to(cuda_device), max_seq_len=w.capacity)
        ctx.decode_step(0, n, sched, q_all[n].contiguous(), view, w.batch, out)
        direct.append(out.clone())
    assert ctx.check() == 0
    ctx.close()

    ctx = H.make_ctx(w)
    q_buf = torch.empty_like(q_all[0]).contiguous()
    t_buf = torch.zeros(w.batch, dtype=torch.int32, device=cuda_device)
    out_g = torch.empty_like(out)
    view = P.make_view(k, v, t_buf, max_seq_len=w.capacity)
    side = torch.cuda.Stream()
    graphs = {}
    with torch.cuda.stream(side):
        for kind, step in (("retrieve", 0), ("share", 1)):
            q_buf.copy_(q_all[step]); t_buf.copy_(W.seq_lens_at(w, step).to(cuda_device))
            ctx.decode_step(0, step, sched, q_buf, view, w.batch, out_g, stream=side)     # warm-up outside capture
            side.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                ctx.decode_step(0, step, sched, q_buf, view, w.batch, out_g, stream=torch.cuda.current_stream())
            graphs[kind] = g
    torch.cuda.synchronize()
    for n in range(w.steps):
        q_buf.copy_(q_all[n]); t_buf.copy_(W.seq_lens_at(w, n).to(cuda_device))
        graphs["retrieve" if n % w.refresh == 0 else "share"].replay()
        torch.cuda.synchronize()
        assert torch.equal(out_g, direct[n]), f"step {n}"
    assert ctx.check() == 0
    ctx.close()


@pytest.mark.gpu
def test_group_sets_long_and_paged_sampled(cuda_device):
    # the group-shared variant at the 128K shape and at the ragged paged serving mix
    w = W.C4_LLAMA3_128K.scaled(steps=5)
    units = [(0, 0), (1, 13), (3, 31)]
    st = H.run_schedule_parity(w, cuda_device, units, group_sets=True)
    assert st["checked"] == 5 * len(units) and not st["select_fallback"]
    w = W.C5_SERVING.scaled(layers=4, steps=5, batch=6)
    units = [(0, 0), (2, 9), (5, 31), (3, 16)]
    st = H.run_schedule_parity(w, cuda_device, units, layers=[0, 1, 3], paged=True, group_sets=True)
    assert st["checked"] == 5 * 3 * len(units)


# ----------------------------------------------------------------- checkpoint of the set state
@pytest.mark.gpu
@pytest.mark.parametrize("gated", [False, True])
def test_state_export_import_resumes_bit_for_bit(cuda_device, gated):
    """Export the shared-set state in the middle of a block, import it into a fresh context and
    continue there: outputs and index sets equal those of the uninterrupted context, for the
    fixed schedule (with layer groups) and for the cosine gate (block history included)."""
    w = small(layers=4, layer_group=2, steps=9, refresh=4, q_heads=8, kv_heads=2, context=2100, seed=97,
              sigma=0.7 if gated else 0.05, sim_threshold=0.8 if gated else None)
    kv = {l: (k, v) for l, k, v in W.make_layer_kv(w, cuda_device)}
    q = W.make_queries(w, cuda_device)
    sched = H.make_sched(w, cuda_device)
    ctx_a, ctx_b = H.make_ctx(w), None
    out_a = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    out_b = torch.empty_like(out_a)
    cut = 6          # after step 5: the second block is two steps old
    for n in range(w.steps):
        view_t = W.seq_lens_at(w, n).to(cuda_device)
        if n == cut:
            blob = ctx_a.state_export()
            assert blob.numel() == ctx_a.lib.prhs_state_bytes(ctx_a.h)
            ctx_b = H.make_ctx(w)
            ctx_b.state_import(blob)
            with pytest.raises(P.PrhsError):                 # another configuration refuses the buffer
                other = H.make_ctx(w.scaled(top_k=w.top_k + 8))
                try:
                    other.state_import(blob)
                finally:
                    other.close()
        for l in range(w.layers):
            view = P.make_view(kv[l][0], kv[l][1], view_t, max_seq_len=w.capacity)
            ctx_a.decode_step(l, n, sched, q[l, n].contiguous(), view, w.batch, out_a)
            if ctx_b is not None:
                ctx_b.decode_step(l, n, sched, q[l, n].contiguous(), view, w.batch, out_b)
                assert torch.equal(out_a, out_b), f"layer {l} step {n}"
                ia, ca = ctx_a.get_index_set(w.batch)
                ib, cb = ctx_b.get_index_set(w.batch)
                assert torch.equal(ca, cb)
                for b in range(w.batch):
                    for h in range(w.q_heads):
                        assert torch.equal(ia[b, h, : int(ca[b, h])], ib[b, h, : int(cb[b, h])])
    assert ctx_a.check() == 0 and ctx_b.check() == 0
    ctx_a.close(); ctx_b.close()


@pytest.mark.gpu
def test_validate_index_lists(cuda_device):
    w = small(context=2000, seed=98)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    t_dev = W.seq_lens_at(w, 0).to(cuda_device)
    view = P.make_view(k, v, t_dev, max_seq_len=w.capacity)
    ctx = H.make_ctx(w)
    sched = H.make_sched(w, cuda_device)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    ctx.decode_step(0, 0, sched, q, view, w.batch, out)
    cap = ctx.index_capacity
    idx = torch.empty(w.batch, w.q_heads, cap, dtype=torch.int32, device=cuda_device)
    cnt = torch.empty(w.batch, w.q_heads, dtype=torch.int32, device=cuda_device)
    ctx.build_index_set(0, 0, sched, view, w.batch, idx, cnt)
    nbad, marks = ctx.validate_index_lists(view, idx, cnt, w.batch)
    assert nbad == 0 and int(marks.sum()) == 0                   # the library's own lists are clean
    bad = idx.clone()
    bad[0, 1, 5] = bad[0, 1, 4]                                   # a duplicate
    bad[1, 0, 3], bad[1, 0, 2] = idx[1, 0, 2].item(), idx[1, 0, 3].item()    # out of order
    bad[1, 3, 0] = -7                                             # out of range
    cnt2 = cnt.clone()
    cnt2[0, 2] = cap + 1                                          # longer than the stride
    nbad, marks = ctx.validate_index_lists(view, bad, cnt2, w.batch)
    assert nbad == 4
    assert marks.tolist() == [[0, 1, 1, 0], [1, 0, 0, 1]]
    ctx.decode_step(0, 1, sched, q, P.make_view(k, v, W.seq_lens_at(w, 1).to(cuda_device), max_seq_len=w.capacity),
                    w.batch, out)                                 # the scratch it borrowed is back in order
    assert ctx.check() == 0
    ctx.close()


@pytest.mark.gpu
def test_maximum_context_length(cuda_device):
    """One sequence at the library's largest context (2^20 positions, 4096 winners): the sparse
    sample, the single-bitmap layout and a million-row tensor map, against the oracle."""
    n = (1 << 20) - 8
    w = small("max_context", context=n, steps=2, refresh=2, batch=1, q_heads=2, kv_heads=1, top_k=4096,
              window=256, sinks=4, heavy_hitters=64, decay_span=512, seed=99)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), check_scores=True)
    assert st["checked"] == 2 * 2 and not st["select_fallback"]


@pytest.mark.gpu
@pytest.mark.parametrize("anchor,m,r", [(True, -1, 1), (False, 0, 1), (True, 5, 2), (False, 48, 2), (True, 3, 0)])
def test_dilation_options(cuda_device, anchor, m, r):
    # the other reading of who attends over the dilated set (the retrieving call too), and an
    # explicit number of dilated winners instead of k/3 (none, a few, all of them)
    w = small(layers=2, layer_group=2, steps=5, refresh=2, q_heads=4, kv_heads=2, context=2300, seed=33, dilate_r=r,
              halo=0.7)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), dilate_anchor=anchor, dilate_m=m)
    assert st["checked"] == 2 * 5 * w.batch * w.q_heads


@pytest.mark.gpu
def test_per_kernel_profile_counts(cuda_device):
    w = small(steps=4, refresh=2)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0]
    ctx = H.make_ctx(w)
    sched = H.make_sched(w, cuda_device)
    out = torch.empty(w.batch, w.q_heads, 128, dtype=torch.bfloat16, device=cuda_device)
    n0 = ctx.launch_count
    ctx.profile_begin()
    for n in range(w.steps):
        view = P.make_view(k, v, W.seq_lens_at(w, n).to(cuda_device), max_seq_len=w.capacity)
        ctx.decode_step(0, n, sched, q[n].contiguous(), view, w.batch, out)
    prof = ctx.profile_end()
    assert {name: cnt for name, (ms, cnt) in prof.items() if cnt} == {"score": 2, "select": 2, "attn_sparse": 4}
    assert all(ms > 0 for ms, cnt in prof.values() if cnt)
    assert ctx.launch_count - n0 == 8
    ctx.close()


@pytest.mark.gpu
@pytest.mark.parametrize("gated", [False, True])
def test_context_larger_than_the_workload(cuda_device, gated):
    # a context dimensioned for more sequences, layers, longer contexts and larger budgets than
    # the calls use: state and workspaces are indexed by the configured maxima
    w = small(layers=2, layer_group=2, steps=5, refresh=2, q_heads=8, kv_heads=2, context=1900, seed=44,
              sim_threshold=0.8 if gated else None, sigma=0.6 if gated else 0.05)
    over = dict(max_batch=w.batch + 3, num_layers=6, max_context=w.capacity + 5000, max_k=w.top_k + 100,
                max_window=w.window + 9, max_sinks=w.sinks + 3, max_dilate_r=2, min_layer_group=1,
                max_block_sets=4 if gated else 1)
    st = H.run_schedule_parity(w, cuda_device, all_units(w), ctx_over=over, group_sets=not gated)
    assert st["checked"] == 2 * 5 * w.batch * w.q_heads
