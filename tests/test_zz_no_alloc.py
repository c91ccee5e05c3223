"""The allocation-free sparse-attention entry point against the context-based one.

Some callers of the library cannot allocate device memory (a frozen budget, a framework that
owns the heap), so they cannot create a context.  For them the library offers
prhs_sparse_decode_attn_noalloc, whose split-K scratch is a fixed array inside the library.
This file runs last (pytest collects it after the other test files): it calls the new entry
point through the C ABI twice in a row -- the second call finds the first call's leftovers in
the shared array -- and checks both results against the existing entry point, and a sample of
units against the CPU oracle's attention over the same lists (contiguous and paged caches).
"""
import numpy as np
import pytest
import torch

from oracle import prhs_oracle as O
from paper_2602_08329_b200 import binding as P
from paper_2602_08329_b200 import workloads as W
from tests import harness as H

pytestmark = pytest.mark.gpu


def _case(device, seed, batch, q_heads, kv_heads, context, max_list):
    w = W.Workload("noalloc", layers=1, batch=batch, q_heads=q_heads, kv_heads=kv_heads, context=context,
                   steps=2, top_k=64, window=16, sinks=4, refresh=1, heavy_hitters=4, decay_span=32, seed=seed)
    k, v = W.make_kv(w, device)
    q = W.make_queries(w, device)[0, 0].contiguous()
    t_host = torch.tensor([context + 1 - 37 * b for b in range(batch)], dtype=torch.int32)
    g = np.random.default_rng(seed)
    idx = torch.zeros(batch, q_heads, max_list, dtype=torch.int32)
    cnt = torch.zeros(batch, q_heads, dtype=torch.int32)
    for b in range(batch):
        for h in range(q_heads):
            n = int(g.integers(max_list // 2, max_list + 1)) if (b + h) % 5 else 0
            idx[b, h, :n] = torch.from_numpy(np.sort(g.permutation(int(t_host[b]))[:n]).astype(np.int32))
            cnt[b, h] = n
    return w, k, v, q, t_host.to(device), idx.to(device), cnt.to(device)


def _check_against_oracle(units, q, k, v, idx, cnt, gq, out, lse):
    """out / lse of the sampled (b, h) units against attention over the same list (Def. 3.1)."""
    qh, y, ls = H.np32(q), H.np32(out), H.np32(lse)
    for b, h in units:
        C = idx[b, h, : int(cnt[b, h])].cpu().numpy().astype(np.int64)
        y_ref, lse_ref = O.attn_over_set(qh[b, h], H.np32(k[b, h // gq]), H.np32(v[b, h // gq]), C)
        assert np.max(np.abs(y[b, h] - y_ref)) <= H.Y_TOL, (b, h)
        if len(C):
            assert abs(ls[b, h] - lse_ref) <= 1e-4, (b, h)
        else:
            assert ls[b, h] == -np.inf and np.all(y[b, h] == 0), (b, h)


def test_noalloc_matches_context_entry_point_twice(cuda_device):
    # few units with long lists: the split count is above one, so the static scratch
    # (partials and tickets) is really used
    w, k, v, q, t_dev, idx, cnt = _case(cuda_device, 3, batch=2, q_heads=4, kv_heads=2, context=9000,
                                        max_list=6000)
    view = P.make_view(k, v, t_dev, max_seq_len=w.capacity)
    ctx = H.make_ctx(w)
    ref = torch.empty(2, 4, 128, dtype=torch.bfloat16, device=cuda_device)
    ref_lse = torch.empty(2, 4, dtype=torch.float32, device=cuda_device)
    ctx.sparse_decode_attn(q, view, idx, cnt, 2, ref, ref_lse)
    assert ctx.check() == 0
    # a second, different problem between the two calls leaves other contents in the array
    w2, k2, v2, q2, t2, idx2, cnt2 = _case(cuda_device, 4, batch=3, q_heads=8, kv_heads=8, context=5000,
                                           max_list=3000)
    view2 = P.make_view(k2, v2, t2, max_seq_len=w2.capacity)
    ctx2 = H.make_ctx(w2)
    ref2 = torch.empty(3, 8, 128, dtype=torch.bfloat16, device=cuda_device)
    ref2_lse = torch.empty(3, 8, dtype=torch.float32, device=cuda_device)
    ctx2.sparse_decode_attn(q2, view2, idx2, cnt2, 3, ref2, ref2_lse)
    for call in range(2):
        out = torch.full_like(ref, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        P.sparse_decode_attn_noalloc(q, view, idx, cnt, 2, 4, 2, out, lse)
        out2 = torch.full_like(ref2, float("nan"))
        lse2 = torch.full_like(ref2_lse, float("nan"))
        P.sparse_decode_attn_noalloc(q2, view2, idx2, cnt2, 3, 8, 8, out2, lse2)
        torch.cuda.synchronize()
        for got, want, gl, wl in ((out, ref, lse, ref_lse), (out2, ref2, lse2, ref2_lse)):
            assert torch.max(torch.abs(got.float() - want.float())).item() <= H.Y_TOL, f"call {call}"
            fin = torch.isfinite(wl)
            assert torch.equal(torch.isfinite(gl), fin)
            assert torch.max(torch.abs(gl[fin] - wl[fin])).item() <= 1e-4, f"call {call}"
        # and against the definition itself, on a sample of units (an empty list among them)
        _check_against_oracle([(0, 0), (0, 1), (1, 3), (1, 2)], q, k, v, idx, cnt, 2, out, lse)
        _check_against_oracle([(0, 5), (2, 7), (1, 4)], q2, k2, v2, idx2, cnt2, 1, out2, lse2)
    assert P.noalloc_check() == 0
    ctx.close()
    ctx2.close()


def test_noalloc_paged_cache_and_skipped_indices(cuda_device):
    """The same entry point over a paged cache, twice in a row, against the context-based call
    and the oracle; then a list with entries outside [0, t_b): they are skipped, not read, and
    the shared anomaly word reports it once."""
    batch, hq, hkv = 3, 8, 2
    w = W.Workload("noalloc_paged", layers=1, batch=batch, q_heads=hq, kv_heads=hkv, context=7000, steps=2,
                   top_k=64, window=16, sinks=4, refresh=1, heavy_hitters=4, decay_span=32, seed=8,
                   page_size=16, min_context=2500)
    k, v = W.make_kv(w, cuda_device)
    q = W.make_queries(w, cuda_device)[0, 0].contiguous()
    table, pool = W.make_page_table(w)
    kp, vp = W.to_paged(w, k, table, pool), W.to_paged(w, v, table, pool)
    t_host = W.seq_lens_at(w, 0)
    g = np.random.default_rng(8)
    cap = 4000
    idx = torch.zeros(batch, hq, cap, dtype=torch.int32)
    cnt = torch.zeros(batch, hq, dtype=torch.int32)
    for b in range(batch):
        for h in range(hq):
            n = int(g.integers(cap // 3, min(cap, int(t_host[b])) + 1))
            idx[b, h, :n] = torch.from_numpy(np.sort(g.permutation(int(t_host[b]))[:n]).astype(np.int32))
            cnt[b, h] = n
    idx, cnt = idx.to(cuda_device), cnt.to(cuda_device)
    view = P.make_view(kp, vp, t_host.to(cuda_device), page_table=table.to(cuda_device), max_seq_len=w.capacity)
    ctx = H.make_ctx(w)
    ref = torch.empty(batch, hq, 128, dtype=torch.bfloat16, device=cuda_device)
    ref_lse = torch.empty(batch, hq, dtype=torch.float32, device=cuda_device)
    ctx.sparse_decode_attn(q, view, idx, cnt, batch, ref, ref_lse)
    assert ctx.check() == 0
    for call in range(2):
        out = torch.full_like(ref, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        P.sparse_decode_attn_noalloc(q, view, idx, cnt, batch, hq, hkv, out, lse)
        torch.cuda.synchronize()
        assert torch.max(torch.abs(out.float() - ref.float())).item() <= H.Y_TOL, f"call {call}"
        assert torch.max(torch.abs(lse - ref_lse)).item() <= 1e-4, f"call {call}"
        _check_against_oracle([(0, 0), (1, 5), (2, 7)], q, k, v, idx, cnt, hq // hkv, out, lse)
    assert P.noalloc_check() == 0
    # entries outside [0, t_b) in one unit's list
    bad = idx.clone()
    keep = int(cnt[1, 2])
    bad[1, 2, 3] = int(t_host[1])           # one past the end
    bad[1, 2, 10] = -5
    bad[1, 2, 11] = 10 ** 7
    out = torch.full_like(ref, float("nan"))
    lse = torch.full_like(ref_lse, float("nan"))
    P.sparse_decode_attn_noalloc(q, view, bad, cnt, batch, hq, hkv, out, lse)
    with pytest.raises(P.PrhsError) as e:
        P.noalloc_check()
    assert e.value.status == 7                                   # PRHS_ERR_DEVICE_FLAG, reported ...
    assert P.noalloc_check() == 0                                # ... once, then cleared
    good = np.delete(idx[1, 2, :keep].cpu().numpy().astype(np.int64), [3, 10, 11])
    y_ref, lse_ref = O.attn_over_set(H.np32(q)[1, 2], H.np32(k[1, 0]), H.np32(v[1, 0]), good)
    assert np.max(np.abs(H.np32(out)[1, 2] - y_ref)) <= H.Y_TOL
    assert abs(float(lse[1, 2]) - lse_ref) <= 1e-4
    others = torch.ones(batch, hq, dtype=torch.bool)
    others[1, 2] = False
    assert torch.max(torch.abs(out.float() - ref.float())[others.to(cuda_device)]).item() <= H.Y_TOL
    ctx.close()


def test_noalloc_rejects_shapes_beyond_the_static_array(cuda_device):
    w, k, v, q, t_dev, idx, cnt = _case(cuda_device, 5, batch=1, q_heads=2, kv_heads=1, context=600,
                                        max_list=200)
    view = P.make_view(k, v, t_dev)
    out = torch.empty(1, 2, 128, dtype=torch.bfloat16, device=cuda_device)
    with pytest.raises(P.PrhsError) as e:
        # 33 * 32 = 1056 units > PRHS_NOALLOC_MAX_UNITS; rejected before anything is launched
        P.sparse_decode_attn_noalloc(q, view, idx, cnt, 33, 32, 32, out)
    assert e.value.status == 6 and "PRHS_NOALLOC_MAX_UNITS" in str(e.value)
    with pytest.raises(P.PrhsError) as e:
        P.sparse_decode_attn_noalloc(q, view, idx, cnt, 1, 3, 2, out)          # Hkv does not divide Hq
    assert e.value.status == 1
