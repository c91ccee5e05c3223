"""Seeded synthetic inputs for the sparse decode-attention path.

This module only draws random tensors; it holds none of the method's arithmetic (no
scores, no selection, no attention) and is the one module the CUDA tests and the CPU
oracle's tests both use.  A tensor is generated once, on one device, and the other side
receives a copy of it: inputs are bit-identical on both sides by construction.

The tensors stand in for the long-context decode workloads of the paper's efficiency
study (LLaMA-2-7B-Chat, Sec. 5.4) and of the LLaMA-3 / Mistral models it evaluates
(Sec. 5.1); real prompts, datasets and weights are not used.

Recipe (all bf16, head_dim 128):
  keys      k ~ N(0,1) i.i.d.; the `decay_span` positions just before the initial context
            end are scaled by `decay_scale` (distance-decay bias); `heavy_hitters`
            positions per (sequence, KV head), drawn without replacement from the middle
            of the context, are scaled by `heavy_scale` (high-norm keys); with
            `halo` > 0 each heavy hitter's neighbours at distance j <= 2 additionally
            receive halo**j times the heavy hitter's key (position-clustered variant).
  values    v ~ N(0,1) i.i.d.
  layers    K_{l+1} = 0.9 K_l + 0.44 N(0,1) before the scalings above; the same
            recurrence for the queries; values independent per layer.
  queries   q_0 ~ q_scale N(0,1); q_{n+1} = q_n + sigma N(0,1) per (sequence, head),
            accumulated in fp32 and rounded to bf16 per step.
The cache is pre-filled to `context + steps` positions; at decode step n the visible
length is context + n + 1 (the current token included).
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch

HEAD_DIM = 128


@dataclass(frozen=True)
class Workload:
    name: str
    layers: int
    batch: int
    q_heads: int
    kv_heads: int
    context: int            # N: initial context length (max over the batch if ragged)
    steps: int              # T decode steps
    top_k: int
    window: int
    sinks: int
    refresh: int            # s
    layer_group: int = 1    # G_L
    dilate_r: int = 1
    heavy_hitters: int = 64
    heavy_scale: float = 4.0
    decay_span: int = 512
    decay_scale: float = 1.5
    sigma: float = 0.05
    q_scale: float = 1.0
    halo: float = 0.0
    seed: int = 0
    page_size: int = 0      # 0 = contiguous cache, 16 = paged
    min_context: int = 0    # > 0: ragged contexts uniform in [min_context, context]
    k_frac: float = 0.0     # > 0: per-sequence k = floor(k_frac * N_b)
    psaw_layer_start: int = 0   # l_s of the sliding attention window (1-based); 0 = off
    psaw_phi: float = 0.7
    psaw_alpha: float = 1.0
    sim_threshold: float | None = None   # tau of the cosine gate; None = fixed sharing schedule

    @property
    def capacity(self) -> int:
        return self.context + self.steps

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five configurations named by the benchmark definition (C1..C5).
C1_TINY = Workload("c1_tiny", layers=1, batch=1, q_heads=8, kv_heads=2, context=4096, steps=4,
                   top_k=256, window=64, sinks=4, refresh=2, heavy_hitters=16, decay_span=0,
                   decay_scale=1.0, seed=0)
C2_LLAMA2_7B = Workload("c2_llama2_7b_layer", layers=1, batch=8, q_heads=32, kv_heads=32,
                        context=32768, steps=16, top_k=1024, window=128, sinks=4, refresh=4,
                        seed=2)
C3_MISTRAL = Workload("c3_mistral_7b_stack", layers=32, batch=16, q_heads=32, kv_heads=8,
                      context=32768, steps=32, top_k=1024, window=128, sinks=4, refresh=4,
                      layer_group=4, seed=3)
C4_LLAMA3_128K = Workload("c4_llama3_8b_128k", layers=1, batch=4, q_heads=32, kv_heads=8,
                          context=131072, steps=16, top_k=2048, window=256, sinks=4, refresh=4,
                          seed=4)
C5_SERVING = Workload("c5_serving_mix", layers=32, batch=64, q_heads=32, kv_heads=8,
                      context=65536, steps=64, top_k=0, window=128, sinks=4, refresh=4,
                      layer_group=4, seed=5, page_size=16, min_context=4096, k_frac=0.03)

CONFIGS = {w.name: w for w in (C1_TINY, C2_LLAMA2_7B, C3_MISTRAL, C4_LLAMA3_128K, C5_SERVING)}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def context_lengths(w: Workload) -> torch.Tensor:
    """Initial context N_b per sequence (CPU int32 [B])."""
    if w.min_context <= 0:
        return torch.full((w.batch,), w.context, dtype=torch.int32)
    g = _gen(w.seed * 1000003 + 11, "cpu")
    return torch.randint(w.min_context, w.context + 1, (w.batch,), generator=g, dtype=torch.int32)


def top_k_per_seq(w: Workload) -> torch.Tensor | None:
    """k_b = floor(k_frac * N_b), fixed from the initial context (CPU int32 [B]) or None."""
    if w.k_frac <= 0:
        return None
    return torch.floor(context_lengths(w).to(torch.float64) * w.k_frac).to(torch.int32)


def heavy_positions(w: Workload) -> torch.Tensor:
    """Heavy-hitter positions per (sequence, KV head): CPU int64 [B][Hkv][heavy_hitters].

    Drawn without replacement from [sinks, N_b - window - decay_span); identical in every
    layer.  Generated on the CPU so that both sides can inspect them.
    """
    g = _gen(w.seed * 1000003 + 7, "cpu")
    n_ctx = context_lengths(w)
    out = torch.zeros(w.batch, w.kv_heads, max(w.heavy_hitters, 1), dtype=torch.int64)
    for b in range(w.batch):
        lo, hi = w.sinks, max(w.sinks + 1, int(n_ctx[b]) - w.window - w.decay_span)
        for h in range(w.kv_heads):
            perm = torch.randperm(hi - lo, generator=g)[: w.heavy_hitters] + lo
            out[b, h, : len(perm)] = perm
    return out[:, :, : w.heavy_hitters]


def _shape_keys(w: Workload, base: torch.Tensor, heavy: torch.Tensor, n_ctx: torch.Tensor) -> torch.Tensor:
    """Apply halo, heavy-hitter and distance-decay scalings to fp32 keys [B][Hkv][cap][d]."""
    k = base.clone()
    dev = base.device
    B, H = w.batch, w.kv_heads
    if w.heavy_hitters > 0:
        hp = heavy.to(dev)
        bi = torch.arange(B, device=dev)[:, None, None].expand_as(hp)
        hi_ = torch.arange(H, device=dev)[None, :, None].expand_as(hp)
        hk = base[bi, hi_, hp] * w.heavy_scale
        k[bi, hi_, hp] = hk
        if w.halo > 0:
            for j in (1, 2):
                for sgn in (-1, 1):
                    pos = (hp + sgn * j).clamp_(0, base.shape[2] - 1)
                    k[bi, hi_, pos] = k[bi, hi_, pos] + (w.halo ** j) * hk
    if w.decay_span > 0 and w.decay_scale != 1.0:
        pos = torch.arange(base.shape[2], device=dev)[None, :]
        n = n_ctx.to(dev)[:, None].to(torch.int64)
        recent = (pos >= n - w.decay_span) & (pos < n)
        k = torch.where(recent[:, None, :, None], k * w.decay_scale, k)
    return k


def make_layer_kv(w: Workload, device, layers=None):
    """Yield (layer, K, V) with K, V bf16 [B][Hkv][capacity][128] on `device`.

    Layers are produced in order (the inter-layer recurrence needs the previous layer's
    unscaled keys), one at a time so that a caller can bound its memory.
    """
    g = _gen(w.seed * 1000003 + 1, device)
    heavy = heavy_positions(w) if w.heavy_hitters > 0 else None
    n_ctx = context_lengths(w)
    shape = (w.batch, w.kv_heads, w.capacity, HEAD_DIM)
    base = None
    want = set(range(w.layers)) if layers is None else set(layers)
    for layer in range(max(want) + 1):
        noise = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        base = noise if base is None else base.mul_(0.9).add_(noise, alpha=0.44)
        v = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        if layer in want:
            yield layer, _shape_keys(w, base, heavy, n_ctx).to(torch.bfloat16), v.to(torch.bfloat16)
        del noise, v


def make_kv(w: Workload, device, layer: int = 0):
    """K, V of one layer (bf16 [B][Hkv][capacity][128])."""
    for l, k, v in make_layer_kv(w, device, layers=[layer]):
        return k, v
    raise ValueError(layer)


def make_queries(w: Workload, device) -> torch.Tensor:
    """Queries bf16 [layers][steps][B][Hq][128]: Lipschitz drift over steps, AR(1) over layers."""
    g = _gen(w.seed * 1000003 + 3, device)
    shape = (w.batch, w.q_heads, HEAD_DIM)
    out = torch.empty((w.layers, w.steps) + shape, dtype=torch.bfloat16, device=device)
    q0 = None
    for layer in range(w.layers):
        n0 = torch.randn(shape, generator=g, device=device, dtype=torch.float32) * w.q_scale
        q0 = n0 if q0 is None else 0.9 * q0 + 0.44 * n0
        q = q0.clone()
        for n in range(w.steps):
            if n > 0:
                q = q + w.sigma * torch.randn(shape, generator=g, device=device, dtype=torch.float32)
            out[layer, n] = q.to(torch.bfloat16)
    return out


def seq_lens_at(w: Workload, step: int) -> torch.Tensor:
    """Visible length t_b at decode step n: N_b + n + 1 (CPU int32 [B])."""
    return context_lengths(w) + (step + 1)


def make_page_table(w: Workload):
    """Random page table for a paged cache: CPU int32 [B][max_pages], plus the pool size.

    Every sequence owns ceil(capacity_b / page_size) distinct pages; page ids are a random
    permutation of the pool.
    """
    assert w.page_size > 0
    g = _gen(w.seed * 1000003 + 5, "cpu")
    n_ctx = context_lengths(w)
    need = [(int(n) + w.steps + w.page_size - 1) // w.page_size for n in n_ctx]
    pool = sum(need)
    perm = torch.randperm(pool, generator=g).to(torch.int32)
    table = torch.zeros(w.batch, max(need), dtype=torch.int32)
    o = 0
    for b, n in enumerate(need):
        table[b, :n] = perm[o:o + n]
        o += n
    return table, pool


def to_paged(w: Workload, x: torch.Tensor, table: torch.Tensor, pool: int) -> torch.Tensor:
    """Scatter a contiguous [B][Hkv][cap][128] cache into pages [pool][Hkv][page][128]."""
    ps = w.page_size
    B, H, cap, d = x.shape
    out = torch.zeros(pool, H, ps, d, dtype=x.dtype, device=x.device)
    n_ctx = context_lengths(w)
    for b in range(B):
        n_pages = (int(n_ctx[b]) + w.steps + ps - 1) // ps
        rows = min(n_pages * ps, cap)
        src = torch.zeros(H, n_pages * ps, d, dtype=x.dtype, device=x.device)
        src[:, :rows] = x[b, :, :rows]
        ids = table[b, :n_pages].to(x.device).long()
        out[ids] = src.view(H, n_pages, ps, d).permute(1, 0, 2, 3)
    return out
