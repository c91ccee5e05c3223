"""CPU oracle for the Pre-hoc Sparsity (PrHS / CIS) sparse decode-attention path.

TEST INFRASTRUCTURE ONLY.  This module is a plain, slow, obviously-correct restatement
of what the path computes, written from the paper's definitions.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no code with
the CUDA library and never imports it; the CUDA library never imports this module.

Precision.  The paper does not fix a precision.  Inputs are bf16 values widened exactly
to float64; every dot product, softmax sum and mass is formed in float64.  The one place
where floating point decides an integer -- the top-k ranking -- is taken on the logits
rounded once to float32, the precision the CUDA path ranks in.

Indexing.  0-based, half-open.  `t` is the number of cached positions visible to the
current query, the current token (position t-1) included.  The paper is 1-based; its
three groups (Sec. 4.1 "Selection Criteria") become
    sinks  = [0, S0)        middle candidates = [S0, t-W)        local = [t-W, t)
which are pairwise disjoint.

Every function below is pinned by tests/test_oracle_pins.py against closed forms,
brute-force enumeration, textbook identities and the paper's inequalities, except
cross-layer reuse (`PrhsOracle` with layer_group > 1), which the paper only motivates
and does not define: that part is "parity unpinned" beyond structural invariants.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np

__all__ = [
    "dense_scores", "rank_logits", "softmax_full", "logsumexp", "dense_attention",
    "topk_middle", "dilate", "build_set", "attn_over_set", "retained_mass",
    "dropped_mass", "delta_from_lse", "mi_bound_g", "coverage", "bf16_round", "psaw_start",
    "Schedule", "PrhsOracle", "cosine", "gate_decision",
]


# --------------------------------------------------------------------------- helpers
def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bf16 (ties to even); result as float32.

    Used only to compare against the CUDA path's bf16 output tensor.
    """
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    bits = x32.view(np.uint32).astype(np.uint64)
    lsb = (bits >> 16) & 1
    rounded = ((bits + 0x7FFF + lsb) >> 16) << 16
    out = rounded.astype(np.uint32).view(np.float32)
    return np.where(np.isfinite(x32), out, x32).astype(np.float32)


# ------------------------------------------------------------------ Eq. (2): attention
def dense_scores(q: np.ndarray, K: np.ndarray, t: int) -> np.ndarray:
    """Logits a_i = q . k_i / sqrt(d) for every cached position i < t  (Eq. 2), float64."""
    d = q.shape[-1]
    return (K[:t].astype(np.float64) @ q.astype(np.float64)) / math.sqrt(d)


def rank_logits(a: np.ndarray) -> np.ndarray:
    """The logits in the precision the ranking decision is taken in (float32)."""
    return a.astype(np.float32)


def logsumexp(a: np.ndarray) -> float:
    """log sum_i exp(a_i) in float64; -inf for an empty vector."""
    if a.size == 0:
        return -math.inf
    mx = float(np.max(a))
    return mx + math.log(float(np.sum(np.exp(a.astype(np.float64) - mx))))


def softmax_full(a: np.ndarray) -> np.ndarray:
    """A_i = exp(a_i) / sum_j exp(a_j) over all visible positions (Eq. 2)."""
    e = np.exp(a.astype(np.float64) - np.max(a))
    return e / np.sum(e)


def dense_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray, t: int):
    """y = sum_i A_i v_i over i < t (Eq. 2).  Returns (y float64 [d], lse float)."""
    a = dense_scores(q, K, t)
    A = softmax_full(a)
    return A @ V[:t].astype(np.float64), logsumexp(a)


# ------------------------------------------------- Sec. 4.1: top-k over the middle range
def psaw_start(layer: int, num_layers: int, t: int, phi: float, alpha: float, layer_start: int) -> int:
    """P_l(t) of the progressive sliding attention window (Eq. 11).

    `layer` is 0-based; the paper's l is layer + 1 and runs to N = num_layers.  `layer_start`
    is the paper's l_s (1-based; Sec. 5.1 default floor(3N/4)); 0 switches the window off.
    P = 0 for l < l_s, else floor((1 - phi^(alpha (l - l_s) / (N - l_s))) t).  The result is
    used as a 0-based position: positions [S0, P) are masked, [0, S0) and [P, t) stay visible.
    """
    ell = layer + 1
    if layer_start <= 0 or ell < layer_start or num_layers <= layer_start:
        return 0
    expo = alpha * (ell - layer_start) / (num_layers - layer_start)
    return int(math.floor((1.0 - phi ** expo) * t))


def topk_middle(a: np.ndarray, t: int, sinks: int, window: int, k: int, psaw_lo: int = 0) -> np.ndarray:
    """S* = the k positions of largest logit among the middle candidates [S0, t-W).

    With a sliding-window start `psaw_lo` (Eq. 11) the candidates are [max(S0, P), t-W).

    Returned in descending-logit order p_1, p_2, ... (Sec. 4.1 ranks the winners by falling
    attention weight); equal logits are ordered by lower position first.  Softmax is monotone in the logit, so ranking logits ranks attention weights.
    The ranking uses the float32-rounded logits (see module docstring).
    """
    lo, hi = max(sinks, psaw_lo), t - window
    if hi <= lo or k <= 0:
        return np.zeros(0, dtype=np.int64)
    cand = np.arange(lo, hi, dtype=np.int64)
    a32 = rank_logits(a[lo:hi])
    # stable sort on the negated logit: descending logit, ascending position among equals
    order = np.argsort(-a32.astype(np.float64), kind="stable")
    return cand[order[: min(k, hi - lo)]]


def group_logits(per_head: list) -> np.ndarray:
    """Group-shared ranking logits of a KV head: the element-wise maximum over its query heads.

    NOT in the paper (its index sets are per head, Sec. 4.1): a labelled variant for
    grouped-query attention in which the heads that share a KV head also share ONE index set,
    so that a gathered K/V row serves the whole group.  A position is ranked by the largest
    float32 logit any head of the group gives it; top-k, dilation and the set are then built
    exactly as for a single head.  Every winner is in the own top-k of at least one head
    (the head that attains its maximum), which is what the tests pin.
    """
    return np.maximum.reduce([rank_logits(a) for a in per_head])


# ------------------------------------------------------------- Eq. (10): neighbour dilation
def dilate(s_star: np.ndarray, m: int, r: int, t_anchor: int) -> np.ndarray:
    """S^ = S* ∪ ⋃_{i<m} { p_i + j : -r <= j <= r }, clipped to [0, t_anchor)  (Eq. 10).

    `s_star` is in descending-weight order, so its first m entries are the m highest-
    weight winners.  Returns a sorted array of unique positions.
    """
    out = set(int(p) for p in s_star)
    for p in s_star[: max(0, min(m, len(s_star)))]:
        for j in range(-r, r + 1):
            x = int(p) + j
            if 0 <= x < t_anchor:
                out.add(x)
    return np.array(sorted(out), dtype=np.int64)


# ---------------------------------------------------------------- Sec. 4.1: critical set
def build_set(t: int, sinks: int, window: int, middle: np.ndarray, psaw_lo: int = 0) -> np.ndarray:
    """C = [0, S0) ∪ M ∪ [t-W, t) at the CURRENT length t; sorted, unique (Sec. 4.1).

    On a sharing step M is the anchor's (dilated) middle set (Def. 3.2); the sink and
    local groups are positional and follow the current t.  With a sliding-window start
    `psaw_lo` = P_l(t) (Sec. 4.2) only the visible positions [0, S0) ∪ [P, t) are kept.
    """
    out = set(range(0, min(sinks, t)))
    out.update(int(x) for x in middle if 0 <= int(x) < t)
    out.update(range(max(0, t - window), t))
    s0 = min(sinks, t)
    return np.array(sorted(x for x in out if x < s0 or x >= psaw_lo), dtype=np.int64)


# ------------------------------------------------------ Def. 3.1: token-sparse attention
def attn_over_set(q: np.ndarray, K: np.ndarray, V: np.ndarray, C: np.ndarray):
    """Attention restricted to index set C and renormalised over it (Def. 3.1).

    Returns (y float64 [d], lse_C float) with lse_C = log sum_{i in C} exp(a_i).
    """
    d = q.shape[-1]
    if len(C) == 0:
        return np.zeros(d, dtype=np.float64), -math.inf
    a = (K[C].astype(np.float64) @ q.astype(np.float64)) / math.sqrt(d)
    mx = np.max(a)
    e = np.exp(a - mx)
    return (e / np.sum(e)) @ V[C].astype(np.float64), float(mx + math.log(np.sum(e)))


# ---------------------------------------------------- Sec. 2.3: retained / dropped mass
def retained_mass(a: np.ndarray, C: np.ndarray) -> float:
    """tau_C = sum_{i in C} A_i with A the FULL softmax over all visible positions."""
    return float(np.sum(softmax_full(a)[C]))


def dropped_mass(a: np.ndarray, C: np.ndarray) -> float:
    """delta_C = 1 - tau_C, summed directly over the complement to avoid cancellation."""
    A = softmax_full(a)
    mask = np.ones(a.shape[0], dtype=bool)
    mask[C] = False
    return float(np.sum(A[mask]))


def delta_from_lse(lse_C: float, lse_full: float) -> float:
    """delta = 1 - exp(lse_C - lse_full): the same quantity from the two log-sums."""
    if lse_C == -math.inf:
        return 1.0
    return float(-math.expm1(lse_C - lse_full))


def mi_bound_g(delta: float, L: int) -> float:
    """g(delta) = 2 [ h_b(delta) + delta log L ]  (Eq. 4), natural logarithm."""
    if delta <= 0.0:
        return 0.0
    hb = -delta * math.log(delta)
    if delta < 1.0:
        hb -= (1.0 - delta) * math.log1p(-delta)
    return 2.0 * (hb + delta * math.log(L))


def coverage(shared: np.ndarray, target: np.ndarray) -> float:
    """|shared ∩ target| / |target|: the overlap measure of Fig. 4."""
    if len(target) == 0:
        return 1.0
    return len(np.intersect1d(shared, target)) / float(len(target))


# ------------------------------------------------------------- the per-step state machine
@dataclass
class Schedule:
    """The knobs of CIS (Sec. 4.1, defaults Sec. 5.1) plus the cross-layer group size."""
    top_k: int
    window: int
    sinks: int
    refresh_interval: int = 1      # s: block size; the first step of a block retrieves
    layer_group: int = 1           # G_L: layers sharing one leader's set (not in the paper body)
    dilate_r: int = 1
    dilate_m: int = -1             # -1 -> floor(k/3)
    dilate_anchor: bool = False    # True: the anchor's own attention also uses S^
    top_k_per_seq: np.ndarray | None = None
    sim_threshold: float | None = None   # tau of the cosine gate (Eq. 9; Sec. 5.1 default 0.8); None = fixed schedule
    psaw_phi: float = 0.7          # Eq. 11 (defaults Sec. 5.1)
    psaw_alpha: float = 1.0
    psaw_layer_start: int = 0      # l_s, 1-based; 0 = no sliding window
    num_layers: int = 1            # N of Eq. 11
    group_sets: bool = False       # labelled variant, NOT in the paper: one set per KV head (see group_logits)

    def k_for(self, b: int) -> int:
        return int(self.top_k_per_seq[b]) if self.top_k_per_seq is not None else self.top_k

    def m_for(self, b: int) -> int:
        return self.k_for(b) // 3 if self.dilate_m < 0 else self.dilate_m

    def psaw_for(self, layer: int, t: int) -> int:
        return psaw_start(layer, self.num_layers, t, self.psaw_phi, self.psaw_alpha, self.psaw_layer_start)


def cosine(q1: np.ndarray, q2: np.ndarray) -> float:
    """sim(i, j) = q_i . q_j / (|q_i| |q_j|)  (Eq. 9), float64."""
    a, b = q1.astype(np.float64), q2.astype(np.float64)
    return float(a @ b / (math.sqrt(float(a @ a)) * math.sqrt(float(b @ b))))


def gate_decision(q: np.ndarray, earlier: list, tau: float):
    """Cosine gate of CIS (Sec. 4.1 "Similarity Criteria").

    `earlier` lists the queries of the earlier steps of the block, oldest first.  Returns
    (ref, sims): ref = index into `earlier` of the MOST RECENT query with sim > tau, or -1
    if none (the head must retrieve); sims = the similarities, aligned with `earlier`.
    """
    sims = [cosine(q, e) for e in earlier]
    for j in range(len(earlier) - 1, -1, -1):
        if sims[j] > tau:
            return j, sims
    return -1, sims


@dataclass
class _Block:
    """What one (layer group, sequence, head) remembers inside the current block."""
    start: int = -1                                     # first step of the block
    queries: list = field(default_factory=list)         # q of every step so far, by position
    set_of_pos: list = field(default_factory=list)      # which set each step attended over
    sets: list = field(default_factory=list)            # (s_star, s_hat) per retrieval, in order
    own_at: int = -1                                    # step of the latest retrieval


class PrhsOracle:
    """Runs the decode-step schedule one (layer, step) at a time.

    Blocks of `refresh_interval` steps (Sec. 4.1): the first step of a block retrieves.  A later
    step of the block, on the first layer of its layer group,
      * without a similarity threshold shares the block's first set (fixed schedule);
      * with `sim_threshold` = tau applies the cosine gate per head: it shares the set used by
        the most recent earlier step of the block whose query has cosine similarity > tau,
        and retrieves a new set if there is none.
    A retrieval stores S* and its dilation S^ (Eq. 10).  The retrieving call attends over C
    built from the undilated S* unless `dilate_anchor` is set (Sec. 5.2.2 counts the budget
    of dilation for the sharing steps); every sharer attends over C built from S^ (Def. 3.2) with its own
    q, K, V.  The other layers of a group follow the decision and the set of its first layer.

    `override_ref` / `override_s_star` (per (b, h)) let a test substitute a decision or a
    retrieved S* that it has checked to be legal (a similarity within rounding of tau, a
    near-tie at the k-th logit), so that everything downstream can be compared exactly.
    """

    def __init__(self, sched: Schedule, num_q_heads: int, num_kv_heads: int):
        self.s = sched
        self.hq, self.hkv = num_q_heads, num_kv_heads
        self.gq = num_q_heads // num_kv_heads
        self.blocks: dict = {}          # (group, b, h) -> _Block
        self.last: dict = {}            # (group, b, h) -> (step, set id, own) of the latest leader call
        self.retrievals = 0             # head-level retrievals so far (for the retrieval ratio)
        self.calls = 0                  # head-level (layer, step) calls so far

    def is_retrieval(self, layer: int, step: int) -> bool:
        """True where the FIXED schedule retrieves (first layer of a group, first step of a block)."""
        return layer % self.s.layer_group == 0 and step % self.s.refresh_interval == 0

    def _plan(self, layer, step, b, h, q_bh, override_ref):
        """Decide what (layer, step) does for head (b, h): returns (block, set id, own, ref)."""
        g = layer // self.s.layer_group
        key = (g, b, h)
        if layer % self.s.layer_group != 0:           # follower: the leader's decision of this step
            if key not in self.last or self.last[key][0] != step:
                raise RuntimeError("group leader has not been called for this step")
            return self.blocks[key], self.last[key][1], False, None
        pos = step % self.s.refresh_interval
        blk = self.blocks.get(key)
        if pos == 0:
            blk = self.blocks[key] = _Block(start=step)
        elif blk is None or blk.start != step - pos or len(blk.queries) != pos:
            raise RuntimeError("group leader has not retrieved for this block")
        if pos == 0:
            ref = -1
        elif override_ref is not None and (b, h) in override_ref:
            ref = int(override_ref[(b, h)])
        elif self.s.sim_threshold is None:
            ref = 0
        else:
            ref, _ = gate_decision(q_bh, blk.queries, self.s.sim_threshold)
        own = ref < 0
        set_id = len(blk.sets) if own else blk.set_of_pos[ref]
        return blk, set_id, own, ref

    def decode_step(self, layer, step, q, K, V, seq_lens, units=None, want_delta=True,
                    override_ref=None, override_s_star=None):
        """q [B][Hq][d]; K, V [B][Hkv][cap][d]; seq_lens [B].

        `units` optionally restricts the work to a list of (b, h) pairs (sampled parity).
        Returns dict with per-unit 'y' (float64), 'lse', 'delta', 'set', 'retrieved' (bool),
        'ref' (position in the block shared from, -1 = retrieved) and, where retrieved,
        's_star', 's_hat', 'lse_full', 'scores32'.
        """
        B = q.shape[0]
        if units is None:
            units = [(b, h) for b in range(B) for h in range(self.hq)]
        leader = layer % self.s.layer_group == 0
        out = {"y": {}, "lse": {}, "delta": {}, "set": {}, "s_star": {}, "lse_full": {},
               "scores32": {}, "retrieved": {}, "ref": {}, "s_hat": {}}
        if self.s.group_sets and self.s.sim_threshold is not None:
            raise ValueError("the cosine gate is per head: not defined with group-shared sets")
        group_plan: dict = {}           # (b, kv) -> plan of the group (group_sets only)
        for (b, h) in units:
            t = int(seq_lens[b])
            kv = h // self.gq
            a = None
            if self.s.group_sets:
                # the group's first head carries the block state; one plan and one retrieval per group
                h0 = kv * self.gq
                first = (b, kv) not in group_plan
                if first:
                    blk, set_id, own, ref = self._plan(layer, step, b, h0, q[b, h0], override_ref)
                    if own:
                        heads = [dense_scores(q[b, h0 + j], K[b, kv], t) for j in range(self.gq)]
                        ag = group_logits(heads)
                        if override_s_star is not None and (b, h0) in override_s_star:
                            s_star = np.asarray(override_s_star[(b, h0)], dtype=np.int64)
                        else:
                            s_star = topk_middle(ag, t, self.s.sinks, self.s.window, self.s.k_for(b),
                                                 self.s.psaw_for(layer, t))
                        blk.sets.append((s_star, dilate(s_star, self.s.m_for(b), self.s.dilate_r, t)))
                        group_plan[(b, kv)] = (blk, set_id, own, ref, ag)
                    else:
                        group_plan[(b, kv)] = (blk, set_id, own, ref, None)
                    if leader:
                        blk.queries.append(np.array(q[b, h0], dtype=np.float64))
                        blk.set_of_pos.append(set_id)
                        self.last[(layer // self.s.layer_group, b, h0)] = (step, set_id, own)
                blk, set_id, own, ref, ag = group_plan[(b, kv)]
                if own:
                    out["s_star"][(b, h)] = blk.sets[set_id][0]
                    out["s_hat"][(b, h)] = blk.sets[set_id][1]
                    out["scores32"][(b, h)] = ag
                    self.retrievals += 1
                if leader:
                    out["ref"][(b, h)] = ref
            else:
                blk, set_id, own, ref = self._plan(layer, step, b, h, q[b, h], override_ref)
            if own and not self.s.group_sets:
                a = dense_scores(q[b, h], K[b, kv], t)
                if override_s_star is not None and (b, h) in override_s_star:
                    s_star = np.asarray(override_s_star[(b, h)], dtype=np.int64)
                else:
                    s_star = topk_middle(a, t, self.s.sinks, self.s.window, self.s.k_for(b),
                                         self.s.psaw_for(layer, t))
                blk.sets.append((s_star, dilate(s_star, self.s.m_for(b), self.s.dilate_r, t)))
                out["s_star"][(b, h)] = s_star
                out["s_hat"][(b, h)] = blk.sets[-1][1]
                out["scores32"][(b, h)] = rank_logits(a)
                self.retrievals += 1
            if leader and not self.s.group_sets:
                g = layer // self.s.layer_group
                blk.queries.append(np.array(q[b, h], dtype=np.float64))
                blk.set_of_pos.append(set_id)
                out["ref"][(b, h)] = ref
                self.last[(g, b, h)] = (step, set_id, own)
            self.calls += 1
            out["retrieved"][(b, h)] = own
            s_star, s_hat = blk.sets[set_id]
            M = s_star if (own and not self.s.dilate_anchor) else s_hat
            C = build_set(t, self.s.sinks, self.s.window, M, self.s.psaw_for(layer, t))
            y, lse_c = attn_over_set(q[b, h], K[b, kv], V[b, kv], C)
            out["set"][(b, h)], out["y"][(b, h)], out["lse"][(b, h)] = C, y, lse_c
            if want_delta:
                if a is None:
                    a = dense_scores(q[b, h], K[b, kv], t)
                lse_full = logsumexp(a)
                out["lse_full"][(b, h)] = lse_full
                out["delta"][(b, h)] = delta_from_lse(lse_c, lse_full)
        return out

    def retrieval_ratio(self) -> float:
        """rho-hat of Sec. 5.1: head-level retrievals / head-level (layer, step) calls so far."""
        return self.retrievals / max(1, self.calls)
