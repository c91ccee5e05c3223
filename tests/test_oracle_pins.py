"""Pins for the CPU oracle: every function is checked against something other than itself.

Closed forms, brute-force enumeration, library routines on special cases, identities and
inequalities stated by the paper.  Each pin is chosen so that a plausible mistake in the
oracle (a dropped term, a wrong sign or index, a transposed operand, an off-by-one range
end) fails at least one of them.  No GPU is needed.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import prhs_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def bf16(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).float().numpy()


def rand_case(seed, t=300, d=128, scale=1.0):
    g = rng(seed)
    q = bf16(g.standard_normal(d) * scale)
    K = bf16(g.standard_normal((t, d)))
    V = bf16(g.standard_normal((t, d)))
    return q, K, V


# ----------------------------------------------------------------------------- bf16 helper
def test_bf16_round_matches_torch_rne():
    g = rng(1)
    x = np.concatenate([g.standard_normal(5000) * 10.0 ** g.integers(-6, 6, 5000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38]]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).float().numpy()
    assert np.array_equal(O.bf16_round(x), want)


# ------------------------------------------------------------------- dense attention, Eq. 2
def test_dense_attention_matches_library_sdpa():
    q, K, V = rand_case(2, t=257)
    y, lse = O.dense_attention(q, K, V, 257)
    tq = torch.from_numpy(q).double()[None, None, None, :]
    tk = torch.from_numpy(K).double()[None, None]
    tv = torch.from_numpy(V).double()[None, None]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv)[0, 0, 0].numpy()
    assert np.allclose(y, want, atol=1e-12)
    want_lse = torch.logsumexp((tk[0, 0] @ tq[0, 0, 0]) / math.sqrt(128), 0).item()
    assert abs(lse - want_lse) < 1e-12


def test_dense_scores_scale_and_orientation():
    # a_i = q.k_i / sqrt(d): a single non-zero coordinate makes the expected value obvious,
    # and a non-square K catches a transposed operand.
    d, t = 128, 7
    q = np.zeros(d, np.float32); q[3] = 2.0
    K = np.zeros((t, d), np.float32); K[:, 3] = np.arange(t)
    a = O.dense_scores(q, K, t)
    assert np.allclose(a, 2.0 * np.arange(t) / math.sqrt(128))
    assert O.dense_scores(q, K, 4).shape == (4,)          # only positions < t are visible


def test_identical_keys_give_uniform_attention():
    g = rng(3)
    t, d = 100, 128
    q = bf16(g.standard_normal(d))
    K = np.tile(bf16(g.standard_normal(d)), (t, 1))
    V = bf16(g.standard_normal((t, d)))
    y, _ = O.dense_attention(q, K, V, t)
    assert np.allclose(y, V.astype(np.float64).mean(0), atol=1e-12)
    assert np.allclose(O.softmax_full(O.dense_scores(q, K, t)), 1.0 / t)


def test_one_dominant_key_returns_its_value():
    q, K, V = rand_case(4, t=64)
    K[:] *= 0.01
    K[17] = q * (40.0 * math.sqrt(128) / float(q @ q))      # logit +40 at position 17
    y, _ = O.dense_attention(q, K, V, 64)
    assert np.allclose(y, V[17], atol=1e-12 + 64 * math.exp(-39.0) * 10)


# ---------------------------------------------------------------------- top-k, Sec. 2.3/4.1
def test_topk_brute_force_maximises_retained_mass():
    # Enumerate every subset of the middle range: S* must attain the maximum retained mass
    # (the argmax characterisation of the top-k oracle, Eq. 5).
    for seed in range(6):
        g = rng(10 + seed)
        t, S0, W = int(g.integers(8, 15)), int(g.integers(0, 3)), int(g.integers(0, 4))
        k = int(g.integers(1, 5))
        a = g.standard_normal(t) * 2.0
        s_star = O.topk_middle(a, t, S0, W, k)
        cand = range(S0, t - W)
        A = O.softmax_full(a)
        kk = min(k, len(cand))
        best = max(sum(A[list(s)]) for s in itertools.combinations(cand, kk))
        assert len(s_star) == kk and len(set(s_star)) == kk
        assert all(S0 <= p < t - W for p in s_star)
        assert abs(sum(A[s_star]) - best) < 1e-15
        assert np.all(np.diff(a[s_star]) <= 0)             # descending weight order


def test_topk_tie_break_lower_index_and_nesting():
    t, S0, W = 200, 4, 16
    a = np.full(t, 0.25)
    assert np.array_equal(O.topk_middle(a, t, S0, W, 10), np.arange(S0, S0 + 10))
    a = rng(5).standard_normal(t)
    a[50] = a[20] = a[120] = 1.5                            # a three-way tie inside the winners
    prev = np.zeros(0, dtype=np.int64)
    for k in range(1, 40):
        cur = O.topk_middle(a, t, S0, W, k)
        assert np.array_equal(cur[: len(prev)], prev)       # Top_k is a prefix of Top_{k+1}
        prev = cur
    pos = {int(p): i for i, p in enumerate(prev)}
    assert pos[20] < pos[50] < pos[120]


def test_topk_matches_library_topk_without_ties():
    a = rng(6).standard_normal(1000)
    got = O.topk_middle(a, 1000, 8, 32, 64)
    want = torch.topk(torch.from_numpy(a[8:968].astype(np.float32)), 64).indices.numpy() + 8
    assert np.array_equal(got, want)


def test_topk_range_ends_and_empty_middle():
    a = np.arange(20, dtype=np.float64)                     # largest logits are the most recent
    got = O.topk_middle(a, 20, 2, 5, 3)
    assert np.array_equal(got, [14, 13, 12])                # position t-W=15 is local, not middle
    a = -np.arange(20, dtype=np.float64)
    assert np.array_equal(O.topk_middle(a, 20, 2, 5, 3), [2, 3, 4])   # position S0=2 is middle
    assert len(O.topk_middle(a, 7, 2, 5, 3)) == 0
    assert len(O.topk_middle(a, 20, 2, 5, 100)) == 13       # k larger than the range


# ------------------------------------------------------------------------ dilation, Eq. 10
def test_dilation_hand_case():
    got = O.dilate(np.array([10, 50, 11]), m=2, r=1, t_anchor=100)
    assert np.array_equal(got, [9, 10, 11, 49, 50, 51])
    # the third winner (11) is not among the top-m: its neighbour 12 must not appear
    assert 12 not in got


def test_dilation_properties():
    g = rng(7)
    for _ in range(20):
        t = int(g.integers(50, 400))
        k = int(g.integers(1, 30))
        s_star = g.permutation(t)[:k]
        m, r = int(g.integers(0, k + 1)), int(g.integers(0, 3))
        s_hat = O.dilate(s_star, m, r, t)
        assert set(s_star) <= set(s_hat)
        assert len(s_hat) <= k + 2 * r * m                  # workload bound of App. A3
        assert np.all(np.diff(s_hat) > 0) and s_hat[0] >= 0 and s_hat[-1] < t
        assert np.array_equal(O.dilate(s_star, m, 0, t), np.sort(s_star))
        assert np.array_equal(O.dilate(s_star, 0, r, t), np.sort(s_star))
    # isolated winners away from the ends: the bound is attained exactly
    s_star = np.arange(10, 400, 10)
    assert len(O.dilate(s_star, 13, 2, 1000)) == len(s_star) + 2 * 2 * 13
    # clipping at both ends
    assert np.array_equal(O.dilate(np.array([0, 9]), 2, 1, 10), [0, 1, 8, 9])


# --------------------------------------------------------------------- critical set, Sec 4.1
def test_set_sizes_printed_by_the_paper():
    with open(os.path.join(GOLDEN, "paper_sizes.txt")) as f:
        rows = [l.split("#")[0].split() for l in f if l.split("#")[0].strip()]
    assert len(rows) >= 2
    for total, s0, k, w in (map(int, r) for r in rows):
        t = 5000
        a = rng(total).standard_normal(t)
        C = O.build_set(t, s0, w, O.topk_middle(a, t, s0, w, k))
        assert len(C) == total == s0 + k + w


def test_paper_defaults_fixture():
    with open(os.path.join(GOLDEN, "paper_defaults.txt")) as f:
        kv = dict(l.split("#")[0].split() for l in f if l.split("#")[0].strip())
    s = O.Schedule(top_k=432, window=64, sinks=16)
    assert s.dilate_r == int(kv["dilate_r"])
    assert s.m_for(0) == 432 // int(kv["dilate_m_divisor"]) == 144
    assert s.psaw_phi == float(kv["psaw_phi"]) and s.psaw_alpha == float(kv["psaw_alpha"])


def test_build_set_union_and_bounds():
    C = O.build_set(100, 4, 10, np.array([3, 50, 95, 60]))
    assert np.array_equal(C, [0, 1, 2, 3, 50, 60] + list(range(90, 100)))
    assert np.array_equal(O.build_set(5, 4, 10, np.array([], dtype=np.int64)), np.arange(5))
    g = rng(8)
    for _ in range(20):
        t, s0, w, k = 500, int(g.integers(0, 9)), int(g.integers(0, 40)), int(g.integers(1, 60))
        r, m = int(g.integers(0, 3)), int(g.integers(0, k + 1))
        s_star = O.topk_middle(g.standard_normal(t), t, s0, w, k)
        C = O.build_set(t + 3, s0, w, O.dilate(s_star, m, r, t))
        assert len(C) <= s0 + k + 2 * r * m + w and np.all(np.diff(C) > 0)


# ------------------------------------------------ sparse attention = dense when nothing is dropped
def test_full_budget_equals_dense_and_delta_zero():
    q, K, V = rand_case(9, t=300)
    t = 300
    a = O.dense_scores(q, K, t)
    C = O.build_set(t, 4, 16, O.topk_middle(a, t, 4, 16, k=t))        # k >= t
    assert np.array_equal(C, np.arange(t))
    y, lse_c = O.attn_over_set(q, K, V, C)
    yd, lse = O.dense_attention(q, K, V, t)
    assert np.allclose(y, yd, atol=1e-13) and abs(lse - lse_c) < 1e-12
    assert O.delta_from_lse(lse_c, lse) == pytest.approx(0.0, abs=1e-12)
    assert O.dropped_mass(a, C) == 0.0


def test_sparse_attention_is_renormalised_full_softmax():
    # A~_i = A_i / tau on the set (App. "Unified Information Bounds", Setup)
    q, K, V = rand_case(10, t=200, scale=2.0)
    a = O.dense_scores(q, K, 200)
    C = np.array([0, 1, 5, 77, 150, 199])
    A = O.softmax_full(a)
    y, lse_c = O.attn_over_set(q, K, V, C)
    want = (A[C] / A[C].sum()) @ V[C].astype(np.float64)
    assert np.allclose(y, want, atol=1e-13)
    assert math.exp(lse_c - O.logsumexp(a)) == pytest.approx(A[C].sum(), rel=1e-12)


# -------------------------------------------------------------------------- delta, Sec. 2.3
def test_delta_definitions_agree():
    q, K, V = rand_case(11, t=400, scale=3.0)
    a = O.dense_scores(q, K, 400)
    C = O.build_set(400, 4, 32, O.topk_middle(a, 400, 4, 32, 40))
    tau = O.retained_mass(a, C)
    _, lse_c = O.attn_over_set(q, K, V, C)
    d1, d2 = O.dropped_mass(a, C), O.delta_from_lse(lse_c, O.logsumexp(a))
    assert d1 == pytest.approx(1.0 - tau, abs=1e-14) and d2 == pytest.approx(d1, rel=1e-10)
    # total-variation identity (Lemma "Total-variation of truncation") and the KL identity
    A = O.softmax_full(a)
    At = np.zeros_like(A); At[C] = A[C] / tau
    assert 0.5 * np.abs(A - At).sum() == pytest.approx(d1, rel=1e-12)
    kl = float(np.sum(At[C] * np.log(At[C] / A[C])))
    assert kl == pytest.approx(-math.log(tau), rel=1e-12)


def test_delta_closed_form_identical_keys_tiny_shape():
    # uniform attention: delta = 1 - |C|/t.  Tiny config: t = 4097, |C| = 4 + 256 + 64 = 324
    t, d = 4097, 128
    q = bf16(rng(12).standard_normal(d))
    K = np.tile(bf16(rng(13).standard_normal(d)), (t, 1))
    a = O.dense_scores(q, K, t)
    C = O.build_set(t, 4, 64, O.topk_middle(a, t, 4, 64, 256))
    assert len(C) == 324
    assert O.dropped_mass(a, C) == pytest.approx(1.0 - 324.0 / 4097.0, rel=1e-12)
    _, lse_c = O.attn_over_set(q, K, K, C)
    assert O.delta_from_lse(lse_c, O.logsumexp(a)) == pytest.approx(1 - 324 / 4097, rel=1e-12)


def test_delta_closed_form_geometric_recency():
    # logits a_i = lam * i; window-only selector: delta = (rho^W - rho^t) / (1 - rho^t),
    # rho = exp(-lam)  (geometric tail sum, App. "Exponential Recency Beyond Sink")
    t, d, W = 300, 128, 25
    q = np.zeros(d, np.float32); q[0] = 1.0
    K = np.zeros((t, d), np.float32); K[:, 0] = np.arange(t) * 0.5
    lam = 0.5 / math.sqrt(d)
    rho = math.exp(-lam)
    a = O.dense_scores(q, K, t)
    C = O.build_set(t, 0, W, np.zeros(0, dtype=np.int64))
    want = (rho ** W - rho ** t) / (1 - rho ** t)
    assert O.dropped_mass(a, C) == pytest.approx(want, rel=1e-12)
    _, lse_c = O.attn_over_set(q, K, K, C)
    assert O.delta_from_lse(lse_c, O.logsumexp(a)) == pytest.approx(want, rel=1e-10)


def test_delta_monotone_in_k_and_window():
    q, K, V = rand_case(14, t=600, scale=2.0)
    a = O.dense_scores(q, K, 600)
    last = 1.0
    for k in (0, 1, 5, 20, 100, 400, 600):
        dlt = O.dropped_mass(a, O.build_set(600, 4, 16, O.topk_middle(a, 600, 4, 16, k)))
        assert dlt <= last + 1e-15
        last = dlt
    assert last == 0.0
    # a larger window with the SAME middle set never increases delta
    M = O.topk_middle(a, 600, 4, 64, 50)
    last = 1.0
    for w in (0, 1, 8, 64, 300, 600):
        dlt = O.dropped_mass(a, O.build_set(600, 4, w, M))
        assert dlt <= last + 1e-15
        last = dlt


# ----------------------------------------------------- CIS guarantee (Theorem 2 and its lemmas)
def test_cis_inequalities_hold_on_every_input():
    for seed in range(8):
        g = rng(100 + seed)
        t, d, S0, W, k, r = 700, 128, 4, 32, 48, 1
        q = bf16(g.standard_normal(d) * 2.0)
        dq = bf16(g.standard_normal(d) * g.choice([0.02, 0.1, 0.5]))
        q2 = bf16(q + dq)
        K = bf16(g.standard_normal((t, d)))
        a, a2 = O.dense_scores(q, K, t), O.dense_scores(q2, K, t)
        A, A2 = O.softmax_full(a), O.softmax_full(a2)
        d_att = np.abs(A2 - A).sum()
        kmax = np.linalg.norm(K.astype(np.float64), axis=1).max()
        delta_q = np.linalg.norm((q2 - q).astype(np.float64))
        # softmax Lipschitz and logit perturbation lemmas
        assert d_att <= 2 * np.abs(a2 - a).max() + 1e-12
        assert np.abs(a2 - a).max() <= kmax * delta_q / math.sqrt(d) + 1e-12
        # oracle continuity, reuse lower bound and the CIS proposition (fixed cache)
        # top-k over ALL positions here: the lemmas are stated for the unrestricted oracle
        s1, s2 = O.topk_middle(a, t, 0, 0, k), O.topk_middle(a2, t, 0, 0, k)
        s_hat = O.dilate(s1, k // 3, r, t)
        tau1, tau2 = A[s1].sum(), A2[s2].sum()
        tau_hat_q, tau_pre = A[s_hat].sum(), A2[s_hat].sum()
        assert abs(tau2 - tau1) <= d_att + 1e-12
        assert tau_pre >= tau_hat_q - d_att - 1e-12
        assert tau_pre >= tau2 - 2 * d_att - 1e-12
        # centroid drift (Theorem 1)
        pos = np.arange(t)
        assert abs(A2 @ pos - A @ pos) <= (t - 1) * d_att + 1e-9


def test_dilated_set_covers_next_topk_on_clustered_keys():
    # n_c clusters (c-1, c, c+1) with logits (h-g, h, h-g) under q; everything else far below.
    # A drift that moves every logit by at most eps, g < eps < D/2, can swap ranks inside a
    # cluster but cannot bring in an outside key: S^(q) covers S*(q') completely while the
    # undilated S*(q) does not (the picture of Fig. 4).
    d, t, n_c = 128, 600, 12
    centres = np.arange(40, 40 + 40 * n_c, 40)
    sd = math.sqrt(d)
    h, gap, eps = 8.0, 0.05, 0.2
    K = np.zeros((t, d), np.float32)
    K[:, 0] = 1.0 * sd                                   # logit 1 everywhere (D = h - 1 - ...)
    K[centres, 0] = h * sd
    K[centres - 1, 0] = (h - gap) * sd
    K[centres + 1, 0] = (h - gap) * sd
    K[centres + 1, 1] = eps * sd                          # the drift direction favours c+1
    q = np.zeros(d, np.float32); q[0] = 1.0
    q2 = q.copy(); q2[1] = 1.0
    a, a2 = O.dense_scores(q, K, t), O.dense_scores(q2, K, t)
    assert np.abs(a2 - a).max() <= eps + 1e-6          # keys are stored in float32
    s1 = O.topk_middle(a, t, 4, 16, n_c)
    s2 = O.topk_middle(a2, t, 4, 16, n_c)
    assert set(s1) == set(centres) and set(s2) == set(centres + 1)
    s_hat = O.dilate(s1, n_c, 1, t)
    assert O.coverage(s_hat, s2) == 1.0
    assert O.coverage(np.sort(s1), s2) == 0.0


# -------------------------------------------------------------- cosine gate, Eq. 9 / Sec. 4.1
def test_cosine_similarity_against_library_and_closed_forms():
    g = rng(40)
    a, b = g.standard_normal(128), g.standard_normal(128)
    want = torch.nn.functional.cosine_similarity(torch.from_numpy(a)[None], torch.from_numpy(b)[None]).item()
    assert O.cosine(a, b) == pytest.approx(want, rel=1e-12)
    assert O.cosine(a, 3.5 * a) == pytest.approx(1.0, abs=1e-15)          # scale invariant
    assert O.cosine(a, -a) == pytest.approx(-1.0, abs=1e-15)
    e0, e1 = np.eye(128)[0], np.eye(128)[1]
    assert O.cosine(e0, e1) == 0.0
    assert O.cosine(e0, e0 + e1) == pytest.approx(math.sqrt(0.5), rel=1e-15)


def test_gate_picks_the_most_recent_similar_query():
    e = np.eye(128)
    q = e[0] + 0.1 * e[1]
    earlier = [e[0], e[1], e[0] + 0.2 * e[1], e[2]]      # sims: .995, .0995, .995.., 0
    ref, sims = O.gate_decision(q, earlier, 0.8)
    assert ref == 2 and sims[0] > 0.8 and sims[2] > 0.8 and sims[3] == 0.0   # 0 also passes; 2 is later
    assert O.gate_decision(q, earlier, 0.9999)[0] == -1                     # none similar enough
    assert O.gate_decision(q, [], 0.8)[0] == -1
    assert O.gate_decision(q, earlier, -1.0)[0] == 3                         # everything passes


def test_gated_schedule_limits():
    q, K, V = _stack(25, layers=1)
    t = lambda n: np.array([200 + n + 1, 150 + n + 1])
    base = dict(top_k=20, window=8, sinks=2, refresh_interval=4)
    fixed = O.PrhsOracle(O.Schedule(**base), 4, 2)
    always = O.PrhsOracle(O.Schedule(**base, sim_threshold=-1.0), 4, 2)     # gate always passes
    never = O.PrhsOracle(O.Schedule(**base, sim_threshold=1.0), 4, 2)       # gate never passes
    every = O.PrhsOracle(O.Schedule(**{**base, "refresh_interval": 1}), 4, 2)
    for n in range(6):
        a = fixed.decode_step(0, n, q[0, n], K[0], V[0], t(n))
        b = always.decode_step(0, n, q[0, n], K[0], V[0], t(n))
        c = never.decode_step(0, n, q[0, n], K[0], V[0], t(n))
        d = every.decode_step(0, n, q[0, n], K[0], V[0], t(n))
        for u in a["set"]:
            assert np.array_equal(a["set"][u], b["set"][u])       # tau = -1 is the fixed schedule
            assert np.array_equal(c["set"][u], d["set"][u])       # tau = 1 retrieves every step
            assert c["retrieved"][u] and (a["retrieved"][u] == (n % 4 == 0))
            assert b["ref"][u] == (-1 if n % 4 == 0 else n % 4 - 1)   # shares from the most recent step
    assert fixed.retrieval_ratio() == pytest.approx(2 / 6) and never.retrieval_ratio() == 1.0


def test_gated_schedule_mixed_heads():
    # head 0 keeps its query, head 1 jumps at step 2: only head 1 retrieves there, and step 3
    # shares from the most recent similar step (2 for head 1, still the block's first set for head 0)
    g = rng(41)
    K = bf16(g.standard_normal((1, 1, 300, 128)))
    V = bf16(g.standard_normal((1, 1, 300, 128)))
    base_q = bf16(g.standard_normal((2, 128)) * 2)
    other = bf16(g.standard_normal(128) * 2)
    orc = O.PrhsOracle(O.Schedule(top_k=16, window=8, sinks=2, refresh_interval=4, sim_threshold=0.8), 2, 1)
    outs = []
    for n in range(4):
        q = np.array(base_q, copy=True)[None]
        if n >= 2:
            q[0, 1] = other
        outs.append(orc.decode_step(0, n, q, K, V, np.array([280 + n])))
    assert [o["retrieved"][(0, 0)] for o in outs] == [True, False, False, False]
    assert [o["retrieved"][(0, 1)] for o in outs] == [True, False, True, False]
    assert [o["ref"][(0, 1)] for o in outs] == [-1, 0, -1, 2]
    s2 = outs[2]["s_star"][(0, 1)]
    want3 = O.build_set(283, 2, 8, O.dilate(s2, 16 // 3, 1, 282))
    assert np.array_equal(outs[3]["set"][(0, 1)], want3)
    assert orc.retrieval_ratio() == pytest.approx(3 / 8)


# ------------------------------------------------------- sliding attention window, Eq. 11
def test_psaw_window_start_worked_values():
    with open(os.path.join(GOLDEN, "psaw_window_start.txt")) as f:
        rows = [l.split("#")[0].split() for l in f if l.split("#")[0].strip()]
    assert len(rows) >= 9
    for phi, alpha, ell, t, want in rows:
        got = O.psaw_start(int(ell) - 1, 32, int(t), float(phi), float(alpha), 24)
        assert got == int(want), (phi, alpha, ell, t)
    # off switch, monotone in depth, never reaches t, alpha = 0 prunes nothing
    assert O.psaw_start(31, 32, 32768, 0.7, 1.0, 0) == 0
    ps = [O.psaw_start(l, 32, 50000, 0.7, 1.0, 24) for l in range(32)]
    assert ps[:24] == [0] * 24 and all(a <= b for a, b in zip(ps, ps[1:])) and ps[-1] < 50000
    assert all(O.psaw_start(l, 32, 50000, 0.7, 0.0, 24) == 0 for l in range(32))


def test_psaw_clips_retrieval_range_and_set():
    g = rng(30)
    t, S0, W, k, P = 400, 4, 16, 24, 150
    a = g.standard_normal(t)
    s_star = O.topk_middle(a, t, S0, W, k, psaw_lo=P)
    # brute force on the clipped range
    cand = np.arange(P, t - W)
    want = cand[np.argsort(-a[P:t - W], kind="stable")[:k]]
    assert np.array_equal(s_star, want) and s_star.min() >= P
    # the set keeps sinks, drops everything else below P
    M = O.dilate(O.topk_middle(a, t, S0, W, k), k // 3, 1, t)       # an unclipped shared set
    C0, C1 = O.build_set(t, S0, W, M), O.build_set(t, S0, W, M, psaw_lo=P)
    assert set(C1) == {x for x in C0 if x < S0 or x >= P}
    assert O.dropped_mass(a, C1) >= O.dropped_mass(a, C0) - 1e-15      # a subset retains less
    # a window start beyond t - W clips the local window too, sinks always stay
    C2 = O.build_set(t, S0, W, M, psaw_lo=t - 5)
    assert np.array_equal(C2, list(range(S0)) + list(range(t - 5, t)))
    assert np.array_equal(O.build_set(t, S0, W, M, psaw_lo=0), C0)


def test_schedule_with_psaw_layers():
    q, K, V = _stack(24, layers=4)
    s = O.Schedule(top_k=16, window=8, sinks=2, refresh_interval=2, layer_group=2, psaw_phi=0.5,
                   psaw_alpha=1.0, psaw_layer_start=2, num_layers=4)
    orc = O.PrhsOracle(s, 4, 2)
    for n in range(2):
        t = np.array([210 + n + 1, 190 + n + 1])
        for l in range(4):
            out = orc.decode_step(l, n, q[l, n], K[l], V[l], t)
            for (b, h), C in out["set"].items():
                P = O.psaw_start(l, 4, int(t[b]), 0.5, 1.0, 2)
                assert P == (0 if l < 2 else int((1 - 0.5 ** ((l - 1) / 2)) * int(t[b])))
                assert all(x < 2 or x >= P for x in C)
                if l == 3:
                    assert P == int(t[b]) // 2 and C[2] >= P


# ------------------------------------------------------------------------- MI bound, Eq. 4
def test_mi_bound_function():
    L = 4096
    assert O.mi_bound_g(0.0, L) == 0.0
    # binary entropy at 1/2 is log 2
    assert O.mi_bound_g(0.5, 1) == pytest.approx(2 * math.log(2), rel=1e-14)
    xs = np.linspace(1e-6, L / (1 + L), 400)
    g = np.array([O.mi_bound_g(x, L) for x in xs])
    assert np.all(np.diff(g) > 0)                         # monotone on (0, L/(1+L)]
    x, hstep = 0.01, 1e-7
    slope = (O.mi_bound_g(x + hstep, L) - O.mi_bound_g(x - hstep, L)) / (2 * hstep)
    assert slope == pytest.approx(2 * math.log(L * (1 - x) / x), rel=1e-6)


# ------------------------------------------------------------------ the decode-step schedule
def _stack(seed, layers=4, B=2, Hq=4, Hkv=2, cap=220, d=128):
    g = rng(seed)
    K = bf16(g.standard_normal((layers, B, Hkv, cap, d)))
    V = bf16(g.standard_normal((layers, B, Hkv, cap, d)))
    q = bf16(g.standard_normal((layers, 8, B, Hq, d)) * 2.0)
    return q, K, V


def test_schedule_every_step_retrieval_is_plain_topk():
    q, K, V = _stack(20, layers=1)
    s = O.Schedule(top_k=20, window=8, sinks=2, refresh_interval=1, layer_group=1)
    orc = O.PrhsOracle(s, 4, 2)
    for n in range(3):
        t = np.array([200 + n + 1, 150 + n + 1])
        out = orc.decode_step(0, n, q[0, n], K[0], V[0], t)
        for (b, h), C in out["set"].items():
            a = O.dense_scores(q[0, n, b, h], K[0, b, h // 2], int(t[b]))
            want = O.build_set(int(t[b]), 2, 8, O.topk_middle(a, int(t[b]), 2, 8, 20))
            assert np.array_equal(C, want)
            assert len(C) == 2 + 20 + 8
            # delta at an anchor equals the top-k oracle's delta*
            assert out["delta"][(b, h)] == pytest.approx(O.dropped_mass(a, want), rel=1e-9, abs=1e-13)


def test_schedule_sharing_reuses_the_anchor_middle_set():
    q, K, V = _stack(21, layers=1)
    s = O.Schedule(top_k=20, window=8, sinks=2, refresh_interval=4, dilate_r=1)
    orc = O.PrhsOracle(s, 4, 2)
    sets = {}
    for n in range(6):
        t = np.array([200 + n + 1, 150 + n + 1])
        out = orc.decode_step(0, n, q[0, n], K[0], V[0], t)
        sets[n] = out
        assert orc.is_retrieval(0, n) == (n % 4 == 0)
    for (b, h) in sets[0]["set"]:
        t0 = (201, 151)[b]
        s_star = sets[0]["s_star"][(b, h)]
        s_hat = O.dilate(s_star, 20 // 3, 1, t0)
        for n in (1, 2, 3):
            tn = t0 + n
            assert np.array_equal(sets[n]["set"][(b, h)], O.build_set(tn, 2, 8, s_hat))
            # positions that left the window since the anchor are dropped unless dilated in
            gone = set(range(t0 - 8, tn - 8)) - set(s_hat)
            assert not (gone & set(sets[n]["set"][(b, h)]))
        # the anchor's own attention is undilated; step 4 retrieves afresh
        assert np.array_equal(sets[0]["set"][(b, h)], O.build_set(t0, 2, 8, s_star))
        assert len(sets[4]["s_star"][(b, h)]) == 20
        # sharing steps carry no retrieval output
        assert (b, h) not in sets[1]["s_star"]


def test_schedule_cross_layer_followers_use_the_leader_set():
    q, K, V = _stack(22, layers=4)
    s = O.Schedule(top_k=16, window=8, sinks=2, refresh_interval=2, layer_group=2, dilate_r=1)
    orc = O.PrhsOracle(s, 4, 2)
    plain = O.PrhsOracle(O.Schedule(top_k=16, window=8, sinks=2, refresh_interval=2), 4, 2)
    for n in range(4):
        t = np.array([210 + n + 1, 190 + n + 1])
        outs = [orc.decode_step(l, n, q[l, n], K[l], V[l], t) for l in range(4)]
        for u in outs[0]["set"]:
            assert np.array_equal(outs[1]["set"][u], outs[0]["set"][u]) or n % 2 == 0
            assert np.array_equal(outs[3]["set"][u], outs[2]["set"][u]) or n % 2 == 0
            if n % 2 == 0:      # follower at the refresh step: leader's DILATED set
                b, h = u
                s_hat = O.dilate(outs[0]["s_star"][u], 16 // 3, 1, int(t[b]))
                assert np.array_equal(outs[1]["set"][u], O.build_set(int(t[b]), 2, 8, s_hat))
            # followers attend with their own q, K, V over that set
            b, h = u
            y, _ = O.attn_over_set(q[1, n, b, h], K[1, b, h // 2], V[1, b, h // 2], outs[1]["set"][u])
            assert np.allclose(outs[1]["y"][u], y)
        # layer_group = 1 is the same as no cross-layer sharing
        p = plain.decode_step(0, n, q[0, n], K[0], V[0], t)
        for u in p["set"]:
            assert np.array_equal(p["set"][u], outs[0]["set"][u])
    with pytest.raises(RuntimeError):
        O.PrhsOracle(s, 4, 2).decode_step(1, 0, q[1, 0], K[1], V[1], np.array([211, 191]))
    with pytest.raises(RuntimeError):
        O.PrhsOracle(s, 4, 2).decode_step(0, 1, q[0, 1], K[0], V[0], np.array([211, 191]))


def test_schedule_sampled_units_match_full_run():
    q, K, V = _stack(23, layers=1)
    s = O.Schedule(top_k=12, window=8, sinks=2, refresh_interval=2)
    full, part = O.PrhsOracle(s, 4, 2), O.PrhsOracle(s, 4, 2)
    for n in range(3):
        t = np.array([205 + n, 180 + n])
        a = full.decode_step(0, n, q[0, n], K[0], V[0], t)
        b = part.decode_step(0, n, q[0, n], K[0], V[0], t, units=[(1, 3)])
        assert list(b["y"]) == [(1, 3)]
        assert np.array_equal(a["y"][(1, 3)], b["y"][(1, 3)])


# ------------------------------------------------ labelled variant: one set per KV head (not in the paper)
def test_group_sets_properties():
    """Group-shared sets (ranking by the maximum logit over the heads of a KV group).

    What fixes the rule without retyping it: with one head per KV head it IS the per-head
    method; heads with identical queries reproduce the per-head set; every winner lies in the
    own top-k of at least one head of the group (the head attaining its maximum has fewer than
    k positions above it); and no head retains more mass over the group's undilated set than
    over its own top-k of the same size (Sec. 3.2: top-k maximises the retained mass).
    """
    q, K, V = _stack(31, layers=2, Hq=8, Hkv=2)
    kw = dict(top_k=16, window=8, sinks=2, refresh_interval=2, layer_group=2, dilate_r=0)
    grp = O.PrhsOracle(O.Schedule(group_sets=True, **kw), 8, 2)
    own = O.PrhsOracle(O.Schedule(**kw), 8, 2)
    for n in range(3):
        t = np.array([200 + n + 1, 170 + n + 1])
        for layer in range(2):
            a = grp.decode_step(layer, n, q[layer, n], K[layer], V[layer], t)
            b = own.decode_step(layer, n, q[layer, n], K[layer], V[layer], t)
            for (bb, h), C in a["set"].items():
                h0 = (h // 4) * 4
                assert np.array_equal(C, a["set"][(bb, h0)])                     # one set per group
                y, _ = O.attn_over_set(q[layer, n, bb, h], K[layer, bb, h // 4], V[layer, bb, h // 4], C)
                assert np.allclose(a["y"][(bb, h)], y)                          # own q, shared rows
                if layer == 0 and n % 2 == 0:
                    union = set()
                    for j in range(4):
                        union |= set(b["s_star"][(bb, h0 + j)].tolist())
                    assert set(a["s_star"][(bb, h)].tolist()) <= union
                    assert a["delta"][(bb, h)] >= b["delta"][(bb, h)] - 1e-12
    assert grp.retrieval_ratio() == own.retrieval_ratio() == pytest.approx(1 / 3)
    # one head per KV head: the variant is the method itself
    q1, K1, V1 = _stack(32, layers=1, Hq=2, Hkv=2)
    g1 = O.PrhsOracle(O.Schedule(top_k=12, window=8, sinks=2, refresh_interval=2, group_sets=True), 2, 2)
    p1 = O.PrhsOracle(O.Schedule(top_k=12, window=8, sinks=2, refresh_interval=2), 2, 2)
    for n in range(3):
        t = np.array([150 + n, 190 + n])
        x, y = g1.decode_step(0, n, q1[0, n], K1[0], V1[0], t), p1.decode_step(0, n, q1[0, n], K1[0], V1[0], t)
        for u in x["set"]:
            assert np.array_equal(x["set"][u], y["set"][u]) and np.array_equal(x["y"][u], y["y"][u])
    # identical queries inside a group: the group's set is every head's own set
    qs = q[0, 0].copy()
    qs[:, 1:4] = qs[:, 0:1]
    qs[:, 5:8] = qs[:, 4:5]
    t = np.array([201, 171])
    x = O.PrhsOracle(O.Schedule(group_sets=True, **kw), 8, 2).decode_step(0, 0, qs, K[0], V[0], t)
    y = O.PrhsOracle(O.Schedule(**kw), 8, 2).decode_step(0, 0, qs, K[0], V[0], t)
    for u in x["set"]:
        assert np.array_equal(x["s_star"][u], y["s_star"][u])
    # sampled units give the same result as a full run
    part = O.PrhsOracle(O.Schedule(group_sets=True, **kw), 8, 2).decode_step(0, 0, q[0, 0], K[0], V[0], t,
                                                                              units=[(1, 6)])
    full = O.PrhsOracle(O.Schedule(group_sets=True, **kw), 8, 2).decode_step(0, 0, q[0, 0], K[0], V[0], t)
    assert np.array_equal(part["set"][(1, 6)], full["set"][(1, 6)])
    with pytest.raises(ValueError):
        O.PrhsOracle(O.Schedule(group_sets=True, sim_threshold=0.8, **kw), 8, 2).decode_step(
            0, 0, q[0, 0], K[0], V[0], t)
