"""Pins for the fp64 CPU oracle: each test checks one step against something other than the oracle
itself -- a closed form, an identity the paper states, a stock library routine on a special case, or
brute force on tiny inputs.  No GPU is involved."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import Problem
from paper_2602_08686_b200 import inputs as gen

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_case(seed, Nu=2, H=4, Hkv=2, L=96, W=8, d=16, dtype=oracle.F32):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(Nu, H, W, d, generator=g)
    k = torch.randn(Nu, Hkv, L, d, generator=g)
    v = torch.randn(Nu, Hkv, L, d, generator=g)
    if dtype == oracle.BF16:
        q, k, v = q.bfloat16(), k.bfloat16(), v.bfloat16()
    prob = Problem(Nu, H, Hkv, L, W, head_dim=d, dtype=dtype, budget_per_head=24, pool_size=3)
    return prob, q, k, v


def torch_window_attention(q, k, G):
    """Causal softmax of the last-W queries from torch's own fp64 softmax routine."""
    q, k = q.double(), k.double()
    Nu, H, W, d = q.shape
    L = k.shape[2]
    kk = k.repeat_interleave(G, dim=1)                        # head h reads KV head h // G
    s = torch.einsum("uhid,uhtd->uhit", q, kk) / math.sqrt(d)
    pos_q = (L - W) + torch.arange(W).view(W, 1)
    mask = torch.arange(L).view(1, L) > pos_q
    s = s.masked_fill(mask, float("-inf"))
    return torch.softmax(s, dim=-1)


# ----------------------------------------------------------------------------- O1-O3
@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_mass_identity(dtype):
    """Every softmax row sums to one, so sum_t c_h[t] = W and the scaled window mass has mean one
    (the sentence after Eq. 4)."""
    prob, q, k, _ = rand_case(1, dtype=dtype)
    c = oracle.colsum(prob, gen.as_numpy(q), gen.as_numpy(k))
    np.testing.assert_allclose(c.sum(-1), prob.window, rtol=0, atol=1e-12)
    alpha = (prob.seq_len / prob.window) * c
    np.testing.assert_allclose(alpha.mean(-1), 1.0, rtol=0, atol=1e-12)


def test_closed_form_zero_queries():
    """q = 0 makes every visible key equally likely: A[i,t] = 1/(n+i+1) for t <= n+i."""
    prob, q, k, _ = rand_case(2, Nu=1, H=2, Hkv=1, L=40, W=5)
    q = torch.zeros_like(q)
    A = oracle.window_attention(prob, gen.as_numpy(q), gen.as_numpy(k))
    n, W, L = prob.n, prob.window, prob.seq_len
    for i in range(W):
        np.testing.assert_allclose(A[0, :, i, : n + i + 1], 1.0 / (n + i + 1), rtol=1e-14)
        assert (A[0, :, i, n + i + 1:] == 0).all()
    c = oracle.colsum(prob, gen.as_numpy(q), gen.as_numpy(k))
    pre = sum(1.0 / (n + i + 1) for i in range(W))
    np.testing.assert_allclose(c[0, :, :n], pre, rtol=1e-13)
    for r in range(W):
        np.testing.assert_allclose(c[0, :, n + r], sum(1.0 / (n + i + 1) for i in range(r, W)), rtol=1e-13)


def test_closed_form_single_spike():
    """One key with logit a for every row, all other logits zero: A[i,t*] = e^a / (e^a + n + i)."""
    d, L, W, tstar, a = 16, 50, 6, 17, 3.25
    n = L - W
    q = torch.zeros(1, 1, W, d)
    k = torch.zeros(1, 1, L, d)
    q[..., 3] = 2.0
    k[0, 0, tstar, 3] = a * math.sqrt(d) / 2.0
    prob = Problem(1, 1, 1, L, W, head_dim=d, dtype=oracle.F32)
    A = oracle.window_attention(prob, gen.as_numpy(q), gen.as_numpy(k))
    for i in range(W):
        z = math.exp(a) + n + i
        assert A[0, 0, i, tstar] == pytest.approx(math.exp(a) / z, rel=1e-13)
        assert A[0, 0, i, 0] == pytest.approx(1.0 / z, rel=1e-13)


@pytest.mark.parametrize("H,Hkv", [(2, 2), (6, 2), (4, 1)])
@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_attention_matches_library_softmax(H, Hkv, dtype):
    """Against torch's fp64 softmax: catches a wrong scale, mask, transposed operand or GQA mapping."""
    prob, q, k, _ = rand_case(3, H=H, Hkv=Hkv, dtype=dtype)
    A = oracle.window_attention(prob, gen.as_numpy(q), gen.as_numpy(k))
    ref = torch_window_attention(q, k, H // Hkv).numpy()
    np.testing.assert_allclose(A, ref, rtol=1e-11, atol=1e-15)
    c = oracle.colsum(prob, gen.as_numpy(q), gen.as_numpy(k))
    np.testing.assert_allclose(c, ref.sum(2), rtol=1e-11, atol=1e-15)


def test_one_hot_limit():
    """Orthogonal keys with a large scale: each window row puts (almost) all its mass on its own key."""
    d, L, W = 16, 24, 4
    n = L - W
    q = torch.zeros(1, 1, W, d)
    k = torch.zeros(1, 1, L, d)
    for i in range(W):
        q[0, 0, i, i] = 40.0
        k[0, 0, 2 + 3 * i, i] = 40.0
    prob = Problem(1, 1, 1, L, W, head_dim=d, dtype=oracle.F32)
    c = oracle.colsum(prob, gen.as_numpy(q), gen.as_numpy(k))
    for i in range(W):
        assert c[0, 0, 2 + 3 * i] == pytest.approx(1.0, abs=1e-9)
    assert n > 2 + 3 * (W - 1)


# ----------------------------------------------------------------------------- O5
@pytest.mark.parametrize("size", [1, 3, 5, 7, 15])
@pytest.mark.parametrize("n", [1, 2, 6, 50])
def test_pool_matches_library(size, n):
    x = torch.rand(n, dtype=torch.float64, generator=torch.Generator().manual_seed(size * 100 + n))
    mx = torch.nn.functional.max_pool1d(x.view(1, 1, n), size, stride=1, padding=size // 2).view(n)
    av = torch.nn.functional.avg_pool1d(x.view(1, 1, n), size, stride=1, padding=size // 2,
                                        count_include_pad=True).view(n)
    np.testing.assert_array_equal(oracle.pool1d(oracle.POOL_MAX, size, x.numpy()), mx.numpy())
    np.testing.assert_allclose(oracle.pool1d(oracle.POOL_AVG, size, x.numpy()), av.numpy(), rtol=1e-14)
    np.testing.assert_array_equal(oracle.pool1d(oracle.POOL_NONE, size, x.numpy()), x.numpy())


# ----------------------------------------------------------------------------- O4, O6
def test_head_table_hand_cases():
    """Eq. 6 inside a GQA group: one-hot weights return that head's scaled mass, a constant weight
    scales the group max, and G = 1 is the identity."""
    prob, q, k, _ = rand_case(4, Nu=1, H=4, Hkv=2, L=64, W=4)
    prob.pool_kind, prob.pool_size = oracle.POOL_NONE, 1
    qn, kn = gen.as_numpy(q), gen.as_numpy(k)
    c = oracle.colsum(prob, qn, kn)
    alpha = (prob.seq_len / prob.window) * c[..., : prob.n]
    w = np.array([[0.0, 1.0, 1.0, 0.0]], np.float32)
    s, cm = oracle.score(prob, qn, kn, w)
    np.testing.assert_allclose(s[0, 0], alpha[0, 1], rtol=1e-14)
    np.testing.assert_allclose(s[0, 1], alpha[0, 2], rtol=1e-14)
    w = np.full((1, 4), 1.25, np.float32)
    s, _ = oracle.score(prob, qn, kn, w)
    np.testing.assert_allclose(s[0, 0], 1.25 * np.maximum(alpha[0, 0], alpha[0, 1]), rtol=1e-14)
    np.testing.assert_allclose(cm[0], c[0].sum(0), rtol=1e-14)
    prob1 = Problem(1, 4, 4, 64, 4, head_dim=16, dtype=oracle.F32, pool_kind=oracle.POOL_NONE, pool_size=1)
    k4 = k.repeat_interleave(2, dim=1)
    s1, _ = oracle.score(prob1, qn, gen.as_numpy(k4), np.ones((1, 4), np.float32))
    np.testing.assert_allclose(s1[0], alpha[0], rtol=1e-14)


def test_score_pools_then_weights_then_maxes():
    """AVG pooling does not commute with the group max: the order is pool per head, weight, max."""
    prob, q, k, _ = rand_case(5, Nu=1, H=4, Hkv=2, L=80, W=4)
    prob.pool_kind, prob.pool_size = oracle.POOL_AVG, 5
    qn, kn = gen.as_numpy(q), gen.as_numpy(k)
    w = np.array([[0.7, 1.3, 1.1, 0.9]], np.float32)
    s, _ = oracle.score(prob, qn, kn, w)
    alpha = torch.from_numpy((prob.seq_len / prob.window) * oracle.colsum(prob, qn, kn)[..., : prob.n])
    pooled = torch.nn.functional.avg_pool1d(alpha, 5, stride=1, padding=2, count_include_pad=True).numpy()
    ref = (pooled[0] * w[0].astype(np.float64)[:, None]).reshape(2, 2, -1).max(1)
    np.testing.assert_allclose(s[0], ref, rtol=1e-13)


# ----------------------------------------------------------------------------- O7
def test_entropy_bucket_extremes():
    L, W, H, Hkv = 64, 4, 2, 1
    prob = Problem(1, H, Hkv, L, W, head_dim=16, budget_per_head=16, n_buckets=16)
    sens = np.linspace(0.8, 1.2, 16).astype(np.float32)
    scores = np.ones((1, Hkv, L - W))
    uni = np.full((1, L), W * H / L)
    out = oracle.budget(prob, scores, uni, sens)
    assert out["entropy"][0] == pytest.approx(math.log(L), rel=1e-13)
    assert out["bucket"][0] == 15 and out["tau"][0] == float(sens[15])
    hot = np.zeros((1, L))
    hot[0, 7] = W * H
    out = oracle.budget(prob, scores, hot, sens)
    assert out["entropy"][0] == 0.0 and out["bucket"][0] == 0
    two = np.zeros((1, L))
    two[0, 3] = two[0, 9] = W * H / 2          # entropy ln 2 -> ln2/ln64 = 1/6 -> bucket floor(16/6) = 2
    out = oracle.budget(prob, scores, two, sens)
    assert out["entropy"][0] == pytest.approx(math.log(2), rel=1e-13) and out["bucket"][0] == 2
    prob.bucket_override = 5
    assert oracle.budget(prob, scores, two, sens)["bucket"][0] == 5


def test_entropy_of_closed_form_mass():
    """q = 0: the mass is the closed form of test_closed_form_zero_queries; its entropy is computed here
    by hand from that form."""
    prob, q, k, _ = rand_case(6, Nu=1, H=2, Hkv=1, L=40, W=5)
    q = torch.zeros_like(q)
    s, cm = oracle.score(prob, gen.as_numpy(q), gen.as_numpy(k), np.ones((1, 2), np.float32))
    n, W, L, H = prob.n, prob.window, prob.seq_len, 2
    p = [sum(1.0 / (n + i + 1) for i in range(W)) / W] * n
    p += [sum(1.0 / (n + i + 1) for i in range(r, W)) / W for r in range(W)]
    ent = -sum(x * math.log(x) for x in p)
    out = oracle.budget(prob, s, cm, np.ones(16, np.float32))
    assert out["entropy"][0] == pytest.approx(ent, rel=1e-12)
    assert sum(p) == pytest.approx(1.0, abs=1e-14)


# ----------------------------------------------------------------------------- O8
def brute_allocate(n, f, P, dem):
    """Water level by exact rational interpolation between break points, then largest remainders."""
    dem = [int(x) for x in dem]
    clamp = lambda lam, dg: min(max(lam * dg, Fraction(f)), Fraction(n))
    S = lambda lam: sum(clamp(lam, dg) for dg in dem)
    bps = sorted({Fraction(0)} | {Fraction(f, dg) for dg in dem} | {Fraction(n, dg) for dg in dem})
    lam = None
    for a, b in zip(bps, bps[1:]):
        Sa, Sb = S(a), S(b)
        if Sa <= P <= Sb:
            lam = a if Sa == Sb else a + (b - a) * (P - Sa) / (Sb - Sa)
            break
    assert lam is not None
    x = [clamp(lam, dg) for dg in dem]
    assert sum(x) == P
    e = [math.floor(v) for v in x]
    left = P - sum(e)
    order = sorted(range(len(dem)), key=lambda g: (-(x[g] - e[g]), g))
    for g in order[:left]:
        assert x[g] != e[g]
        e[g] += 1
    return e


def test_allocate_matches_rational_brute_force():
    rng = np.random.default_rng(0)
    cases = 0
    for Hkv in (1, 2, 3, 4):
        for _ in range(400):
            n = int(rng.integers(1, 40))
            f = int(rng.integers(0, n + 1))
            P = int(rng.integers(f * Hkv, n * Hkv + 1))
            lo = max(f, 1)
            dem = rng.integers(lo, max(lo, n) + 1, Hkv)
            if rng.random() < 0.3:
                dem[rng.integers(0, Hkv)] = lo
            got = oracle.allocate(n, f, P, dem)
            want = brute_allocate(n, f, P, dem)
            assert list(got) == want, (n, f, P, dem)
            assert got.sum() == P and got.min() >= f and got.max() <= n
            cases += 1
    assert cases == 1600


def iterative_allocate(n, f, P, dem):
    """The budget clamp stated as a fixed-point loop (reading of the clamp-to-total rule): share the rows in
    proportion to the demands; pin every head whose share falls below the floor at the floor and take it out;
    when no head is below the floor, pin every head whose share exceeds the cap at the cap; repeat until nothing
    is pinned.  Exact integer comparisons; then floor plus largest remainders, ties to the lowest head."""
    dem = [int(x) for x in dem]
    active = list(range(len(dem)))
    e = [None] * len(dem)
    R = P
    while active:
        D = sum(dem[g] for g in active)
        low = [g for g in active if R * dem[g] < f * D]
        if low:
            for g in low:
                e[g] = f
            R -= f * len(low)
            active = [g for g in active if g not in low]
            continue
        high = [g for g in active if R * dem[g] > n * D]
        if high:
            for g in high:
                e[g] = n
            R -= n * len(high)
            active = [g for g in active if g not in high]
            continue
        break
    if active:
        D = sum(dem[g] for g in active)
        for g in active:
            e[g] = R * dem[g] // D
        left = R - sum(e[g] for g in active)
        for g in sorted(active, key=lambda g: (-((R * dem[g]) % D), g))[:left]:
            e[g] += 1
    return e


def test_allocate_matches_the_iterative_statement_at_workload_sizes():
    """Eight KV heads and prefixes up to 131040 (the workloads' sizes), where the rational brute force is too slow:
    the water-filling oracle against the fixed-point loop, an independent statement of the same rule."""
    rng = np.random.default_rng(5)
    cases = 0
    for Hkv, n, W in ((8, 32736, 32), (8, 131040, 32), (4, 65472, 64), (8, 2016, 32), (2, 2016, 32)):
        for _ in range(600):
            B = int(rng.choice([128, 512, 2048, int(rng.integers(W + 1, n))]))
            B = max(W + 1, min(B, n))
            f = int(rng.choice([0, 1, 8, int(rng.integers(0, B - W + 1))]))
            f = min(f, B - W)
            P = Hkv * (B - W)
            style = rng.integers(0, 4)
            if style == 0:      # counts of scores above a threshold: anywhere in [0, n]
                dem = rng.integers(0, n + 1, Hkv)
            elif style == 1:    # a few starved heads next to saturated ones
                dem = np.where(rng.random(Hkv) < 0.4, rng.integers(0, 4, Hkv), rng.integers(n // 2, n + 1, Hkv))
            elif style == 2:    # near-equal demands: the remainders decide
                dem = int(rng.integers(1, n)) + rng.integers(0, 3, Hkv)
            else:               # small demands: many heads at the floor or at the cap
                dem = rng.integers(0, 2 * (B - W) + 2, Hkv)
            dem = np.clip(dem, max(f, 1), n)
            got = list(oracle.allocate(n, f, P, dem))
            assert got == iterative_allocate(n, f, P, dem), (Hkv, n, f, P, dem)
            assert sum(got) == P and min(got) >= f and max(got) <= n
            cases += 1
    assert cases == 3000


def test_allocate_iterative_statement_agrees_with_rational_brute_force():
    """The two pins against each other on small cases (so that neither is only checked through the oracle)."""
    rng = np.random.default_rng(6)
    for _ in range(500):
        Hkv = int(rng.integers(1, 6))
        n = int(rng.integers(1, 40))
        f = int(rng.integers(0, n + 1))
        P = int(rng.integers(f * Hkv, n * Hkv + 1))
        dem = rng.integers(max(f, 1), max(f, 1, n) + 1, Hkv)
        assert iterative_allocate(n, f, P, dem) == brute_allocate(n, f, P, dem), (n, f, P, dem)


def test_allocate_two_sided_clamp_case():
    """A tiny demand next to a huge one: the low head sits at the floor, the high head at the cap."""
    assert list(oracle.allocate(10, 2, 18, [1, 1000])) == [8, 10]
    assert list(oracle.allocate(10, 2, 12, [1, 1000])) == [2, 10]
    assert list(oracle.allocate(100, 1, 30, [5, 5, 5])) == [10, 10, 10]
    assert list(oracle.allocate(100, 1, 31, [5, 5, 5])) == [11, 10, 10]     # ties: lowest head first
    assert list(oracle.allocate(100, 1, 32, [5, 5, 5])) == [11, 11, 10]


def test_budget_invariants_and_equal_demands():
    prob, q, k, _ = rand_case(7, Nu=3, H=8, Hkv=4, L=200, W=8)
    prob.budget_per_head, prob.floor_per_head = 40, 3
    qn, kn = gen.as_numpy(q), gen.as_numpy(k)
    hw = np.random.default_rng(1).uniform(0.5, 1.5, (3, 8)).astype(np.float32)
    s, cm = oracle.score(prob, qn, kn, hw)
    for ov in (-1, 0, 7, 15):
        prob.bucket_override = ov
        out = oracle.budget(prob, s, cm, np.linspace(0.5, 2.0, 16).astype(np.float32))
        b = out["budgets"]
        assert (b.sum(1) == 4 * 40).all()
        assert (b - 8 >= 3).all() and (b - 8 <= prob.n).all()
        assert (out["offsets"][:, 1:] - out["offsets"][:, :-1] == b).all() and (out["offsets"][:, 0] == 0).all()
        for u in range(3):
            for g in range(4):
                assert out["counts"][u, g] == int((s[u, g] >= out["tau"][u]).sum())
    # all-zero candidate counts -> uniform split
    out = oracle.budget(prob, s, cm, np.full(16, 1e9, np.float32))
    assert (out["counts"] == 0).all() and (out["budgets"] == 40).all()


# ----------------------------------------------------------------------------- O9
def test_select_matches_brute_force_sort():
    rng = np.random.default_rng(2)
    L, W, Hkv, Nu = 70, 6, 3, 2
    n = L - W
    prob = Problem(Nu, 3, Hkv, L, W, head_dim=16, budget_per_head=20)
    scores = rng.integers(0, 9, (Nu, Hkv, n)).astype(np.float64)      # many exact ties
    budgets = np.array([[20, 30, 10], [6, 48, 6]], np.int32)
    offsets = np.concatenate([np.zeros((Nu, 1), np.int32), budgets.cumsum(1).astype(np.int32)], 1)
    idx = oracle.select(prob, scores, budgets, offsets)
    for u in range(Nu):
        for g in range(Hkv):
            e = budgets[u, g] - W
            order = sorted(range(n), key=lambda t: (-scores[u, g, t], t))
            want = sorted(order[:e]) + list(range(n, L))
            got = idx[u, offsets[u, g]: offsets[u, g + 1]]
            assert list(got) == want
    const = np.ones((Nu, Hkv, n))
    idx = oracle.select(prob, const, budgets, offsets)
    assert list(idx[0, :20]) == list(range(14)) + list(range(n, L))    # constant scores: lowest indices win


# ----------------------------------------------------------------------------- O10 and the whole pass
def test_gather_is_direct_indexing():
    prob, q, k, v = rand_case(8, Nu=2, H=4, Hkv=2, L=64, W=4, dtype=oracle.BF16)
    prob.budget_per_head = 10
    kn, vn = gen.as_numpy(k), gen.as_numpy(v)
    budgets = np.array([[12, 8], [5, 15]], np.int32)
    offsets = np.array([[0, 12, 20], [0, 5, 20]], np.int32)
    rng = np.random.default_rng(3)
    idx = np.stack([np.concatenate([np.sort(rng.choice(64, b, replace=False)) for b in budgets[u]]) for u in range(2)])
    ko, vo = oracle.gather(prob, kn, vn, idx.astype(np.int32), budgets, offsets)
    for u in range(2):
        for g in range(2):
            sl = slice(offsets[u, g], offsets[u, g + 1])
            np.testing.assert_array_equal(ko[u, sl], kn[u, g, idx[u, sl]])
            np.testing.assert_array_equal(vo[u, sl], vn[u, g, idx[u, sl]])


def small_cfg(**kw):
    base = dict(n_layers=2, batch=1, n_q_heads=4, n_kv_heads=2, seq_len=512, window=16, budget_per_head=64,
                n_needles=4)
    base.update(kw)
    return gen.shrink(gen.CONFIGS["c2"], **base)


def problem_of(cfg, Nu):
    return Problem(Nu, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq_len, cfg.window, head_dim=cfg.head_dim,
                   dtype=oracle.BF16 if cfg.dtype == "bf16" else oracle.F32, pool_kind=cfg.pool_kind,
                   pool_size=cfg.pool_size, budget_per_head=cfg.budget_per_head, floor_per_head=cfg.floor_per_head,
                   n_buckets=cfg.n_buckets)


def test_full_budget_reproduces_fullkv():
    """B >= L keeps every row of every head in order: the compressed cache is the input, bit for bit."""
    cfg = small_cfg(seq_len=128, budget_per_head=128)
    b = gen.make_batch(cfg)
    prob = problem_of(cfg, cfg.n_units)
    out = oracle.compress(prob, *(gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w", "sens")))
    kn, vn = gen.as_numpy(b["k"]), gen.as_numpy(b["v"])
    np.testing.assert_array_equal(out["k_out"].reshape(kn.shape), kn)
    np.testing.assert_array_equal(out["v_out"].reshape(vn.shape), vn)
    assert (out["budgets"] == 128).all()
    prob.budget_per_head = 1000                                         # B > L: rows per head stay L
    out = oracle.compress(prob, *(gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w", "sens")))
    np.testing.assert_array_equal(out["k_out"].reshape(kn.shape), kn)


def check_needles(cfg, kept, needles, e):
    """Every planted key is retained when the head's prefix budget covers all needle neighbourhoods
    (MAX pooling spreads a needle's score over pool_size positions) and the sink's; with a smaller
    budget, everything retained from the prefix must lie in such a neighbourhood."""
    r = cfg.pool_size // 2
    hood = set(range(0, r + 1))
    for p in needles:
        hood |= set(range(p - r, p + r + 1))
    if e >= len(hood):
        assert all(p in kept for p in needles)
    else:
        assert all(t in hood for t in kept if t < cfg.n)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_whole_pass_invariants_and_needles(dtype):
    cfg = small_cfg(dtype=dtype)
    b = gen.make_batch(cfg)
    prob = problem_of(cfg, cfg.n_units)
    out = oracle.compress(prob, *(gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w", "sens")))
    L, W, B, Hkv = cfg.seq_len, cfg.window, cfg.budget_per_head, cfg.n_kv_heads
    assert (out["budgets"].sum(1) == Hkv * B).all()
    for u in range(cfg.n_units):
        for g in range(Hkv):
            idx = out["indices"][u, out["offsets"][u, g]: out["offsets"][u, g + 1]]
            assert len(idx) == out["budgets"][u, g]
            assert (np.diff(idx) > 0).all() and idx[0] >= 0 and idx[-1] == L - 1
            assert list(idx[-W:]) == list(range(L - W, L))              # the window is always kept
            kept = set(idx.tolist())
            assert 0 in kept                                            # the sink
            check_needles(cfg, kept, b["needles"][u, g].tolist(), len(idx) - W)


def test_discarded_mass_identity_and_tail_bound():
    """Eq. A2: the L1 distance between an attention row and its renormalised restriction to the kept
    set is exactly twice the discarded mass; Eq. 9 follows (Frobenius <= 2 sqrt(rows) eps_tail)."""
    cfg = small_cfg(n_layers=1)
    b = gen.make_batch(cfg)
    prob = problem_of(cfg, 1)
    qn, kn = gen.as_numpy(b["q"]), gen.as_numpy(b["k"])
    out = oracle.compress(prob, qn, kn, gen.as_numpy(b["v"]), gen.as_numpy(b["head_w"]), gen.as_numpy(b["sens"]))
    A = oracle.window_attention(prob, qn, kn)
    kept = oracle.kept_mass(prob, qn, kn, out["indices"], out["budgets"], out["offsets"])
    G = cfg.n_q_heads // cfg.n_kv_heads
    for h in range(cfg.n_q_heads):
        g = h // G
        S = out["indices"][0, out["offsets"][0, g]: out["offsets"][0, g + 1]]
        mask = np.zeros(cfg.seq_len, bool)
        mask[S] = True
        m = A[0, h][:, ~mask].sum(1)
        np.testing.assert_allclose(1.0 - kept[0, h], m, atol=1e-13)
        ptil = np.where(mask, A[0, h], 0.0) / (1.0 - m)[:, None]
        l1 = np.abs(A[0, h] - ptil).sum(1)
        np.testing.assert_allclose(l1, 2.0 * m, rtol=1e-9, atol=1e-14)
        fro = np.linalg.norm(A[0, h] - ptil)
        eps_tail = math.sqrt((m ** 2).mean())
        assert fro <= 2.0 * math.sqrt(cfg.window) * eps_tail + 1e-12
        assert (m >= 0).all() and (m < 1).all()


def test_operating_points_from_the_paper():
    """The kept fractions and fixed-ratio budgets the paper prints (tests/golden/operating_points.txt)."""
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "operating_points.txt")) if ln.strip() and ln[0] != "#"]
    for L, kept, pct in rows:
        L, kept = int(L), int(kept)
        if pct != "-":
            assert abs(100.0 * kept / L - float(pct)) < 0.006           # printed with two decimals (truncated)
        else:
            assert kept * 64 == L                                       # 512 / 32768
    c2, c4 = gen.CONFIGS["c2"], gen.CONFIGS["c4"]
    assert (str(c2.seq_len), str(c2.budget_per_head), "1.56") in [tuple(r) for r in rows]
    assert (str(c4.seq_len), str(c4.budget_per_head), "-") in [tuple(r) for r in rows]


# ---------------------------------------------------------------------------- O5b: value-norm ratio (Eq. 4)
def test_vnorm_hand_example():
    """Rows of norms 5, 0, 10, 1 (3-4-5 triangles): mean 4, so rho = 1.25, 0, 2.5, 0.25; with eps = 1 the
    denominator is 5 (Alg. 1 (B): r / (mu + eps))."""
    v = np.zeros((1, 1, 4, 8), np.float32)
    v[0, 0, 0, :2] = (3, 4)
    v[0, 0, 2, 3:5] = (6, 8)
    v[0, 0, 3, 7] = -1
    prob = Problem(1, 1, 1, 4, 1, head_dim=8, dtype=oracle.F32)
    np.testing.assert_allclose(oracle.vnorm(prob, v, eps=0.0)[0, 0], [1.25, 0.0, 2.5, 0.25], rtol=1e-15)
    np.testing.assert_allclose(oracle.vnorm(prob, v, eps=1.0)[0, 0], [1.0, 0.0, 2.0, 0.2], rtol=1e-15)


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_vnorm_identities_and_library_norm(dtype):
    """mean_t rho = mu / (mu + eps) (Eq. 4 divides by the mean); eps = 0 makes rho invariant to the scale of V
    (the point of the 'head-relative normalisation'); rows of equal norm all get mu / (mu + eps); and the norms
    agree with torch.linalg.vector_norm on the exactly widened inputs."""
    prob, _, _, v = rand_case(11, Nu=2, H=4, Hkv=2, L=70, W=6, d=16, dtype=dtype)
    vn = gen.as_numpy(v)
    r = torch.linalg.vector_norm(v.double(), dim=-1).numpy()              # [Nu,Hkv,L]
    mu = r.mean(-1, keepdims=True)
    for eps in (0.0, 1e-6, 0.5):
        rho = oracle.vnorm(prob, vn, eps=eps)
        np.testing.assert_allclose(rho, r / (mu + eps), rtol=1e-13)
        np.testing.assert_allclose(rho.mean(-1), (mu / (mu + eps))[..., 0], rtol=1e-13)
    if dtype == oracle.F32:
        np.testing.assert_allclose(oracle.vnorm(prob, 4.0 * vn, eps=0.0), oracle.vnorm(prob, vn, eps=0.0), rtol=1e-13)
        unit = vn / np.linalg.norm(vn, axis=-1, keepdims=True) * 3.0        # every row has norm 3 (to fp32 rounding)
        np.testing.assert_allclose(oracle.vnorm(prob, unit.astype(np.float32), eps=1.0), 0.75, rtol=1e-6)


@pytest.mark.parametrize("pool_kind,pool_size", [(oracle.POOL_NONE, 1), (oracle.POOL_MAX, 5), (oracle.POOL_AVG, 3)])
def test_score_applies_the_value_norm_after_pooling_and_before_the_head_max(pool_kind, pool_size):
    """u_h = pool(alpha_h) * rho_g (Eq. 4; the pooling smooths the attention mass only), then Eq. 6's weighted
    max over the group.  rho is shared by a group's heads and non-negative, so the score equals rho times the
    score without it -- which pooling alpha * rho instead would break -- and the column mass does not change."""
    prob, q, k, v = rand_case(5, Nu=2, H=4, Hkv=2, L=80, W=8, d=16)
    v[:, :, 10] *= 25.0                                                    # one loud value row per head
    prob.pool_kind, prob.pool_size = pool_kind, pool_size
    qn, kn, vn = gen.as_numpy(q), gen.as_numpy(k), gen.as_numpy(v)
    w = (0.5 + torch.rand(2, 4, generator=torch.Generator().manual_seed(1))).numpy().astype(np.float32)
    plain, cm0 = oracle.score(prob, qn, kn, w)
    prob.value_norm, prob.value_norm_eps = True, 1e-3
    rho = oracle.vnorm(prob, vn)
    with_rho, cm1 = oracle.score(prob, qn, kn, w, v=vn)
    np.testing.assert_allclose(with_rho, plain * rho[:, :, :prob.n], rtol=1e-13)
    np.testing.assert_array_equal(cm0, cm1)
    if pool_size > 1:      # the other order of the two steps gives something else next to the loud row
        assert not np.allclose(with_rho[:, :, 9], (plain * rho[:, :, :prob.n])[:, :, 10])
    # the whole pass uses the same scores
    prob.budget_per_head = 24
    out = oracle.compress(prob, qn, kn, vn, w, gen.as_numpy(gen.make_sens(gen.CONFIGS["c1"])))
    np.testing.assert_array_equal(out["scores"], with_rho)


# ---------------------------------------------------------------------------- the paper's own selection (Eq. 6 over all heads, Eq. 8)
def test_shared_elastic_selection_against_brute_force():
    """shared_elastic: u^[t] = max over ALL heads of w_h * u_h[t] (Eq. 6), the set is Eq. 8's -- every candidate
    when they fit the budget, else the Top-B of them -- and all KV heads keep it.  Built here from the per-head
    mode's scores by numpy set operations and a stable sort."""
    prob, q, k, v = rand_case(21, Nu=3, H=8, Hkv=4, L=120, W=8, d=16)
    prob.pool_size, prob.budget_per_head, prob.floor_per_head = 1, 40, 0
    qn, kn, vn = gen.as_numpy(q), gen.as_numpy(k), gen.as_numpy(v)
    w = (0.5 + torch.rand(3, 8, generator=torch.Generator().manual_seed(2))).numpy().astype(np.float32)
    per_head, cm = oracle.score(prob, qn, kn, w)
    prob.shared_elastic = True
    shared, cm2 = oracle.score(prob, qn, kn, w)
    np.testing.assert_array_equal(shared, np.broadcast_to(per_head.max(1, keepdims=True), per_head.shape))
    np.testing.assert_array_equal(cm, cm2)
    u_hat = shared[:, 0]
    n, W, B = prob.n, prob.window, prob.budget_per_head
    # three thresholds: none, few (elastic under-retention) and many candidates (clamped to the budget)
    for q_tau, regime in ((1.01, "none"), (0.9, "few"), (0.3, "many")):
        tau = np.float32(np.quantile(u_hat, q_tau) if q_tau <= 1 else u_hat.max() * 2)
        sens = np.full(prob.n_buckets, tau, np.float32)
        bud = oracle.budget(prob, shared, cm, sens)
        idx = oracle.select(prob, shared, bud["budgets"], bud["offsets"])
        for u in range(3):
            cand = np.nonzero(u_hat[u] >= np.float64(tau))[0]
            if len(cand) <= B - W:
                want = cand
                assert regime in ("none", "few")
            else:
                order = np.argsort(-u_hat[u], kind="stable")         # ties to the lowest index
                want = np.sort(order[:B - W])
                assert regime == "many"
            want = np.concatenate([want, np.arange(n, n + W)])
            assert (bud["budgets"][u] == len(want)).all()
            for g in range(4):
                got = idx[u, bud["offsets"][u, g]: bud["offsets"][u, g + 1]]
                np.testing.assert_array_equal(got, want)
        if regime == "none":
            assert (bud["budgets"] == W).all()
    # the floor bounds the prefix part from below even with no candidate
    prob.floor_per_head = 5
    bud = oracle.budget(prob, shared, cm, np.full(prob.n_buckets, 1e9, np.float32))
    assert (bud["budgets"] == W + 5).all()
    # whole pass: every KV head gathers the same positions
    prob.floor_per_head = 0
    out = oracle.compress(prob, qn, kn, vn, w, np.full(prob.n_buckets, np.float32(np.quantile(u_hat, 0.9)), np.float32))
    for u in range(3):
        rows = out["budgets"][u, 0]
        sets = [out["indices"][u, out["offsets"][u, g]: out["offsets"][u, g] + rows] for g in range(4)]
        assert all((s == sets[0]).all() for s in sets)
        for g in range(4):
            np.testing.assert_array_equal(out["k_out"][u, out["offsets"][u, g]: out["offsets"][u, g] + rows],
                                          kn[u, g, sets[0]])


def test_shared_elastic_with_one_kv_head_and_a_full_pool_equals_the_per_head_mode():
    """With a single KV head and more candidates than the budget both modes keep the Top-(B - W)."""
    prob, q, k, v = rand_case(22, Nu=2, H=4, Hkv=1, L=90, W=6, d=16)
    prob.budget_per_head, prob.floor_per_head = 30, 0
    qn, kn = gen.as_numpy(q), gen.as_numpy(k)
    w = np.ones((2, 4), np.float32)
    sens = np.zeros(prob.n_buckets, np.float32)             # every position is a candidate
    a_sc, a_cm = oracle.score(prob, qn, kn, w)
    a = oracle.budget(prob, a_sc, a_cm, sens)
    prob.shared_elastic = True
    b_sc, b_cm = oracle.score(prob, qn, kn, w)
    b = oracle.budget(prob, b_sc, b_cm, sens)
    np.testing.assert_array_equal(a_sc, b_sc)
    np.testing.assert_array_equal(a["budgets"], b["budgets"])
    assert (b["budgets"] == 30).all()


# ---------------------------------------------------------------------------- prompt-global alpha (Alg. 1 (A))
def test_global_alpha_identities():
    """global_alpha: A-bar is the mean attention over all layers and heads of the prompt, so
    (a) every unit of a prompt reports the same column mass, which sums to W H (each of the W H softmax rows of a
        unit sums to one) -- the reason alpha has mean one over the L keys (text after Eq. 4);
    (b) with unit weights, no pooling and no value norm, every head's score IS alpha = (L/W) mass / H;
    (c) alpha does not depend on the order of the prompt's layers, nor on the other prompt's data;
    (d) a prompt of one layer with one head gives the per-head mode's scores;
    (e) the weights enter as Eq. 6's max inside the group: score = alpha * max_{h in g} w_h."""
    prob, q, k, v = rand_case(31, Nu=4, H=4, Hkv=2, L=64, W=8, d=16)
    prob.pool_kind, prob.pool_size = oracle.POOL_NONE, 1
    qn, kn = gen.as_numpy(q), gen.as_numpy(k)
    ones = np.ones((4, 4), np.float32)
    per_head, cm_units = oracle.score(prob, qn, kn, ones)
    prob.global_alpha, prob.units_per_prompt = True, 2
    sc, cm = oracle.score(prob, qn, kn, ones)
    L, W, H, n = 64, 8, 4, prob.n
    np.testing.assert_allclose(cm.sum(-1), W * H, rtol=1e-12)                                  # (a)
    np.testing.assert_array_equal(cm[0], cm[1])
    np.testing.assert_array_equal(cm[2], cm[3])
    np.testing.assert_allclose(cm[0], (cm_units[0] + cm_units[1]) / 2, rtol=1e-13)             # mean over the layers
    alpha = (L / W) * cm / H
    np.testing.assert_allclose(alpha.mean(-1), 1.0, rtol=1e-12)
    for g in range(2):
        np.testing.assert_allclose(sc[:, g], alpha[:, :n], rtol=1e-13)                         # (b)
    perm = [1, 0, 2, 3]
    sc_p, _ = oracle.score(prob, qn[perm], kn[perm], ones)
    np.testing.assert_allclose(sc_p[0], sc[0], rtol=1e-13)                                     # (c)
    np.testing.assert_array_equal(sc_p[2:], sc[2:])
    w = (0.5 + torch.rand(4, 4, generator=torch.Generator().manual_seed(3))).numpy().astype(np.float32)
    sc_w, _ = oracle.score(prob, qn, kn, w)
    wmax = w.astype(np.float64).reshape(4, 2, 2).max(-1)
    np.testing.assert_allclose(sc_w, alpha[:, None, :n] * wmax[:, :, None], rtol=1e-13)        # (e)
    prob1, q1, k1, _ = rand_case(32, Nu=3, H=1, Hkv=1, L=40, W=4, d=16)
    a, _ = oracle.score(prob1, gen.as_numpy(q1), gen.as_numpy(k1), np.ones((3, 1), np.float32))
    prob1.global_alpha, prob1.units_per_prompt = True, 1
    b, _ = oracle.score(prob1, gen.as_numpy(q1), gen.as_numpy(k1), np.ones((3, 1), np.float32))
    np.testing.assert_allclose(a, b, rtol=1e-13)                                               # (d)


def test_global_alpha_pools_alpha_and_shares_the_risk_coordinate():
    """The pooling acts on the prompt's alpha (library max pooling), and the entropy bucket is one per prompt."""
    prob, q, k, v = rand_case(33, Nu=4, H=4, Hkv=2, L=64, W=8, d=16)
    prob.pool_kind, prob.pool_size = oracle.POOL_MAX, 5
    prob.global_alpha, prob.units_per_prompt = True, 2
    qn, kn = gen.as_numpy(q), gen.as_numpy(k)
    sc, cm = oracle.score(prob, qn, kn, np.ones((4, 4), np.float32))
    alpha = torch.from_numpy((64 / 8) * cm[:, :prob.n] / 4)
    pooled = torch.nn.functional.max_pool1d(alpha[:, None], 5, 1, 2)[:, 0].numpy()
    np.testing.assert_allclose(sc[:, 0], pooled, rtol=1e-13)
    bud = oracle.budget(prob, sc, cm, gen.as_numpy(gen.make_sens(gen.CONFIGS["c1"])))
    assert bud["bucket"][0] == bud["bucket"][1] and bud["bucket"][2] == bud["bucket"][3]
    assert bud["entropy"][0] == bud["entropy"][1]


# ---------------------------------------------------------------------------- decode-side check (Prop. 4.1)
@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_attend_against_library_softmax_and_the_discarded_mass_identity(dtype):
    """Full attention of decode queries equals torch's fp64 softmax attention; over the gathered rows it is the
    renormalised restriction p~ of Prop. 4.1, the kept mass is exp(lse_S - lse_all), |p - p~|_1 = 2 m (Eq. A2),
    and keeping every row changes nothing."""
    prob, q, k, v = rand_case(41, Nu=2, H=4, Hkv=2, L=60, W=6, d=16, dtype=dtype)
    g = torch.Generator().manual_seed(4)
    qd = torch.randn(2, 4, 3, 16, generator=g)
    if dtype == oracle.BF16:
        qd = qd.bfloat16()
    kk, vv = k.double().repeat_interleave(2, 1), v.double().repeat_interleave(2, 1)       # [Nu,H,L,d]
    x = torch.einsum("uhjd,uhtd->uhjt", qd.double(), kk) / 4.0
    p = torch.softmax(x, -1)
    out, lse = oracle.attend(prob, gen.as_numpy(qd), gen.as_numpy(k), gen.as_numpy(v))
    np.testing.assert_allclose(out, torch.einsum("uhjt,uhtd->uhjd", p, vv).numpy(), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lse, torch.logsumexp(x, -1).numpy(), rtol=1e-12)
    # a selection by the retention pass, then attention over what it gathered
    w = np.ones((2, 4), np.float32)
    sel = oracle.compress(prob, gen.as_numpy(q), gen.as_numpy(k), gen.as_numpy(v), w, np.zeros(prob.n_buckets, np.float32))
    out_c, lse_c = oracle.attend(prob, gen.as_numpy(qd), sel["k_out"], sel["v_out"], sel["budgets"], sel["offsets"])
    for u in range(2):
        for h in range(4):
            gq = h // 2
            S = sel["indices"][u, sel["offsets"][u, gq]: sel["offsets"][u, gq + 1]]
            pS = p[u, h][:, S]                                   # [n_dec, |S|]
            kept = pS.sum(-1).numpy()
            np.testing.assert_allclose(np.exp(lse_c[u, h] - lse[u, h]), kept, rtol=1e-11)
            p_tilde = torch.zeros_like(p[u, h])
            p_tilde[:, S] = pS / pS.sum(-1, keepdim=True)
            np.testing.assert_allclose((p[u, h] - p_tilde).abs().sum(-1).numpy(), 2 * (1 - kept), rtol=1e-9, atol=1e-13)
            np.testing.assert_allclose(out_c[u, h], (p_tilde @ vv[u, h]).numpy(), rtol=1e-10, atol=1e-13)
    prob.budget_per_head = 60                                    # FullKV: the compressed cache is the cache
    full = oracle.compress(prob, gen.as_numpy(q), gen.as_numpy(k), gen.as_numpy(v), w, np.zeros(prob.n_buckets, np.float32))
    out_f, lse_f = oracle.attend(prob, gen.as_numpy(qd), full["k_out"], full["v_out"], full["budgets"], full["offsets"])
    np.testing.assert_allclose(out_f, out, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse_f, lse, rtol=1e-13)


# ----------------------------------------------------------------------------- the gate table (Sec. 4.3, Alg. 1 (D))
def test_gate_table_lookup_reaches_every_cell():
    """tau = T_gate[l, b_ent, b_ppl, B_l] (Alg. 1 (D)) on the paper's 20 x 4 entropy x perplexity grid: a hand-built
    table with a different value in every cell; the entropy bin is forced through bucket_override and the other
    coordinates come per unit, so every cell of the grid is reached and must come back as the threshold."""
    n_layers, n_ent, n_ppl, n_bud = 3, 20, 4, 2
    cells = n_layers * n_ent * n_ppl * n_bud
    table = (0.8 + 0.2 * np.random.default_rng(3).permutation(cells) / cells).astype(np.float32)
    table = table.reshape(n_layers, n_ent, n_ppl, n_bud)
    assert len(set(table.ravel().tolist())) == cells
    prob, q, k, _ = rand_case(21, Nu=n_layers * n_bud, H=4, Hkv=2, L=64, W=8)
    s, cm = oracle.score(prob, gen.as_numpy(q), gen.as_numpy(k), np.ones((prob.n_units, 4), np.float32))
    prob.n_buckets, prob.gate_layers, prob.ppl_bins, prob.budget_levels = n_ent, n_layers, n_ppl, n_bud
    seen = set()
    for b_ent in range(n_ent):
        for b_ppl in range(n_ppl):
            coords = [(u // n_bud, b_ppl, u % n_bud) for u in range(prob.n_units)]
            prob.gate_coords, prob.bucket_override = coords, b_ent
            out = oracle.budget(prob, s, cm, table)
            for u, (l, p, b) in enumerate(coords):
                assert out["tau"][u] == table[l, b_ent, p, b]
                # and the threshold is the one the counts were taken with
                assert (out["counts"][u] == (s[u] >= float(table[l, b_ent, p, b])).sum(-1)).all()
                seen.add((l, b_ent, p, b))
    assert len(seen) == cells


def test_gate_table_takes_its_entropy_bin_from_the_window_mass():
    """Without an override the first table axis is the entropy bin of Eq. 7: uniform mass gives the last of the
    20 bins, mass on one position the first."""
    L, W, H = 50, 4, 2
    prob = Problem(1, H, 1, L, W, head_dim=16, dtype=oracle.F32, budget_per_head=20, n_buckets=20,
                   gate_layers=1, ppl_bins=4, budget_levels=1, gate_coords=[(0, 2, 0)])
    table = np.arange(80, dtype=np.float32).reshape(1, 20, 4, 1)
    scores = np.zeros((1, 1, L - W))
    uniform = np.full((1, L), W * H / L)
    assert oracle.budget(prob, scores, uniform, table)["tau"][0] == table[0, 19, 2, 0]
    one_hot = np.zeros((1, L))
    one_hot[0, 7] = W * H
    assert oracle.budget(prob, scores, one_hot, table)["tau"][0] == table[0, 0, 2, 0]


def test_gate_coordinates_out_of_range_are_refused():
    prob, q, k, _ = rand_case(22, Nu=1)
    s, cm = oracle.score(prob, gen.as_numpy(q), gen.as_numpy(k), np.ones((1, 4), np.float32))
    prob.gate_layers, prob.ppl_bins, prob.budget_levels = 2, 4, 1
    table = np.ones((2, prob.n_buckets, 4, 1), np.float32)
    for bad in [(2, 0, 0), (0, 4, 0), (0, 0, 1), (-1, 0, 0)]:
        prob.gate_coords = [bad]
        with pytest.raises(RuntimeError):
            oracle.budget(prob, s, cm, table)


@pytest.mark.parametrize("n_src,n_dst", [(32, 32), (32, 28), (32, 40), (32, 80), (2, 7), (5, 1), (1, 6)])
def test_depth_map_is_relative_depth_interpolation(n_src, n_dst):
    """Reuse of a table compiled for one depth on a model of another (the appendix on cross-architecture use):
    numpy's piecewise-linear interpolation over relative depth is the same map; same depth is the identity, first
    and last layers map onto first and last, and a table that rises with depth still rises."""
    rng = np.random.default_rng(n_src * 100 + n_dst)
    src = rng.uniform(0.8, 1.0, (n_src, 20, 4)).astype(np.float32)
    got = oracle.depth_map(src, n_dst)
    assert got.shape == (n_dst, 20, 4) and got.dtype == np.float32
    xs = np.linspace(0.0, 1.0, n_src) if n_src > 1 else np.zeros(1)
    xd = np.linspace(0.0, 1.0, n_dst) if n_dst > 1 else np.zeros(1)
    want = np.stack([np.interp(xd, xs, src[:, i, j].astype(np.float64)) for i in range(20) for j in range(4)], -1)
    np.testing.assert_allclose(got.reshape(n_dst, 80), want, rtol=1e-6, atol=0)
    if n_dst == n_src:
        np.testing.assert_array_equal(got, src)
    np.testing.assert_array_equal(got[0], src[0])
    if n_dst > 1:
        np.testing.assert_array_equal(got[-1], src[-1])
    rising = np.sort(src, axis=0)
    assert (np.diff(oracle.depth_map(rising, n_dst).astype(np.float64), axis=0) >= 0).all()
    # a table that is linear in depth stays linear in relative depth (closed form)
    lin = (0.8 + 0.2 * np.arange(n_src) / max(n_src - 1, 1)).astype(np.float32).reshape(n_src, 1)
    if n_src > 1 and n_dst > 1:
        np.testing.assert_allclose(oracle.depth_map(lin, n_dst)[:, 0], 0.8 + 0.2 * np.arange(n_dst) / (n_dst - 1),
                                   rtol=1e-6)
