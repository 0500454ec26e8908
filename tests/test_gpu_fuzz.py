"""Seeded random shapes and parameters: the fused GPU pass against the oracle's steps run on the GPU's own
scores (exact for budgets and indices) and against the oracle's scores (tolerance), with the optional modes mixed in."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_08686_b200 import inputs as gen
from test_gpu_parity import SCORE_RTOL, check_gather, params_of, problem_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_08686_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def draw(seed):
    r = np.random.default_rng(seed)
    Hkv = int(r.choice([1, 2, 3, 4, 8]))
    G = int(r.choice([1, 2, 4, 7]))
    W = int(r.choice([1, 5, 16, 32, 64]))
    L = int(r.integers(max(W + 40, 130), 2600))
    dtype = str(r.choice(["bf16", "bf16", "f32"]))
    pool_kind = int(r.choice([0, 1, 1, 2]))
    pool_size = 1 if pool_kind == 0 else int(r.choice([1, 3, 5, 7, 15]))
    budget = int(r.integers(W + 8, min(L + 50, W + 400)))
    n = L - W
    floor = int(r.integers(0, max(1, min(9, budget - W)))) if budget < L else 0
    layers = int(r.integers(1, 4)) * 2
    modes = dict(value_norm=bool(r.integers(0, 2)), shared_elastic=bool(r.integers(0, 4) == 0),
                 global_alpha=bool(r.integers(0, 4) == 0), units_per_prompt=2)
    # a third of the cases take their threshold from the four-axis gate table; every case carries its own scheduling
    # settings (they must not change any result)
    modes["gate"] = (int(r.integers(1, 5)), int(r.integers(1, 5)), int(r.integers(1, 4))) if r.integers(0, 3) == 0 else None
    modes["tuning"] = dict(run_tiles=int(r.integers(1, 41)), l2_hints=int(r.integers(0, 2)), pdl=int(r.integers(0, 2)),
                           group_fuse=int(r.integers(0, 2)))
    cfg = gen.shrink(gen.CONFIGS["c2"], config_id=100 + seed, n_layers=layers, batch=1, n_q_heads=Hkv * G, n_kv_heads=Hkv,
                     seq_len=L, window=W, pool_kind=pool_kind, pool_size=pool_size, budget_per_head=budget,
                     floor_per_head=floor, n_needles=2 if n > 64 else 0, dtype=dtype, n_buckets=int(r.choice([1, 7, 16])))
    return cfg, modes


@pytest.mark.parametrize("seed", range(100))
def test_random_case(B, seed):
    cfg, modes = draw(seed)
    gate, tuning = modes.pop("gate", None), modes.pop("tuning", None)
    Nu = cfg.n_units
    b = gen.make_batch(cfg, "cpu")
    # thresholds near the bulk of the scores, so that the candidate counts differ between heads
    prob = problem_of(cfg, Nu, **modes)
    qn, kn, vn, hw = (gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w"))
    sc, cm = oracle.score(prob, qn, kn, hw, v=vn if modes["value_norm"] else None)
    rs = np.random.default_rng(seed)
    coords, gate_kw = None, {}
    if gate is None:
        qs = np.quantile(sc, np.linspace(0.3, 0.995, cfg.n_buckets)).astype(np.float32)
        sens = torch.from_numpy(qs[rs.permutation(cfg.n_buckets)].copy())
    else:       # T_gate[layer, entropy bin, perplexity bin, budget level], thresholds from the same quantile range
        n_l, n_p, n_b = gate
        cells = n_l * cfg.n_buckets * n_p * n_b
        qs = np.quantile(sc, np.linspace(0.3, 0.995, cells)).astype(np.float32)
        sens = torch.from_numpy(qs[rs.permutation(cells)].reshape(n_l, cfg.n_buckets, n_p, n_b).copy())
        coords = np.stack([rs.integers(0, n_l, Nu), rs.integers(0, n_p, Nu), rs.integers(0, n_b, Nu)], 1).astype(np.int32)
        gate_kw = dict(gate_layers=n_l, ppl_bins=n_p, budget_levels=n_b)
    P = params_of(B, prob)
    for f in ("value_norm", "shared_elastic", "global_alpha", "units_per_prompt"):
        setattr(P, f, modes[f])
    if gate is not None:
        P.n_gate_layers, P.n_ppl_bins, P.n_budget_levels = gate
    out = B.compress(*(b[x].cuda() for x in ("q", "k", "v", "head_w")), sens.cuda(), P, want_scores=True,
                     gate_coords=None if coords is None else torch.from_numpy(coords).cuda(),
                     tuning=None if tuning is None else B.make_tuning(**tuning))
    assert B.ckv_device_status(out["ws"]) == B.OK
    gs = out["scores"].double().cpu().numpy()
    rel = np.abs(gs - sc) / np.maximum(np.abs(sc), 1e-20)
    assert rel.max() <= SCORE_RTOL, (rel.max(), cfg, modes)
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    bucket = out["bucket"].cpu().numpy()
    for u in range(Nu):
        prob_u = problem_of(cfg, 1, bucket_override=int(bucket[u]), shared_elastic=modes["shared_elastic"],
                            gate_coords=None if coords is None else coords[u:u + 1], **gate_kw)
        mine = oracle.budget(prob_u, gs[u:u + 1], cm[u:u + 1], sens.numpy())
        assert (mine["budgets"][0] == bud[u]).all(), (u, mine["budgets"], bud[u], cfg, modes)
    want = oracle.select(prob, gs, bud, off)
    for u in range(Nu):
        np.testing.assert_array_equal(idx[u, :off[u, -1]], want[u, :off[u, -1]])
    check_gather(b["k"], b["v"], out["k_out"], out["v_out"], idx, off, prob)


def draw_long(seed):
    r = np.random.default_rng(1000 + seed)
    Hkv, G = int(r.choice([1, 2])), int(r.choice([1, 4, 7]))
    W = int(r.choice([16, 32, 64]))
    L = int(r.integers(30000, 80000))
    pool_kind = int(r.choice([1, 2]))
    cfg = gen.shrink(gen.CONFIGS["c4" if seed % 2 else "c2"], config_id=200 + seed, n_layers=2, batch=1,
                     n_q_heads=Hkv * G, n_kv_heads=Hkv, seq_len=L, window=W, pool_kind=pool_kind,
                     pool_size=int(r.choice([3, 7])), budget_per_head=int(r.integers(W + 64, 3000)),
                     floor_per_head=int(r.integers(0, 9)), n_needles=8)
    modes = dict(value_norm=bool(r.integers(0, 2)), shared_elastic=False, global_alpha=bool(r.integers(0, 3) == 0),
                 units_per_prompt=2, gate=(2, 4, 2) if seed % 3 == 0 else None,
                 tuning=dict(run_tiles=int(r.integers(2, 33)), pdl=int(r.integers(0, 2))))
    return cfg, modes


@pytest.mark.parametrize("seed", range(8))
def test_random_long_case(B, seed, monkeypatch):
    """The same at lengths that take the selection's cluster paths and many key tiles per chunk."""
    monkeypatch.setattr("test_gpu_fuzz.draw", lambda s: draw_long(s))
    test_random_case(B, seed)
