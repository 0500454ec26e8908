"""GPU parity of the paper's own selection mode (Eq. 6 over all heads of the unit, Eq. 8's elastic candidate
pool, one set shared by the KV heads) against the oracle, through the C ABI."""
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


def se_params(B, prob):
    P = params_of(B, prob)
    P.shared_elastic = True
    P.value_norm, P.value_norm_eps = bool(prob.value_norm), float(prob.value_norm_eps)
    return P


@pytest.mark.parametrize("cfg_name,L,value_norm", [("c1", 2048, False), ("c2", 4096, False), ("c2", 3000, True),
                                                   ("c5", 4096, False)])
@pytest.mark.parametrize("regime", ["none", "few", "many"])
def test_shared_elastic_whole_pass(B, cfg_name, L, value_norm, regime):
    cfg = gen.shrink(gen.CONFIGS[cfg_name], n_layers=2, batch=1, seq_len=L, budget_per_head=128, n_needles=4,
                     floor_per_head=0)
    b = gen.make_batch(cfg, "cpu")
    prob = problem_of(cfg, 2, shared_elastic=True, value_norm=value_norm)
    qn, kn, vn, hw = (gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w"))
    sc, cm = oracle.score(prob, qn, kn, hw, v=vn if value_norm else None)
    assert (sc == sc[:, :1]).all()
    W, n, Hkv, Bud = cfg.window, cfg.n, cfg.n_kv_heads, cfg.budget_per_head
    # one threshold for all buckets: above every score, at the 40-th largest, at the median
    tau = {"none": sc.max() * 2, "few": np.sort(sc[:, 0].ravel())[-80], "many": np.median(sc)}[regime]
    sens = torch.full((cfg.n_buckets,), float(tau))
    out = B.compress(*(b[x].cuda() for x in ("q", "k", "v", "head_w")), sens.cuda(), se_params(B, prob),
                     want_scores=True)
    assert B.ckv_device_status(out["ws"]) == B.OK
    gs = out["scores"].double().cpu().numpy()
    assert (gs == gs[:, :1]).all()
    rel = np.abs(gs - sc) / np.maximum(np.abs(sc), 1e-20)
    assert rel.max() <= SCORE_RTOL, rel.max()
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    # the oracle's budget and selection steps on the GPU's own scores: exact
    mine = oracle.budget(prob, gs, cm, sens.numpy())
    np.testing.assert_array_equal(bud, mine["budgets"])
    np.testing.assert_array_equal(off, mine["offsets"])
    want = oracle.select(prob, gs, bud, off)
    for u in range(2):
        kept = bud[u, 0]
        assert (bud[u] == kept).all() and off[u, Hkv] == Hkv * kept and W <= kept <= Bud
        np.testing.assert_array_equal(idx[u, :off[u, Hkv]], want[u, :off[u, Hkv]])
        cand = int((gs[u, 0] >= np.float32(tau)).sum())
        assert kept - W == min(cand, Bud - W)
        for g in range(1, Hkv):
            np.testing.assert_array_equal(idx[u, off[u, g]:off[u, g + 1]], idx[u, :kept])
    if regime == "none":
        assert (bud == W).all()
    if regime == "many":
        assert (bud == Bud).all()
    check_gather(b["k"], b["v"], out["k_out"], out["v_out"], idx, off, prob)


def test_staged_calls_give_the_fused_result(B):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=2500, budget_per_head=96, n_needles=4, floor_per_head=0)
    b = gen.make_batch(cfg, "cuda")
    prob = problem_of(cfg, 2, shared_elastic=True)
    P = se_params(B, prob)
    fused = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    shape = B.make_shape(b["q"], b["k"])
    params = B.make_params(P, b["head_w"], b["sens"])
    ws = B.alloc_workspace(shape, params, "cuda")
    scores = torch.empty_like(fused["scores"])
    colmass = torch.empty(2, cfg.seq_len, device="cuda")
    B.ckv_score(shape, params, b["q"], b["k"], b["head_w"], scores, colmass, ws)
    B.ckv_unit_max(shape, params, scores)
    assert torch.equal(scores, fused["scores"])
    budgets, offsets = torch.zeros_like(fused["budgets"]), torch.zeros_like(fused["offsets"])
    bucket, entropy = torch.zeros_like(fused["bucket"]), torch.zeros_like(fused["entropy"])
    B.ckv_budget(shape, params, scores, colmass, b["sens"], budgets, offsets, bucket, entropy, ws)
    indices = torch.full_like(fused["indices"], -1)
    B.ckv_select(shape, params, scores, budgets, offsets, indices, ws)
    assert torch.equal(budgets, fused["budgets"]) and torch.equal(offsets, fused["offsets"])
    for u in range(2):
        rows = int(offsets[u, -1])
        assert torch.equal(indices[u, :rows], fused["indices"][u, :rows])
