"""GPU parity of the value-norm ratio (Eq. 4's rho, Alg. 1 (B)) and of the whole pass with it switched on,
against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_08686_b200 import inputs as gen
from test_gpu_parity import (SCORE_RTOL, check_gather, check_selection_against_oracle, check_structure, params_of,
                             problem_of)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_08686_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def vn_params(B, prob):
    P = params_of(B, prob)
    P.value_norm, P.value_norm_eps = bool(prob.value_norm), float(prob.value_norm_eps)
    return P


@pytest.mark.parametrize("cfg_name,L", [("c1", 2048), ("c2", 4096), ("c2", 1111), ("c2", 255), ("c5", 4096)])
@pytest.mark.parametrize("eps", [0.0, 1e-6, 0.25])
def test_vnorm_matches_oracle(B, cfg_name, L, eps):
    """rho alone (fp32 and bf16 values, lengths with a ragged last block), then rho folded into given scores."""
    cfg = gen.shrink(gen.CONFIGS[cfg_name], n_layers=2, batch=1, seq_len=L, n_needles=2)
    b = gen.make_batch(cfg, "cpu")
    b["v"][:, :, 7] *= 30.0                       # a loud row and a silent one
    b["v"][:, :, 11] = 0
    prob = problem_of(cfg, 2, value_norm=True, value_norm_eps=eps)
    ref = oracle.vnorm(prob, gen.as_numpy(b["v"]))
    v = b["v"].cuda()
    shape = B.make_shape(b["q"].cuda(), b["k"].cuda())
    params = B.make_params(vn_params(B, prob), b["head_w"], b["sens"])
    ws = B.alloc_workspace(shape, params, "cuda")
    rho = torch.full((2, cfg.n_kv_heads, L), float("nan"), device="cuda")
    B.ckv_vnorm(shape, params, v, rho, None, ws)
    got = rho.double().cpu().numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-5, atol=0)
    assert (got[:, :, 11] == 0).all()
    scores = torch.rand(2, cfg.n_kv_heads, cfg.n, device="cuda") + 0.5
    want = scores * rho[:, :, :cfg.n]
    rho2 = torch.empty_like(rho)
    B.ckv_vnorm(shape, params, v, rho2, scores, ws)
    assert torch.equal(rho2, rho) and torch.equal(scores, want)


@pytest.mark.parametrize("cfg_name,L,score_path", [("c1", 2048, 0), ("c2", 4096, 2), ("c2", 3000, 1), ("c5", 4096, 0)])
def test_whole_pass_with_value_norm(B, cfg_name, L, score_path):
    """ckv_compress with value_norm on: scores within the score tolerance of the oracle's u = pool(alpha) * rho,
    budgets and indices exactly the oracle's steps on the GPU's own scores, gather bit-exact."""
    cfg = gen.shrink(gen.CONFIGS[cfg_name], n_layers=2, batch=1, seq_len=L, budget_per_head=128, n_needles=4)
    b = gen.make_batch(cfg, "cpu")
    g = torch.Generator().manual_seed(9)
    b["v"] = (b["v"].float() * (0.25 + 3.0 * torch.rand(2, cfg.n_kv_heads, L, 1, generator=g))).to(b["v"].dtype)
    prob = problem_of(cfg, 2, value_norm=True, value_norm_eps=1e-6)
    qn, kn, vn, hw, sens = (gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w", "sens"))
    sc, cm = oracle.score(prob, qn, kn, hw, v=vn)
    plain, _ = oracle.score(problem_of(cfg, 2), qn, kn, hw)
    assert np.abs(sc / plain - 1).max() > 0.5     # the ratio does change the scores
    prev = B.ckv_set_score_path(score_path)
    try:
        out = B.compress(*(b[x].cuda() for x in ("q", "k", "v", "head_w", "sens")), vn_params(B, prob), want_scores=True)
        assert B.ckv_device_status(out["ws"]) == B.OK
    finally:
        B.ckv_set_score_path(prev)
    gs = out["scores"].double().cpu().numpy()
    rel = np.abs(gs - sc) / np.maximum(np.abs(sc), 1e-20)
    assert rel.max() <= SCORE_RTOL, rel.max()
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    check_structure(idx, bud, off, prob)
    gpu_bucket = out["bucket"].cpu().numpy()
    for u in range(2):
        prob_u = problem_of(cfg, 1, bucket_override=int(gpu_bucket[u]))
        mine = oracle.budget(prob_u, gs[u:u + 1], cm[u:u + 1], sens)
        assert (mine["budgets"][0] == bud[u]).all()
    np.testing.assert_array_equal(idx, oracle.select(prob, gs, bud, off))
    ref = oracle.budget(prob, sc, cm, sens)
    ref["scores"], ref["idx"] = sc, oracle.select(prob, sc, ref["budgets"], ref["offsets"])
    check_selection_against_oracle(idx, bud, off, ref, prob)
    check_gather(b["k"], b["v"], out["k_out"], out["v_out"], idx, off, prob)
    # the oracle's whole pass agrees with its own steps (same code path as the CPU baseline)
    whole = oracle.compress(prob, qn, kn, vn, hw, sens)
    np.testing.assert_array_equal(whole["scores"], sc)


def test_value_norm_off_is_the_default_and_changes_nothing(B):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=2000, budget_per_head=64, n_needles=2)
    b = gen.make_batch(cfg, "cuda")
    prob = problem_of(cfg, 2)
    a = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], params_of(B, prob), want_scores=True)
    P = params_of(B, prob)
    P.value_norm, P.value_norm_eps = False, 0.5
    c = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    for key in ("scores", "indices", "budgets", "k_out", "v_out"):
        assert torch.equal(a[key], c[key])
