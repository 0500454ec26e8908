"""GPU parity of the prompt-global window mass mode (Alg. 1 (A)) against the oracle, through the C ABI, alone
and combined with the value-norm ratio and the shared elastic selection (the paper's full online pass)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_08686_b200 import inputs as gen
from test_gpu_parity import SCORE_RTOL, check_gather, check_selection_against_oracle, params_of, problem_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_08686_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


def mode_params(B, prob):
    P = params_of(B, prob)
    for f in ("global_alpha", "units_per_prompt", "shared_elastic", "value_norm", "value_norm_eps"):
        setattr(P, f, getattr(prob, f))
    return P


@pytest.mark.parametrize("cfg_name,L,layers,upp,value_norm,shared", [
    ("c1", 2048, 4, 2, False, False), ("c2", 4096, 6, 3, False, False), ("c2", 3000, 4, 4, True, False),
    ("c2", 2500, 4, 2, True, True), ("c5", 4096, 4, 2, False, False)])
def test_global_alpha_whole_pass(B, cfg_name, L, layers, upp, value_norm, shared):
    cfg = gen.shrink(gen.CONFIGS[cfg_name], n_layers=layers, batch=1, seq_len=L, budget_per_head=128, n_needles=4,
                     floor_per_head=0 if shared else 1)
    b = gen.make_batch(cfg, "cpu")
    prob = problem_of(cfg, layers, global_alpha=True, units_per_prompt=upp, value_norm=value_norm,
                      shared_elastic=shared)
    qn, kn, vn, hw, sens = (gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w", "sens"))
    sc, cm = oracle.score(prob, qn, kn, hw, v=vn if value_norm else None)
    out = B.compress(*(b[x].cuda() for x in ("q", "k", "v", "head_w", "sens")), mode_params(B, prob), want_scores=True)
    assert B.ckv_device_status(out["ws"]) == B.OK
    gs = out["scores"].double().cpu().numpy()
    rel = np.abs(gs - sc) / np.maximum(np.abs(sc), 1e-20)
    assert rel.max() <= SCORE_RTOL, rel.max()
    ref = oracle.budget(prob, sc, cm, sens)
    assert np.abs(out["entropy"].double().cpu().numpy() - ref["entropy"]).max() <= 1e-4
    ent = out["entropy"].cpu().numpy().reshape(-1, upp)
    assert (ent == ent[:, :1]).all()                      # one risk coordinate per prompt
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    gpu_bucket = out["bucket"].cpu().numpy()
    for u in range(layers):
        prob_u = problem_of(cfg, 1, bucket_override=int(gpu_bucket[u]), shared_elastic=shared)
        mine = oracle.budget(prob_u, gs[u:u + 1], cm[u:u + 1], sens)
        assert (mine["budgets"][0] == bud[u]).all()
    want = oracle.select(prob, gs, bud, off)
    for u in range(layers):
        np.testing.assert_array_equal(idx[u, :off[u, -1]], want[u, :off[u, -1]])
    if not shared:
        ref["scores"], ref["idx"] = sc, oracle.select(prob, sc, ref["budgets"], ref["offsets"])
        check_selection_against_oracle(idx, bud, off, ref, prob)
    check_gather(b["k"], b["v"], out["k_out"], out["v_out"], idx, off, prob)


def test_staged_calls_with_the_exchange_step(B):
    """ckv_score -> ckv_prompt_mass -> (the ranks' sums added) -> ckv_global_scores: a prompt whose eight layers
    are split over two calls of four gives, with units_total = 8, what one call over all eight gives."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=8, batch=1, seq_len=2000, budget_per_head=96, n_needles=4)
    b = gen.make_batch(cfg, "cuda")
    prob = problem_of(cfg, 8, global_alpha=True, units_per_prompt=8)
    whole = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], mode_params(B, prob), want_scores=True)
    halves, pms = [], []
    prob_h = problem_of(cfg, 4, global_alpha=True, units_per_prompt=4)
    P = mode_params(B, prob_h)
    for r in range(2):
        sl = slice(4 * r, 4 * r + 4)
        q, k, hw = b["q"][sl].contiguous(), b["k"][sl].contiguous(), b["head_w"][sl].contiguous()
        shape = B.make_shape(q, k)
        params = B.make_params(P, hw, b["sens"])
        ws = B.alloc_workspace(shape, params, "cuda")
        scores = torch.empty(4, cfg.n_kv_heads, cfg.n, device="cuda")
        colmass = torch.empty(4, cfg.seq_len, device="cuda")
        B.ckv_score(shape, params, q, k, hw, scores, colmass, ws)
        pm = torch.empty(1, cfg.seq_len, device="cuda")
        B.ckv_prompt_mass(shape, params, colmass, pm)
        halves.append((shape, params, hw, scores, colmass))
        pms.append(pm)
    total = pms[0] + pms[1]                                  # what the all-reduce leaves on both ranks
    for r, (shape, params, hw, scores, colmass) in enumerate(halves):
        B.ckv_global_scores(shape, params, hw, total, 8, scores, colmass)
        ref = whole["scores"][4 * r: 4 * r + 4]
        assert torch.allclose(scores, ref, rtol=2e-6, atol=0), (scores - ref).abs().max()
