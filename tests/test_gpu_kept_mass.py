"""GPU parity of the Prop. 4.1 diagnostic (attention mass of the window rows that the selection keeps) against the
oracle's, on the GPU's own selection."""
import numpy as np
import pytest
import torch

import oracle
from paper_2602_08686_b200 import inputs as gen
from test_gpu_parity import params_of, problem_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_08686_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


@pytest.mark.parametrize("cfg_name,L,path,shared", [("c1", 2048, 0, False), ("c2", 4096, 2, False), ("c2", 3000, 1, False),
                                                    ("c5", 4096, 2, False), ("c5", 1500, 1, False), ("c2", 2500, 2, True),
                                                    ("c4", 8192, 0, False)])
def test_kept_mass_matches_oracle(B, cfg_name, L, path, shared):
    cfg = gen.shrink(gen.CONFIGS[cfg_name], n_layers=2, batch=1, seq_len=L, budget_per_head=128, n_needles=4,
                     floor_per_head=0 if shared else 1)
    b = gen.make_batch(cfg, "cpu")
    prob = problem_of(cfg, 2, shared_elastic=shared)
    P = params_of(B, prob)
    P.shared_elastic = shared
    dev = {x: b[x].cuda() for x in ("q", "k", "v", "head_w", "sens")}
    prev = B.ckv_set_score_path(path)
    try:
        out = B.compress(dev["q"], dev["k"], dev["v"], dev["head_w"], dev["sens"], P, want_scores=True)
    finally:
        B.ckv_set_score_path(prev)
    shape = B.make_shape(dev["q"], dev["k"])
    params = B.make_params(P, dev["head_w"], dev["sens"])
    kept = torch.full((2, cfg.n_q_heads, cfg.window), float("nan"), device="cuda")
    B.ckv_kept_mass(shape, params, dev["q"], out["k_out"], out["indices"], out["budgets"], out["offsets"], kept, out["ws"])
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    want = oracle.kept_mass(prob, gen.as_numpy(b["q"]), gen.as_numpy(b["k"]), idx, bud, off)
    got = kept.double().cpu().numpy()
    np.testing.assert_allclose(got, want, rtol=1e-3, atol=2e-6)
    assert (got > 0).all() and (got <= 1 + 1e-5).all()
    # Eq. 9's right-hand side from the GPU's masses bounds nothing here by itself; it must equal the oracle's
    m_gpu, m_ref = 1 - got, 1 - want
    eps_gpu, eps_ref = np.sqrt((m_gpu ** 2).mean(-1)), np.sqrt((m_ref ** 2).mean(-1))
    np.testing.assert_allclose(eps_gpu, eps_ref, rtol=1e-3, atol=1e-5)


def test_full_budget_keeps_all_mass(B):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=700, budget_per_head=700, n_needles=2)
    b = gen.make_batch(cfg, "cuda")
    P = params_of(B, problem_of(cfg, 2))
    out = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P)
    kept = torch.empty(2, cfg.n_q_heads, cfg.window, device="cuda")
    B.ckv_kept_mass(B.make_shape(b["q"], b["k"]), B.make_params(P, b["head_w"], b["sens"]), b["q"], out["k_out"],
                    out["indices"], out["budgets"], out["offsets"], kept, out["ws"])
    assert torch.allclose(kept, torch.ones_like(kept), rtol=0, atol=2e-5)
