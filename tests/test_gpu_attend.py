"""GPU parity of the decode-side check (attention of decode queries over the full and over the compressed cache)
against the oracle, and the identities of Prop. 4.1 on the GPU's numbers."""
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


@pytest.mark.parametrize("cfg_name,L,n_dec", [("c1", 2048, 4), ("c2", 4096, 8), ("c2", 1111, 1), ("c5", 4096, 4),
                                              ("c4", 8192, 5)])
def test_attend_full_and_compressed(B, cfg_name, L, n_dec):
    cfg = gen.shrink(gen.CONFIGS[cfg_name], n_layers=2, batch=1, seq_len=L, budget_per_head=128, n_needles=4)
    b = gen.make_batch(cfg, "cpu")
    g = torch.Generator().manual_seed(L + n_dec)
    qd = torch.randn(2, cfg.n_q_heads, n_dec, 128, generator=g)
    qd[:, :, 0] = b["q"][:, :, -1].float() * 0.5 + 0.5 * qd[:, :, 0]      # one query close to the last prompt token
    qd = qd.to(b["q"].dtype)
    prob = problem_of(cfg, 2)
    P = params_of(B, prob)
    dev = {x: b[x].cuda() for x in ("q", "k", "v", "head_w", "sens")}
    out = B.compress(dev["q"], dev["k"], dev["v"], dev["head_w"], dev["sens"], P)
    shape = B.make_shape(dev["q"], dev["k"])
    params = B.make_params(P, dev["head_w"], dev["sens"])
    ws = out["ws"]
    o_full = torch.full((2, cfg.n_q_heads, n_dec, 128), float("nan"), device="cuda")
    o_comp = torch.full_like(o_full, float("nan"))
    lse_full = torch.full((2, cfg.n_q_heads, n_dec), float("nan"), device="cuda")
    lse_comp = torch.full_like(lse_full, float("nan"))
    B.ckv_attend(shape, params, qd.cuda(), dev["k"], dev["v"], o_full, lse_full, ws)
    B.ckv_attend(shape, params, qd.cuda(), out["k_out"], out["v_out"], o_comp, lse_comp, ws,
                 budgets=out["budgets"], offsets=out["offsets"])
    qn, kn, vn = gen.as_numpy(qd), gen.as_numpy(b["k"]), gen.as_numpy(b["v"])
    ref_o, ref_lse = oracle.attend(prob, qn, kn, vn)
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    ko, vo = gen.as_numpy(out["k_out"]), gen.as_numpy(out["v_out"])
    ref_oc, ref_lsec = oracle.attend(prob, qn, ko, vo, bud, off)
    for got, want in ((o_full, ref_o), (o_comp, ref_oc)):
        got = got.double().cpu().numpy()
        scale = np.abs(want).max(-1, keepdims=True)
        assert (np.abs(got - want) <= 1e-3 * scale + 1e-6).all(), np.abs(got - want).max()
    np.testing.assert_allclose(lse_full.double().cpu().numpy(), ref_lse, rtol=0, atol=2e-4)
    np.testing.assert_allclose(lse_comp.double().cpu().numpy(), ref_lsec, rtol=0, atol=2e-4)
    kept = torch.exp(lse_comp - lse_full).double().cpu().numpy()
    np.testing.assert_allclose(kept, np.exp(ref_lsec - ref_lse), rtol=1e-3, atol=1e-6)
    assert (kept > 0).all() and (kept <= 1 + 1e-4).all()


def test_attend_over_a_full_budget_cache_equals_full_attention(B):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=900, budget_per_head=900, n_needles=2)
    b = gen.make_batch(cfg, "cuda")
    P = params_of(B, problem_of(cfg, 2))
    out = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P)
    shape, params = B.make_shape(b["q"], b["k"]), B.make_params(P, b["head_w"], b["sens"])
    qd = torch.randn(2, cfg.n_q_heads, 8, 128, device="cuda").to(b["q"].dtype)
    o1, o2 = torch.empty(2, cfg.n_q_heads, 8, 128, device="cuda"), torch.empty(2, cfg.n_q_heads, 8, 128, device="cuda")
    l1, l2 = torch.empty(2, cfg.n_q_heads, 8, device="cuda"), torch.empty(2, cfg.n_q_heads, 8, device="cuda")
    B.ckv_attend(shape, params, qd, b["k"], b["v"], o1, l1, out["ws"])
    B.ckv_attend(shape, params, qd, out["k_out"], out["v_out"], o2, l2, out["ws"], budgets=out["budgets"],
                 offsets=out["offsets"])
    assert torch.equal(o1, o2) and torch.equal(l1, l2)      # same rows in the same order, same slices
