"""Checks that stand in for a memory checker and a fault injector, without faulting anything:
  * an exhaustive sweep of short sequence lengths (every L from W to W + 300) over window sizes, GQA group sizes
    and pooling kinds, each a fused call against the oracle with every output and the work space between canary
    bands -- the ragged tails, short row blocks and halo cases of the hand-addressed kernels;
  * the device-side status word: a code planted from the host is reported once and cleared, and a wait limit of a
    few microseconds makes an ordinary wait of the scan run out, which must come back as CKV_ERR_TIMEOUT with the
    GPU and the work space usable for the next call.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import Problem
from paper_2602_08686_b200 import inputs as gen
from test_gpu_parity import SCORE_RTOL, Guarded, compress_guarded

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2602_08686_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


@pytest.mark.parametrize("pool_kind,pool_size", [(gen.POOL_NONE, 1), (gen.POOL_MAX, 7), (gen.POOL_AVG, 5)])
@pytest.mark.parametrize("G", [1, 4, 7, 8])
@pytest.mark.parametrize("W", [16, 32, 64])
def test_every_short_length(B, W, G, pool_kind, pool_size):
    Hkv, d, Nu = 2, 128, 2
    H = G * Hkv
    g = torch.Generator().manual_seed(1000 * W + 10 * G + pool_kind)
    sens = (0.8 + 0.4 * torch.rand(16, generator=g)).float()
    worst = 0.0
    for L in range(W, W + 301):
        n = L - W
        q = torch.randn(Nu, H, W, d, generator=g).bfloat16()
        k = torch.randn(Nu, Hkv, L, d, generator=g).bfloat16()
        v = torch.randn(Nu, Hkv, L, d, generator=g).bfloat16()
        head_w = (0.5 + torch.rand(Nu, H, generator=g)).float()
        budget = L if n == 0 else W + max(1, n // 3)       # no prefix: everything is kept
        prob = Problem(Nu, H, Hkv, L, W, head_dim=d, dtype=oracle.BF16, pool_kind=pool_kind, pool_size=pool_size,
                       budget_per_head=budget, floor_per_head=min(1, budget - W) if n else 0, n_buckets=16)
        P = B.Params(pool_kind=pool_kind, pool_size=pool_size, budget_per_head=budget,
                     floor_per_head=prob.floor_per_head, n_buckets=16)
        b = dict(q=q.cuda(), k=k.cuda(), v=v.cuda(), head_w=head_w.cuda(), sens=sens.cuda())
        out = compress_guarded(B, b, P, Guarded())
        assert B.ckv_device_status(out["ws"]) == B.OK
        sc, cm = oracle.score(prob, gen.as_numpy(q), gen.as_numpy(k), head_w.numpy())
        gs = out["scores"].double().cpu().numpy()
        if n:
            rel = np.abs(gs - sc) / np.maximum(np.abs(sc), 1e-20)
            assert rel.max() <= SCORE_RTOL, (L, rel.max())
            worst = max(worst, rel.max())
        bud, off, idx = (out[x].cpu().numpy() for x in ("budgets", "offsets", "indices"))
        bucket = out["bucket"].cpu().numpy()
        for u in range(Nu):      # the oracle's budget step on the GPU's scores and entropy bin: exact
            prob_u = Problem(1, H, Hkv, L, W, head_dim=d, dtype=oracle.BF16, pool_kind=pool_kind, pool_size=pool_size,
                             budget_per_head=budget, floor_per_head=prob.floor_per_head, n_buckets=16,
                             bucket_override=int(bucket[u]))
            mine = oracle.budget(prob_u, gs[u:u + 1], cm[u:u + 1], sens.numpy())
            assert (mine["budgets"][0] == bud[u]).all(), (L, u)
        np.testing.assert_array_equal(idx, oracle.select(prob, gs, bud, off), err_msg=f"L={L}")
        ko, vo = oracle.gather(prob, gen.as_numpy(k), gen.as_numpy(v), idx, bud, off)
        np.testing.assert_array_equal(gen.as_numpy(out["k_out"]), ko)
        np.testing.assert_array_equal(gen.as_numpy(out["v_out"]), vo)
    assert worst <= SCORE_RTOL


def small_problem(B, L=6000, layers=3):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=layers, seq_len=L, budget_per_head=128, n_needles=4)
    b = gen.make_batch(cfg, "cuda")
    P = B.Params(pool_kind=cfg.pool_kind, pool_size=cfg.pool_size, budget_per_head=cfg.budget_per_head)
    return cfg, b, P


def test_status_word_planted_from_the_host_is_reported_once(B):
    """No kernel involved in the failure: after an ordinary call the test itself writes a code into the work
    space's status word; ckv_device_status reports CKV_ERR_TIMEOUT, clears it, and later calls do not bring it back."""
    cfg, b, P = small_problem(B)
    out = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    ws = out["ws"]
    assert B.ckv_device_status(ws) == B.OK
    ws[:4].view(torch.int32)[0] = 31
    torch.cuda.synchronize()
    again = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True, ws=ws)
    assert torch.equal(again["indices"], out["indices"])
    assert B.ckv_device_status(ws) == B.ERR_TIMEOUT       # recorded before that call, still there after it
    assert B.ckv_device_status(ws) == B.OK                # reported once
    # work space that no call has used reads OK whatever it holds
    fresh = torch.full((B.ckv_workspace_bytes(B.make_shape(b["q"], b["k"]), B.make_params(P, b["head_w"], b["sens"])),),
                       0x5A, dtype=torch.uint8, device="cuda")
    assert B.ckv_device_status(fresh) == B.OK


def test_a_wait_that_runs_out_is_reported_and_the_next_call_is_correct(B):
    """The wait limit is set to two microseconds, less than a key tile takes to arrive: some wait of the scan runs
    out, the kernel winds down (every wait of it is bounded by the same limit), the call returns and the status
    word says CKV_ERR_TIMEOUT.  With the limit restored the same work space gives the right answer again."""
    cfg, b, P = small_problem(B)
    good = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    ws = good["ws"]
    assert B.ckv_device_status(ws) == B.OK
    prev_path = B.ckv_set_score_path(2)                   # the tensor-core scan, whose waits these are
    prev = B.ckv_set_tunable("wait_limit_us", 2)
    try:
        bad = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True, ws=ws)
        torch.cuda.synchronize()                          # the call came back: nothing hangs
        assert B.ckv_device_status(ws) == B.ERR_TIMEOUT
        del bad
    finally:
        B.ckv_set_tunable("wait_limit_us", prev)
        B.ckv_set_score_path(prev_path)
    assert prev == 2000000
    again = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True, ws=ws)
    assert B.ckv_device_status(ws) == B.OK
    for key in ("scores", "indices", "budgets", "k_out", "v_out"):
        assert torch.equal(again[key], good[key]), key
