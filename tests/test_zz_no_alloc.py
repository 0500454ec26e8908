"""ckv_score_noalloc: the window-score entry point for callers that must not allocate device memory.

Some users of this library run inside a serving engine or training framework whose memory plan has
already handed out all of HBM by the time the retention pass runs: they cannot call cudaMalloc (or an
allocator that may fall back to it) for a work space.  For them the library carries a fixed scratch
array of its own and ``ckv_score_noalloc`` uses it.  This file checks, through the C ABI, that the
variant gives what ``ckv_score`` gives with a caller-owned work space, on two calls in a row (the
second on different inputs, so that anything the first call left in the shared scratch would show), and
that a problem too large for the fixed scratch is refused on the host.

The file name sorts last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import pytest
import torch

from paper_2602_08686_b200 import inputs as gen


def _score_both_ways(B, cfg):
    b = gen.make_batch(cfg, "cuda")
    P = B.Params(pool_kind=cfg.pool_kind, pool_size=cfg.pool_size, budget_per_head=cfg.budget_per_head,
                 floor_per_head=cfg.floor_per_head, n_buckets=cfg.n_buckets)
    shape = B.make_shape(b["q"], b["k"])
    params = B.make_params(P, b["head_w"], b["sens"])
    assert B.ckv_score_workspace_bytes(shape, params) <= B.NOALLOC_SCRATCH_BYTES
    Nu, Hkv, L, n = cfg.n_units, cfg.n_kv_heads, cfg.seq_len, cfg.n
    want_s = torch.full((Nu, Hkv, n), float("nan"), device="cuda")
    want_c = torch.full((Nu, L), float("nan"), device="cuda")
    ws = B.alloc_workspace(shape, params, "cuda")
    B.ckv_score(shape, params, b["q"], b["k"], b["head_w"], want_s, want_c, ws)
    assert B.ckv_device_status(ws) == B.OK
    got_s = torch.full_like(want_s, float("nan"))
    got_c = torch.full_like(want_c, float("nan"))
    B.ckv_score_noalloc(shape, params, b["q"], b["k"], b["head_w"], got_s, got_c)
    assert B.ckv_device_status(None) == B.OK          # the status word inside the fixed scratch
    assert torch.isfinite(got_s).all() and torch.isfinite(got_c).all()
    # the same kernels on the same inputs, and the scan is deterministic: the same bits, not just the same values
    assert torch.equal(got_s, want_s) and torch.equal(got_c, want_c)


@pytest.mark.gpu
def test_noalloc_score_matches_ckv_score_on_two_calls_in_a_row():
    from paper_2602_08686_b200 import binding as B
    B.lib()
    assert torch.cuda.is_available()
    # first call: tensor-core scan (bf16, W 32); second call: other shape, other inputs, and a ragged tail
    _score_both_ways(B, gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=4096, budget_per_head=128, n_needles=8))
    _score_both_ways(B, gen.shrink(gen.CONFIGS["c2"], config_id=7, n_layers=3, n_q_heads=8, n_kv_heads=2,
                                   seq_len=3001, budget_per_head=96, n_needles=4))
    # fp32 inputs take the plain kernels, which use other parts of the scratch
    _score_both_ways(B, gen.CONFIGS["c1"])


def test_noalloc_score_refuses_problems_beyond_its_fixed_scratch():
    """Host-side check (no GPU needed): the size test comes before any CUDA call."""
    import ctypes as C
    from paper_2602_08686_b200 import binding as B
    H, Hkv, W, d, L, Nu = 32, 8, 32, 128, 32768, 32
    shape = B.ckv_shape(Nu, H, Hkv, d, L, W, B.BF16, 0, H * W * d, W * d, d, Hkv * L * d, L * d, d)
    params = B.ckv_params(B.POOL_MAX, 7, 512, 1, 16, -1, H, 0)
    assert B.ckv_score_workspace_bytes(shape, params) > B.NOALLOC_SCRATCH_BYTES
    fake = C.c_void_p(1 << 20)   # never dereferenced: the call fails validation first
    rc = B.lib().ckv_score_noalloc(C.byref(shape), C.byref(params), fake, fake, fake, fake, fake, None)
    assert rc == B.ERR_WORKSPACE
