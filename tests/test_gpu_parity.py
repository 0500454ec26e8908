"""GPU parity: the CUDA library (through its C ABI) against the fp64 oracle on the same seeded inputs.

Protocol (discrete stages never inherit float noise):
  1. scores: max relative error <= 1e-3 over every prefix position; entropy abs error <= 1e-4.
  2. bucket: equal unless n_buckets * entropy / ln L is within 1e-4 of an integer.
  3. ckv_budget fed the oracle's scores rounded to fp32 (both sides see identical bits): budgets and
     offsets exactly equal.  In the fused path the GPU budgets equal the oracle's budget step run on
     the GPU's own scores, exactly.
  4. ckv_select on identical fp32 scores and budgets: identical indices.  Against the oracle's own
     fp64 scores the symmetric difference lies inside the near-tie band (1e-3 relative of the k-th score).
  5. gather: bit-exact given the indices.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import Problem
from paper_2602_08686_b200 import inputs as gen

pytestmark = pytest.mark.gpu

SCORE_RTOL = 1e-3          # tolerance on pooled, weighted scores (max relative error)
TIE_BAND = 1e-3            # selection may differ only inside this relative band around the k-th score


@pytest.fixture(scope="module")
def B():
    from paper_2602_08686_b200 import binding
    binding.lib()
    assert torch.cuda.is_available()
    return binding


@pytest.fixture(params=["auto", "plain"])
def score_path(request, B):
    """Runs a case once with the automatic choice (tensor-core scan where it applies) and once with the
    plain kernels forced."""
    prev = B.ckv_set_score_path(1 if request.param == "plain" else 0)
    yield request.param
    B.ckv_set_score_path(prev)


class Guarded:
    """Device tensors with 256 bytes of a canary pattern on either side (in place of a memory checker): a kernel
    that writes before or past one of its outputs, or outside its work space, changes a canary byte."""
    CANARY = 0xA5

    def __init__(self):
        self.items = []

    def new(self, shape, dtype, fill=None, device="cuda"):
        shape = tuple(int(x) for x in shape)
        nbytes = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        raw = torch.full((256 + (nbytes + 255) // 256 * 256 + 256,), self.CANARY, dtype=torch.uint8, device=device)
        body = raw[256:256 + nbytes].view(dtype).view(shape)
        if fill is not None:
            body.fill_(fill)
        self.items.append((raw, nbytes))
        return body

    def check(self):
        torch.cuda.synchronize()
        for raw, nbytes in self.items:
            assert bool((raw[:256] == self.CANARY).all()), "write before a buffer"
            assert bool((raw[256 + nbytes:] == self.CANARY).all()), "write past a buffer"


def compress_guarded(B, b, P, guard, ws=None, gate_coords=None):
    """The fused call with every output and the work space between canary bands; the dict of binding.compress."""
    shape = B.make_shape(b["q"], b["k"])
    params = B.make_params(P, b["head_w"], b["sens"], gate_coords=gate_coords)
    Nu, Hkv, L, W = shape.n_units, shape.n_kv_heads, shape.seq_len, shape.window
    rows = B.rows_per_unit(shape, params)
    if ws is None:
        ws = guard.new((B.ckv_workspace_bytes(shape, params),), torch.uint8)
    out = dict(k_out=guard.new((Nu, rows, shape.head_dim), b["k"].dtype, 0), v_out=guard.new((Nu, rows, shape.head_dim), b["v"].dtype, 0),
               indices=guard.new((Nu, rows), torch.int32, -1), budgets=guard.new((Nu, Hkv), torch.int32, 0),
               offsets=guard.new((Nu, Hkv + 1), torch.int32, 0), bucket=guard.new((Nu,), torch.int32, 0),
               entropy=guard.new((Nu,), torch.float32, float("nan")),
               scores=guard.new((Nu, Hkv, L - W), torch.float32, float("nan")), ws=ws)
    B.ckv_compress(shape, params, b["q"], b["k"], b["v"], b["head_w"], b["sens"], out["k_out"], out["v_out"],
                   out["indices"], out["budgets"], out["offsets"], ws, scores=out["scores"], bucket=out["bucket"],
                   entropy=out["entropy"])
    guard.check()
    return out


def problem_of(cfg, Nu, **kw):
    prob = Problem(Nu, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq_len, cfg.window, head_dim=cfg.head_dim,
                   dtype=oracle.BF16 if cfg.dtype == "bf16" else oracle.F32, pool_kind=cfg.pool_kind,
                   pool_size=cfg.pool_size, budget_per_head=cfg.budget_per_head, floor_per_head=cfg.floor_per_head,
                   n_buckets=cfg.n_buckets)
    for k, v in kw.items():
        setattr(prob, k, v)
    return prob


def params_of(B, prob):
    return B.Params(pool_kind=prob.pool_kind, pool_size=prob.pool_size, budget_per_head=prob.budget_per_head,
                    floor_per_head=prob.floor_per_head, n_buckets=prob.n_buckets,
                    bucket_override=prob.bucket_override)


def oracle_all(prob, b):
    q, k, v, hw, sens = (gen.as_numpy(b[x]) for x in ("q", "k", "v", "head_w", "sens"))
    scores, colmass = oracle.score(prob, q, k, hw)
    bud = oracle.budget(prob, scores, colmass, sens)
    idx = oracle.select(prob, scores, bud["budgets"], bud["offsets"])
    return dict(scores=scores, colmass=colmass, idx=idx, **bud)


def check_scores(gpu_scores, gpu_colmass, gpu_entropy, ref, prob):
    s = gpu_scores.double().cpu().numpy()
    rel = np.abs(s - ref["scores"]) / np.maximum(np.abs(ref["scores"]), 1e-20)
    assert rel.max() <= SCORE_RTOL, f"score rel err {rel.max():.3e}"
    cm = gpu_colmass.double().cpu().numpy()
    np.testing.assert_allclose(cm, ref["colmass"], rtol=SCORE_RTOL, atol=1e-12)
    assert np.abs(gpu_entropy.double().cpu().numpy() - ref["entropy"]).max() <= 1e-4
    return rel.max()


def check_bucket(gpu_bucket, ref, prob):
    hn = ref["entropy"] / math.log(prob.seq_len) * prob.n_buckets
    near = np.abs(hn - np.round(hn)) < 1e-4
    got = gpu_bucket.cpu().numpy()
    assert ((got == ref["bucket"]) | near).all()


def check_selection_against_oracle(gpu_idx, gpu_budgets, gpu_offsets, ref, prob):
    """Same budgets: the index sets may differ only inside the near-tie band of the oracle's scores."""
    W, n = prob.window, prob.n
    for u in range(prob.n_units):
        if not (gpu_budgets[u] == ref["budgets"][u]).all():
            continue  # different budgets (a score within the band of tau): compared elsewhere
        for g in range(prob.n_kv_heads):
            a = set(gpu_idx[u, gpu_offsets[u, g]: gpu_offsets[u, g + 1]].tolist())
            r = set(ref["idx"][u, ref["offsets"][u, g]: ref["offsets"][u, g + 1]].tolist())
            diff = a ^ r
            if not diff:
                continue
            e = ref["budgets"][u, g] - W
            sc = ref["scores"][u, g]
            kth = np.sort(sc)[::-1][e - 1]
            for t in diff:
                assert t < n and abs(sc[t] - kth) <= TIE_BAND * abs(kth), (u, g, t, sc[t], kth)


def check_structure(idx, budgets, offsets, prob, needles=None, cfg=None):
    L, W, n, Hkv = prob.seq_len, prob.window, prob.n, prob.n_kv_heads
    rows = Hkv * prob.rows_per_head
    assert (budgets.sum(1) == rows).all()
    assert (offsets[:, 0] == 0).all() and (np.diff(offsets, axis=1) == budgets).all()
    for u in range(prob.n_units):
        for g in range(Hkv):
            s = idx[u, offsets[u, g]: offsets[u, g + 1]]
            assert (np.diff(s) > 0).all() and s[0] >= 0 and s[-1] == L - 1
            assert (s[-W:] == np.arange(n, L)).all()
            if prob.budget_per_head < L:
                assert budgets[u, g] - W >= prob.floor_per_head


def check_gather(k, v, k_out, v_out, idx, offsets, prob):
    kn, vn = gen.as_numpy(k), gen.as_numpy(v)
    ko, vo = gen.as_numpy(k_out), gen.as_numpy(v_out)
    for u in range(prob.n_units):
        for g in range(prob.n_kv_heads):
            sl = slice(offsets[u, g], offsets[u, g + 1])
            np.testing.assert_array_equal(ko[u, sl], kn[u, g, idx[u, sl]])
            np.testing.assert_array_equal(vo[u, sl], vn[u, g, idx[u, sl]])


def run_case(B, cfg, units=None, **prob_kw):
    """Staged and fused GPU runs of one case against the oracle; returns the worst score error."""
    b_cpu = gen.make_batch(cfg, "cpu", units)
    Nu = len(b_cpu["units"])
    prob = problem_of(cfg, Nu, **prob_kw)
    ref = oracle_all(prob, b_cpu)
    b = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in b_cpu.items()}
    P = params_of(B, prob)
    shape = B.make_shape(b["q"], b["k"])
    params = B.make_params(P, b["head_w"], b["sens"])
    guard = Guarded()   # every output and the work space sit between canary bands
    ws = guard.new((B.ckv_workspace_bytes(shape, params),), torch.uint8)
    n, Hkv, L = prob.n, prob.n_kv_heads, prob.seq_len
    rows = B.rows_per_unit(shape, params)
    dev = "cuda"

    # ---- staged path -------------------------------------------------------------------------
    scores = guard.new((Nu, Hkv, n), torch.float32, float("nan"))
    colmass = guard.new((Nu, L), torch.float32, float("nan"))
    B.ckv_score(shape, params, b["q"], b["k"], b["head_w"], scores, colmass, ws)
    budgets = guard.new((Nu, Hkv), torch.int32, 0)
    offsets = guard.new((Nu, Hkv + 1), torch.int32, 0)
    bucket = guard.new((Nu,), torch.int32, 0)
    entropy = guard.new((Nu,), torch.float32, 0)
    B.ckv_budget(shape, params, scores, colmass, b["sens"], budgets, offsets, bucket, entropy, ws)
    guard.check()
    err = check_scores(scores, colmass, entropy, ref, prob)
    check_bucket(bucket, ref, prob)

    # (3) budget on identical bits: the oracle's scores rounded to fp32, the oracle's bucket forced
    s32 = torch.from_numpy(ref["scores"]).float()
    cm32 = torch.from_numpy(ref["colmass"]).float()
    for u_bucket in sorted(set(ref["bucket"].tolist())):
        sel = [u for u in range(Nu) if ref["bucket"][u] == u_bucket]
        prob_b = problem_of(cfg, Nu, **{**prob_kw, "bucket_override": int(u_bucket)})
        ref_b = oracle.budget(prob_b, s32.double().numpy(), cm32.double().numpy(), gen.as_numpy(b_cpu["sens"]))
        params_b = B.make_params(params_of(B, prob_b), b["head_w"], b["sens"])
        bud_g = torch.zeros_like(budgets)
        off_g = torch.zeros_like(offsets)
        B.ckv_budget(shape, params_b, s32.cuda(), cm32.cuda(), b["sens"], bud_g, off_g, bucket.clone(),
                     entropy.clone(), ws)
        assert (bud_g.cpu().numpy()[sel] == ref_b["budgets"][sel]).all()
        assert (off_g.cpu().numpy()[sel] == ref_b["offsets"][sel]).all()

    # (4) select on identical bits
    ref_bud = torch.from_numpy(ref["budgets"]).cuda()
    ref_off = torch.from_numpy(ref["offsets"]).cuda()
    idx_g = guard.new((Nu, rows), torch.int32, -1)
    B.ckv_select(shape, params, s32.cuda(), ref_bud, ref_off, idx_g, ws)
    want = oracle.select(prob, s32.double().numpy(), ref["budgets"], ref["offsets"])
    np.testing.assert_array_equal(idx_g.cpu().numpy(), want)
    # the GPU's own scores with the oracle's budgets: near-tie protocol
    B.ckv_select(shape, params, scores, ref_bud, ref_off, idx_g, ws)
    check_selection_against_oracle(idx_g.cpu().numpy(), ref["budgets"], ref["offsets"], ref, prob)

    # (5) gather
    k_out = guard.new((Nu, rows, prob.head_dim), b["k"].dtype, 0)
    v_out = guard.new((Nu, rows, prob.head_dim), b["k"].dtype, 0)
    B.ckv_gather(shape, params, b["k"], b["v"], idx_g, ref_off, k_out, v_out)
    guard.check()
    check_gather(b_cpu["k"], b_cpu["v"], k_out, v_out, idx_g.cpu().numpy(), ref["offsets"], prob)

    # ---- fused path --------------------------------------------------------------------------
    out = compress_guarded(B, b, P, guard, ws=ws)
    assert B.ckv_device_status(ws) == B.OK
    assert torch.equal(out["scores"], scores)                       # deterministic, same kernels
    gs = out["scores"].double().cpu().numpy()
    # the oracle's budget step on the GPU's own scores, with the GPU's bucket: exact equality
    gpu_budgets, gpu_offsets = out["budgets"].cpu().numpy(), out["offsets"].cpu().numpy()
    gpu_bucket = out["bucket"].cpu().numpy()
    for u in range(Nu):
        prob_u = problem_of(cfg, 1, **{**prob_kw, "bucket_override": int(gpu_bucket[u])})
        ref_u = oracle.budget(prob_u, gs[u:u + 1], colmass[u:u + 1].double().cpu().numpy(),
                              gen.as_numpy(b_cpu["sens"]))
        assert (ref_u["budgets"][0] == gpu_budgets[u]).all(), (u, ref_u["budgets"], gpu_budgets[u])
    gpu_idx = out["indices"].cpu().numpy()
    np.testing.assert_array_equal(gpu_idx, oracle.select(prob, gs, gpu_budgets, gpu_offsets))
    check_structure(gpu_idx, gpu_budgets, gpu_offsets, prob)
    check_selection_against_oracle(gpu_idx, gpu_budgets, gpu_offsets, ref, prob)
    check_gather(b_cpu["k"], b_cpu["v"], out["k_out"], out["v_out"], gpu_idx, gpu_offsets, prob)
    return err


# ------------------------------------------------------------------------------------------ cases
def test_config1_fp32_whole(B):
    """Config 1 as specified: one layer, 8/2 heads, fp32, L 2048, W 32, MAX pool 7, B 512."""
    run_case(B, gen.CONFIGS["c1"])


@pytest.mark.parametrize("L", [4096, 4000, 1111, 128, 129])
def test_llama_shape_small(B, L, score_path):
    """Config 2's head layout at lengths that span several key tiles and leave a ragged tail."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=L, budget_per_head=min(128, L // 2),
                     n_needles=8 if L > 1000 else 2)
    run_case(B, cfg)


def test_tensor_core_path_is_taken_and_agrees_with_plain(B):
    """bf16, W 32, L >= 128 must run the tcgen05 kernel (path 2 = required) and match the plain kernels."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=3, seq_len=5000, budget_per_head=128, n_needles=8)
    b = gen.make_batch(cfg, "cuda")
    P = params_of(B, problem_of(cfg, 3))
    prev = B.ckv_set_score_path(2)
    try:
        tc = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
        assert B.ckv_device_status(tc["ws"]) == B.OK
        B.ckv_set_score_path(1)
        pl = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    finally:
        B.ckv_set_score_path(prev)
    rel = ((tc["scores"] - pl["scores"]).abs() / pl["scores"].abs().clamp_min(1e-20)).max().item()
    assert rel < 1e-4, rel


@pytest.mark.parametrize("n_buckets,dup", [(1, False), (5, True), (16, False), (32, True), (40, False)])
def test_fused_budget_equals_staged_budget(B, n_buckets, dup):
    """The fused call's budget stage (entropy partials left by the pooling kernel) against ckv_budget on the
    same scores and column mass (partials from its own kernel): same buckets, budgets and offsets for tables
    of several sizes, with repeated thresholds and with scores equal to a threshold."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=3, n_q_heads=8, n_kv_heads=4, seq_len=2500, budget_per_head=96,
                     n_needles=8, n_buckets=n_buckets)
    b = gen.make_batch(cfg, "cuda")
    sens = b["sens"].clone()
    prob = problem_of(cfg, 3)
    P = params_of(B, prob)
    first = B.compress(b["q"], b["k"], b["v"], b["head_w"], sens, P, want_scores=True)
    # thresholds taken from the scores themselves: candidates exist, and some scores equal the threshold
    flat = first["scores"].flatten().sort(descending=True).values
    picks = flat[torch.linspace(20, 2000, n_buckets).long()]
    sens = picks[torch.randperm(n_buckets, generator=torch.Generator().manual_seed(3))].contiguous()
    if dup and n_buckets > 2:
        sens[1] = sens[0]
        sens[-1] = sens[2]
    for override in (-1, 0, n_buckets - 1):
        prob_o = problem_of(cfg, 3, bucket_override=override)
        P = params_of(B, prob_o)
        out = B.compress(b["q"], b["k"], b["v"], b["head_w"], sens, P, want_scores=True)
        shape = B.make_shape(b["q"], b["k"])
        params = B.make_params(P, b["head_w"], sens)
        ws = B.alloc_workspace(shape, params, "cuda")
        scores = torch.empty_like(out["scores"])
        colmass = torch.empty(3, cfg.seq_len, device="cuda")
        B.ckv_score(shape, params, b["q"], b["k"], b["head_w"], scores, colmass, ws)
        assert torch.equal(scores, out["scores"])
        budgets, offsets = torch.zeros_like(out["budgets"]), torch.zeros_like(out["offsets"])
        bucket, entropy = torch.zeros_like(out["bucket"]), torch.zeros_like(out["entropy"])
        B.ckv_budget(shape, params, scores, colmass, sens, budgets, offsets, bucket, entropy, ws)
        for key, val in (("bucket", bucket), ("budgets", budgets), ("offsets", offsets), ("entropy", entropy)):
            assert torch.equal(out[key], val), (override, key, out[key], val)
        assert len(set(out["budgets"].flatten().tolist())) > 1   # the thresholds do bite


@pytest.mark.parametrize("jump", [60.0, 140.0, 400.0])
def test_logits_far_above_the_running_reference(B, jump):
    """Keys whose logits exceed everything before them by `jump` powers of two: the scan's running sums are
    kept relative to an early reference and must re-base when they leave the fp32 range (jump > 127)."""
    Nu, H, Hkv, L, W = 2, 8, 2, 3000, 32
    g = torch.Generator().manual_seed(int(jump))
    u_dir = torch.zeros(128)
    u_dir[:4] = 0.5                                  # unit vector
    q = 0.3 * torch.randn(Nu, H, W, 128, generator=g) + 8.0 * u_dir
    k = 0.3 * torch.randn(Nu, Hkv, L, 128, generator=g)
    k -= (k @ u_dir)[..., None] * u_dir              # ordinary keys: no component along the queries' direction
    amp = jump * math.sqrt(128.0) / (8.0 * math.log2(math.e))   # logit of a planted key ~ jump (base 2)
    for t, f in ((700, 0.5), (1500, 1.0), (2600, 1.0), (2601, 0.98)):
        k[:, :, t] += f * amp * u_dir
    v = torch.randn(Nu, Hkv, L, 128, generator=g)
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=Nu, n_q_heads=H, n_kv_heads=Hkv, seq_len=L, window=W,
                     budget_per_head=128, n_needles=0)
    b = dict(q=q.bfloat16(), k=k.bfloat16(), v=v.bfloat16(), head_w=0.5 + torch.rand(Nu, H, generator=g),
             sens=gen.make_sens(cfg))
    prob = problem_of(cfg, Nu)
    ref = oracle.score(prob, *(gen.as_numpy(b[x]) for x in ("q", "k", "head_w")))
    for path in (2, 1):
        prev = B.ckv_set_score_path(path)
        try:
            out = B.compress(b["q"].cuda(), b["k"].cuda(), b["v"].cuda(), b["head_w"].cuda(), b["sens"].cuda(),
                             params_of(B, prob), want_scores=True)
            assert B.ckv_device_status(out["ws"]) == B.OK
        finally:
            B.ckv_set_score_path(prev)
        s = out["scores"].double().cpu().numpy()
        assert np.isfinite(s).all()
        big = ref[0] > 1e-30                          # below that both sides are zero to fp32
        rel = np.abs(s - ref[0])[big] / ref[0][big]
        assert rel.max() <= SCORE_RTOL, (path, rel.max())
        assert np.abs(s[~big]).max(initial=0.0) <= 1e-30


@pytest.mark.parametrize("G,W,pool_kind,pool_size", [(4, 32, 1, 7), (2, 64, 1, 3), (8, 16, 1, 5), (3, 16, 0, 1),
                                                     (4, 16, 1, 15)])
def test_grouped_scan_output_matches_per_head_output(B, G, W, pool_kind, pool_size):
    """The scan's per-group maximum and mass (group_fuse) against its per-head column sums: the same scores
    bit for bit (head_w >= 0), the same budgets and indices."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, n_q_heads=2 * G, n_kv_heads=2, seq_len=3000, window=W,
                     pool_kind=pool_kind, pool_size=pool_size, budget_per_head=128, n_needles=8)
    b = gen.make_batch(cfg, "cuda")
    P = params_of(B, problem_of(cfg, 2))
    prev_path = B.ckv_set_score_path(2)
    prev = B.ckv_set_tunable("group_fuse", 1)
    try:
        fused = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
        assert B.ckv_device_status(fused["ws"]) == B.OK
        B.ckv_set_tunable("group_fuse", 0)
        plain = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
        assert B.ckv_device_status(plain["ws"]) == B.OK
    finally:
        B.ckv_set_tunable("group_fuse", prev)
        B.ckv_set_score_path(prev_path)
    assert torch.equal(fused["scores"], plain["scores"])
    for key in ("budgets", "offsets", "indices"):
        assert torch.equal(fused[key], plain[key]), key


@pytest.mark.parametrize("G,W", [(1, 32), (2, 64), (3, 16), (9, 16), (5, 32)])
def test_group_sizes_and_windows(B, G, W):
    """Row blocks: G*W below, equal to and above 128 rows (several blocks, the last one partial)."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, n_q_heads=2 * G, n_kv_heads=2, seq_len=1500, window=W,
                     budget_per_head=100, n_needles=4)
    run_case(B, cfg)


def test_heavy_tail_keys(B, score_path):
    """Config 4's structure (Student-t key scales, stratified needles) at a length the oracle finishes."""
    cfg = gen.shrink(gen.CONFIGS["c4"], n_layers=2, seq_len=8192, budget_per_head=128, n_needles=16)
    run_case(B, cfg)


@pytest.mark.parametrize("budget", [128, 512])
def test_qwen_shape_L4096(B, budget, score_path):
    """Config 5 at L 4096: GQA 7, W 64, AVG pool 5, floor 8, one low-reliability group per layer."""
    cfg = gen.shrink(gen.c5_point(4096, budget), n_layers=2, batch=2)
    run_case(B, cfg)


@pytest.mark.parametrize("override", [0, 7, 15])
def test_bucket_override(B, override):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=1, n_q_heads=8, n_kv_heads=2, seq_len=1500, budget_per_head=96,
                     n_needles=4)
    run_case(B, cfg, bucket_override=override)


@pytest.mark.parametrize("pool_kind,pool_size", [(0, 1), (1, 1), (1, 3), (1, 15), (2, 3), (2, 7), (2, 15)])
def test_pooling_variants(B, pool_kind, pool_size):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=1, n_q_heads=8, n_kv_heads=2, seq_len=1000, budget_per_head=80,
                     n_needles=4, pool_kind=pool_kind, pool_size=pool_size)
    run_case(B, cfg)


@pytest.mark.parametrize("W,L,Bud", [(1, 300, 10), (8, 8, 8), (16, 40, 16), (32, 600, 700), (64, 64, 100),
                                      (5, 261, 6), (32, 257, 33)])
def test_degenerate_shapes(B, W, L, Bud):
    """Window of one row, L == W (empty prefix), B == W (window only), B >= L (FullKV), tiny prefixes."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, n_q_heads=4, n_kv_heads=2, seq_len=L, window=W,
                     budget_per_head=Bud, floor_per_head=0, n_needles=0, pool_size=3)
    b_cpu = gen.make_batch(cfg, "cpu") if L - W > 8 else None
    if b_cpu is None:
        # the needle planter needs a prefix; draw plain random tensors instead
        g = torch.Generator().manual_seed(L * 100 + W)
        b_cpu = dict(q=torch.randn(2, 4, W, 128, generator=g).bfloat16(),
                     k=torch.randn(2, 2, L, 128, generator=g).bfloat16(),
                     v=torch.randn(2, 2, L, 128, generator=g).bfloat16(),
                     head_w=0.5 + torch.rand(2, 4, generator=g), sens=gen.make_sens(cfg), units=[0, 1])
    prob = problem_of(cfg, 2)
    ref = oracle.compress(prob, *(gen.as_numpy(b_cpu[x]) for x in ("q", "k", "v", "head_w", "sens")))
    out = B.compress(b_cpu["q"].cuda(), b_cpu["k"].cuda(), b_cpu["v"].cuda(), b_cpu["head_w"].cuda(),
                     b_cpu["sens"].cuda(), params_of(B, prob), want_scores=True)
    gpu_idx, gpu_bud, gpu_off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    check_structure(gpu_idx, gpu_bud, gpu_off, prob)
    check_gather(b_cpu["k"], b_cpu["v"], out["k_out"], out["v_out"], gpu_idx, gpu_off, prob)
    if Bud >= L:
        np.testing.assert_array_equal(gen.as_numpy(out["k_out"]).reshape(2, 2, L, 128), gen.as_numpy(b_cpu["k"]))
        np.testing.assert_array_equal(gen.as_numpy(out["v_out"]).reshape(2, 2, L, 128), gen.as_numpy(b_cpu["v"]))
    if L > W:
        gs = out["scores"].double().cpu().numpy()
        rel = np.abs(gs - ref["scores"]) / np.maximum(np.abs(ref["scores"]), 1e-20)
        assert rel.max() <= SCORE_RTOL
        np.testing.assert_array_equal(gpu_idx, oracle.select(prob, gs, gpu_bud, gpu_off))


def test_select_exact_ties_and_extremes(B):
    """Constant and few-valued scores fed straight into ckv_select: the lowest indices win."""
    Nu, Hkv, L, W = 2, 3, 5000, 32
    n = L - W
    rng = np.random.default_rng(5)
    scores = rng.integers(0, 4, (Nu, Hkv, n)).astype(np.float32)
    scores[0, 0] = 1.0
    scores[1, 2, ::7] = -2.5                      # negative values order correctly too
    budgets = np.array([[42, 4000, 32 + n], [32, 4042, n]], np.int32)   # e = 10 / all / none / ...
    rows = int(budgets[0].sum())
    assert budgets[1].sum() == rows
    offsets = np.concatenate([np.zeros((Nu, 1), np.int32), budgets.cumsum(1).astype(np.int32)], 1)
    q = torch.zeros(Nu, Hkv, W, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(Nu, Hkv, L, 128, dtype=torch.bfloat16, device="cuda")
    shape = B.make_shape(q, k)
    assert rows % Hkv == 0
    P = B.Params(budget_per_head=rows // Hkv, floor_per_head=0)
    params = B.make_params(P, None, None)
    ws = B.alloc_workspace(shape, params, "cuda")
    idx = torch.full((Nu, rows), -1, dtype=torch.int32, device="cuda")
    B.ckv_select(shape, params, torch.from_numpy(scores).cuda(), torch.from_numpy(budgets).cuda(),
                 torch.from_numpy(offsets).cuda(), idx, ws)
    prob = Problem(Nu, Hkv, Hkv, L, W, budget_per_head=rows // Hkv)
    want = oracle.select(prob, scores.astype(np.float64), budgets, offsets)
    np.testing.assert_array_equal(idx.cpu().numpy(), want)
    assert idx[0, :8].tolist() == list(range(8))


@pytest.mark.parametrize("n", [700, 1024, 1025, 5000, 32736, 32768, 32769, 40000, 65536, 131040, 200000, 262145])
@pytest.mark.parametrize("dist", ["uniform", "lognormal", "tie_block", "signed"])
def test_select_distributions(B, n, dist):
    """ckv_select alone: one CTA, clusters of 2, 4 and 8 CTAs and the digit path, on score vectors with few or
    many equal values at the cut."""
    Nu, Hkv, W = 2, 4, 32
    L = n + W
    rng = np.random.default_rng(n * 7 + len(dist))
    if dist == "uniform":
        scores = rng.random((Nu, Hkv, n), dtype=np.float32)
    elif dist == "lognormal":
        scores = rng.lognormal(0.0, 3.0, (Nu, Hkv, n)).astype(np.float32)
    elif dist == "signed":
        scores = rng.standard_normal((Nu, Hkv, n)).astype(np.float32)
    else:   # more equal scores at the cut than one key per thread can hold
        scores = rng.random((Nu, Hkv, n), dtype=np.float32)
        scores[:, :, rng.permutation(n)[: min(n - 8, 3000)]] = 0.75
    a, b = min(n - 1, 480), max(1, n // 3)
    b += (-(a + b + n)) % 4
    budgets = np.array([[a, b, 1, n - 1], [n - 1, 1, b, a]], np.int32) + W
    rows = int(budgets[0].sum())
    assert rows % Hkv == 0 and int(budgets[1].sum()) == rows
    offsets = np.concatenate([np.zeros((Nu, 1), np.int32), budgets.cumsum(1).astype(np.int32)], 1)
    q = torch.zeros(Nu, Hkv, W, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(Nu, Hkv, L, 128, dtype=torch.bfloat16, device="cuda")
    shape = B.make_shape(q, k)
    params = B.make_params(B.Params(budget_per_head=rows // Hkv, floor_per_head=0), None, None)
    ws = B.alloc_workspace(shape, params, "cuda")
    idx = torch.full((Nu, rows), -1, dtype=torch.int32, device="cuda")
    B.ckv_select(shape, params, torch.from_numpy(scores).cuda(), torch.from_numpy(budgets).cuda(),
                 torch.from_numpy(offsets).cuda(), idx, ws)
    prob = Problem(Nu, Hkv, Hkv, L, W, budget_per_head=rows // Hkv)
    want = oracle.select(prob, scores.astype(np.float64), budgets, offsets)
    np.testing.assert_array_equal(idx.cpu().numpy(), want)


@pytest.mark.parametrize("n,Nu", [(20000, 80), (40000, 48), (140000, 24)])
def test_select_many_heads_per_cta(B, n, Nu):
    """More heads than the device holds CTAs (clusters of 1, 2 and 8): every CTA loops over several heads, with the
    next head's scores streaming in during the search, and heads that keep nothing or everything of the prefix
    sit between heads that are searched."""
    Hkv, W = 4, 32
    L = n + W
    rng = np.random.default_rng(n + Nu)
    scores = rng.lognormal(0.0, 2.0, (Nu, Hkv, n)).astype(np.float32)
    scores[:, :, ::7] = np.float32(1.5)          # many equal scores, some of them at the cut
    a, b = 480, n // 5
    b += (-(a + b + n)) % 4
    kinds = np.array([0, n, a, b], np.int32)     # nothing, everything, few, many
    budgets = np.stack([np.roll(kinds, u % 4) for u in range(Nu)]) + W
    rows = int(budgets[0].sum())
    assert rows % Hkv == 0
    offsets = np.concatenate([np.zeros((Nu, 1), np.int32), budgets.cumsum(1).astype(np.int32)], 1)
    q = torch.zeros(Nu, Hkv, W, 128, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(Nu, Hkv, L, 128, dtype=torch.bfloat16, device="cuda")   # only its shape is used
    shape = B.make_shape(q, k)
    params = B.make_params(B.Params(budget_per_head=rows // Hkv, floor_per_head=0), None, None)
    ws = B.alloc_workspace(shape, params, "cuda")
    idx = torch.full((Nu, rows), -1, dtype=torch.int32, device="cuda")
    B.ckv_select(shape, params, torch.from_numpy(scores).cuda(), torch.from_numpy(budgets).cuda(),
                 torch.from_numpy(offsets).cuda(), idx, ws)
    assert B.ckv_device_status(ws) == B.OK
    prob = Problem(Nu, Hkv, Hkv, L, W, budget_per_head=rows // Hkv)
    want = oracle.select(prob, scores.astype(np.float64), budgets, offsets)
    np.testing.assert_array_equal(idx.cpu().numpy(), want)


def test_strided_inputs(B):
    """K/V living inside a larger allocation (non-dense unit/head/token strides) give the same result."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, n_q_heads=8, n_kv_heads=2, seq_len=700, budget_per_head=64,
                     n_needles=4)
    b = gen.make_batch(cfg, "cuda")
    prob = problem_of(cfg, 2)
    P = params_of(B, prob)
    dense = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    big_k = torch.zeros(2, 2, 800, 256, dtype=torch.bfloat16, device="cuda")
    big_v = torch.zeros_like(big_k)
    big_k[:, :, 50:750, 128:] = b["k"]
    big_v[:, :, 50:750, 128:] = b["v"]
    kv, vv = big_k[:, :, 50:750, 128:], big_v[:, :, 50:750, 128:]
    big_q = torch.zeros(2, 8, 40, 128, dtype=torch.bfloat16, device="cuda")
    big_q[:, :, 3:35] = b["q"]
    strided = B.compress(big_q[:, :, 3:35], kv, vv, b["head_w"], b["sens"], P, want_scores=True)
    for key in ("scores", "indices", "budgets", "k_out", "v_out"):
        assert torch.equal(dense[key], strided[key]), key


def test_compress_host_matches_device_path(B):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, n_q_heads=8, n_kv_heads=2, seq_len=900, budget_per_head=64,
                     n_needles=4)
    b = gen.make_batch(cfg, "cpu")
    prob = problem_of(cfg, 2)
    P = params_of(B, prob)
    dev = B.compress(*(b[x].cuda() for x in ("q", "k", "v", "head_w", "sens")), P)
    shape = B.make_shape(b["q"], b["k"])
    params = B.make_params(P, b["head_w"], b["sens"])
    rows = B.rows_per_unit(shape, params)
    pin = lambda t: t.pin_memory()
    k_out = pin(torch.zeros(2, rows, 128, dtype=torch.bfloat16))
    v_out = pin(torch.zeros_like(k_out))
    idx = pin(torch.zeros(2, rows, dtype=torch.int32))
    bud = pin(torch.zeros(2, 2, dtype=torch.int32))
    off = pin(torch.zeros(2, 3, dtype=torch.int32))
    staging = torch.empty(B.ckv_staging_bytes(shape, params), dtype=torch.uint8, device="cuda")
    ws = B.alloc_workspace(shape, params, "cuda")
    # page-locked values are read in place by the gather (only the kept rows cross the bus); pageable ones are copied;
    # with the value-norm ratio the values are streamed on the device, hence copied as well: same results every way
    v_pinned = pin(b["v"])
    assert B.ckv_reads_in_place(v_pinned) and not B.ckv_reads_in_place(b["v"])
    for v_host in (v_pinned, b["v"]):
        for t in (k_out, v_out, idx, bud, off):
            t.zero_()
        B.ckv_compress_host(shape, params, pin(b["q"]), pin(b["k"]), v_host, pin(b["head_w"]), pin(b["sens"]),
                            k_out, v_out, idx, bud, off, staging, ws)
        assert torch.equal(idx, dev["indices"].cpu()) and torch.equal(bud, dev["budgets"].cpu())
        assert torch.equal(k_out, dev["k_out"].cpu()) and torch.equal(v_out, dev["v_out"].cpu())
    P.value_norm = True
    dev_vn = B.compress(*(b[x].cuda() for x in ("q", "k", "v", "head_w", "sens")), P)
    params_vn = B.make_params(P, b["head_w"], b["sens"])
    ws_vn = B.alloc_workspace(shape, params_vn, "cuda")
    B.ckv_compress_host(shape, params_vn, pin(b["q"]), pin(b["k"]), v_pinned, pin(b["head_w"]), pin(b["sens"]),
                        k_out, v_out, idx, bud, off, staging, ws_vn)
    assert torch.equal(idx, dev_vn["indices"].cpu()) and torch.equal(v_out, dev_vn["v_out"].cpu())


def test_deterministic_run_to_run(B):
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=3000, budget_per_head=128, n_needles=8)
    b = gen.make_batch(cfg, "cuda")
    P = params_of(B, problem_of(cfg, 2))
    a = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    c = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    for key in ("scores", "indices", "budgets", "k_out", "v_out", "entropy"):
        assert torch.equal(a[key], c[key]), key


@pytest.mark.parametrize("run_tiles", [1, 3, 5, 64])
def test_scan_run_size_does_not_change_the_result(B, run_tiles):
    """The scan hands out its work in runs of key tiles; one tile per run (a single partial pair per run), sizes
    that do not divide the tile count, and one run per chunk all give the oracle's scores and the same selection."""
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=3, seq_len=4500, budget_per_head=128, n_needles=8)
    b = gen.make_batch(cfg, "cuda")
    prob = problem_of(cfg, 3)
    P = params_of(B, prob)
    base = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    prev_path = B.ckv_set_score_path(2)
    prev = B.ckv_set_tunable("run_tiles", run_tiles)
    try:
        out = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
        assert B.ckv_device_status(out["ws"]) == B.OK
    finally:
        B.ckv_set_tunable("run_tiles", prev)
        B.ckv_set_score_path(prev_path)
    rel = ((out["scores"] - base["scores"]).abs() / base["scores"].abs().clamp_min(1e-20)).max().item()
    assert rel < 1e-5, rel
    sc, _ = oracle.score(prob, *(gen.as_numpy(b[x].cpu()) for x in ("q", "k", "head_w")))
    gs = out["scores"].double().cpu().numpy()
    assert (np.abs(gs - sc) / np.maximum(np.abs(sc), 1e-20)).max() <= SCORE_RTOL
    idx, bud, off = (out[x].cpu().numpy() for x in ("indices", "budgets", "offsets"))
    np.testing.assert_array_equal(idx, oracle.select(prob, gs, bud, off))


def test_two_streams_two_work_spaces(B):
    """Calls on different streams with their own work spaces do not disturb each other (the library keeps no
    per-call global state)."""
    cfgs = [gen.shrink(gen.CONFIGS["c2"], n_layers=2, seq_len=3000, budget_per_head=96, n_needles=4),
            gen.shrink(gen.CONFIGS["c5"], n_layers=2, batch=1, seq_len=2100, budget_per_head=128, n_needles=4)]
    batches = [gen.make_batch(c, "cuda") for c in cfgs]
    Ps = [params_of(B, problem_of(c, 2)) for c in cfgs]
    serial = [B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True) for b, P in zip(batches, Ps)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [[], []]
    for rep in range(6):
        for i in (0, 1):
            b = batches[i]
            with torch.cuda.stream(streams[i]):
                outs[i].append(B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], Ps[i], want_scores=True,
                                          stream=streams[i]))
    torch.cuda.synchronize()
    for i in (0, 1):
        for o in outs[i]:
            assert B.ckv_device_status(o["ws"]) == B.OK
            for key in ("scores", "indices", "budgets", "k_out", "v_out"):
                assert torch.equal(o[key], serial[i][key]), (i, key)


def test_per_call_tuning_on_two_threads(B):
    """Scheduling settings travel with the call (params->tuning): two host threads, each on its own stream, run the
    same problem with different settings (run length, L2 hints, dependent launches, score path; one of them with its
    own event pair around the scan) at the same time.  Every call must give the default call's selection, and the
    process-wide defaults must be what they were."""
    import threading
    cfg = gen.shrink(gen.CONFIGS["c2"], n_layers=3, seq_len=4200, budget_per_head=96, n_needles=4)
    b = gen.make_batch(cfg, "cuda")
    P = params_of(B, problem_of(cfg, 3))
    want = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    plain = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True,
                       tuning=B.make_tuning(score_path=1))
    torch.cuda.synchronize()
    ev = (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
    ev[0].record(), ev[1].record()
    torch.cuda.synchronize()
    tunings = [B.make_tuning(run_tiles=3, l2_hints=0, pdl=0, score_path=2, scan_events=ev),
               B.make_tuning(run_tiles=40, group_fuse=1, pdl=1), B.make_tuning(score_path=1)]
    results, errors = [[] for _ in tunings], []

    def worker(i):
        try:
            st = torch.cuda.Stream()
            with torch.cuda.stream(st):
                for _ in range(5):
                    results[i].append(B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True,
                                                 stream=st, tuning=tunings[i]))
            st.synchronize()
        except Exception as e:      # noqa: BLE001 -- reported by the main thread
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(tunings))]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for i, outs_i in enumerate(results):
        ref = plain if i == 2 else want       # the plain kernels round differently from the tensor-core scan
        for o in outs_i:
            assert B.ckv_device_status(o["ws"]) == B.OK
            if i < 2:     # other run length: the row statistics are merged in another order, the last bits may differ
                rel = ((o["scores"] - ref["scores"]).abs() / ref["scores"].abs().clamp_min(1e-20)).max().item()
                assert rel < 1e-5, rel
                assert torch.equal(o["scores"], outs_i[0]["scores"])      # and every call with one setting agrees
            else:
                assert torch.equal(o["scores"], ref["scores"]) and torch.equal(o["indices"], ref["indices"])
    assert ev[0].elapsed_time(ev[1]) > 0.0           # the first thread's scan was bracketed by its own events
    again = B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, want_scores=True)
    assert torch.equal(again["scores"], want["scores"]) and torch.equal(again["indices"], want["indices"])
    # out-of-range settings are argument errors
    with pytest.raises(B.CkvError):
        B.compress(b["q"], b["k"], b["v"], b["head_w"], b["sens"], P, tuning=B.make_tuning(run_tiles=65))
