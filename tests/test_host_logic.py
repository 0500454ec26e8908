"""CPU-only checks of the library's host side: the shared object loads and exports the whole C ABI,
argument errors are reported before anything is launched, the integer budget split used by the
device code agrees with the oracle and with brute force, and the multi-rank sharding works under
gloo with two processes."""
import ctypes as C
import os
import re
import subprocess
import sys

import numpy as np
import pytest

import oracle
from paper_2602_08686_b200 import binding as B
from paper_2602_08686_b200 import build as ckv_build
from paper_2602_08686_b200.sharding import shard_units
from test_oracle_pins import brute_allocate

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    ckv_build.build_lib()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "ckv.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = sorted(set(re.findall(r"\b(ckv_[a-z_]+)\s*\(", header)))
    assert {"ckv_score", "ckv_budget", "ckv_select", "ckv_gather", "ckv_compress"} <= set(names)
    lib = B.lib()
    for n in names:
        assert hasattr(lib, n), n
    assert B.ckv_version() >= 100
    assert B.status_string(B.ERR_TIMEOUT)


def test_header_is_plain_c_and_links(tmp_path):
    """The boundary is a C ABI: the header compiles as C99 and a C program that only knows the header links
    against the library and gets the host-side answers (no GPU involved)."""
    src = tmp_path / "abi.c"
    src.write_text(r"""
#include <stdio.h>
#include <string.h>
#include "ckv.h"
int main(void) {
  ckv_shape s; ckv_params p;
  memset(&s, 0, sizeof s); memset(&p, 0, sizeof p);
  s.n_units = 2; s.n_q_heads = 32; s.n_kv_heads = 8; s.head_dim = 128; s.seq_len = 4096; s.window = 32; s.dtype = CKV_BF16;
  s.q_stride_row = 128; s.q_stride_head = 32 * 128; s.q_stride_unit = 32 * 32 * 128;
  s.kv_stride_tok = 128; s.kv_stride_head = 4096 * 128; s.kv_stride_unit = 8 * 4096 * 128;
  p.pool_kind = CKV_POOL_MAX; p.pool_size = 7; p.budget_per_head = 512; p.floor_per_head = 1; p.n_buckets = 16;
  p.bucket_override = -1; p.head_w_stride_unit = 32;
  printf("%d %zu %zu %s\n", ckv_version(), ckv_workspace_bytes(&s, &p), ckv_score_workspace_bytes(&s, &p),
         ckv_status_string(CKV_ERR_TIMEOUT));
  s.head_dim = 64;
  return ckv_workspace_bytes(&s, &p) == 0 ? 0 : 1;
}
""")
    exe = tmp_path / "abi"
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"), str(src),
                           "-o", str(exe), "-L", libdir, "-l:libckv.so", "-Wl,-rpath," + libdir])
    out = subprocess.run([str(exe)], stdout=subprocess.PIPE, check=True).stdout.decode().split()
    assert int(out[0]) >= 100 and int(out[1]) > int(out[2]) > 0


def llama_shape(L=32768, W=32, Nu=2, H=32, Hkv=8, d=128, dtype=B.BF16):
    return B.ckv_shape(Nu, H, Hkv, d, L, W, dtype, 0, H * W * d, W * d, d, Hkv * L * d, L * d, d)


def default_params(**kw):
    base = dict(pool_kind=B.POOL_MAX, pool_size=7, budget_per_head=512, floor_per_head=1, n_buckets=16,
                bucket_override=-1, head_w_stride_unit=32, sens_stride_unit=0, value_norm=0, value_norm_eps=1e-6,
                shared_elastic=0, global_alpha=0, units_per_prompt=1, reserved_=0)
    base.update(kw)
    return B.ckv_params(*[base[k] for k in ("pool_kind", "pool_size", "budget_per_head", "floor_per_head",
                                            "n_buckets", "bucket_override", "head_w_stride_unit",
                                            "sens_stride_unit", "value_norm", "value_norm_eps", "shared_elastic",
                                            "global_alpha", "units_per_prompt", "reserved_")])


def test_argument_errors_are_found_on_the_host():
    lib = B.lib()
    s, p = llama_shape(), default_params()
    assert B.ckv_workspace_bytes(s, p) > 0
    fake = C.c_void_p(256 * 1024)      # never dereferenced: every call below fails validation first
    big = 1 << 40

    def score(shape, params, ws=fake, ws_bytes=big, q=fake):
        return lib.ckv_score(C.byref(shape), C.byref(params), q, fake, fake, fake, fake, ws, ws_bytes, None)

    assert score(llama_shape(d=64), p) == B.ERR_UNSUPPORTED
    assert score(llama_shape(W=65), p) == B.ERR_UNSUPPORTED
    assert score(llama_shape(H=30), p) == B.ERR_INVALID_ARG
    assert score(llama_shape(L=16), p) == B.ERR_INVALID_ARG                       # window > seq_len
    assert score(s, default_params(pool_size=4)) == B.ERR_INVALID_ARG
    assert score(s, default_params(pool_size=17)) == B.ERR_INVALID_ARG
    assert score(s, default_params(budget_per_head=16)) == B.ERR_INVALID_ARG      # B < W
    assert score(s, default_params(floor_per_head=500)) == B.ERR_INVALID_ARG      # f > B - W
    assert score(s, default_params(bucket_override=16)) == B.ERR_INVALID_ARG
    assert score(s, default_params(value_norm=2)) == B.ERR_INVALID_ARG
    assert score(s, default_params(shared_elastic=3)) == B.ERR_INVALID_ARG
    assert score(s, default_params(global_alpha=1, units_per_prompt=3)) == B.ERR_INVALID_ARG   # 2 units
    assert score(s, default_params(global_alpha=1, units_per_prompt=0)) == B.ERR_INVALID_ARG
    assert B.ckv_workspace_bytes(s, default_params(global_alpha=1, units_per_prompt=2)) > B.ckv_workspace_bytes(s, p)
    assert score(s, default_params(value_norm_eps=-1.0)) == B.ERR_INVALID_ARG
    assert score(s, default_params(value_norm_eps=float("nan"))) == B.ERR_INVALID_ARG
    assert lib.ckv_vnorm(C.byref(s), C.byref(p), None, fake, None, fake, big, None) == B.ERR_INVALID_ARG
    assert lib.ckv_vnorm(C.byref(s), C.byref(p), fake, fake, None, fake, 1024, None) == B.ERR_WORKSPACE
    assert B.ckv_workspace_bytes(s, default_params(value_norm=1)) > B.ckv_workspace_bytes(s, p)   # holds rho
    assert score(s, p, q=None) == B.ERR_INVALID_ARG
    assert score(s, p, q=C.c_void_p(256 * 1024 + 2)) == B.ERR_INVALID_ARG         # misaligned
    assert score(s, p, ws=None) == B.ERR_WORKSPACE
    assert score(s, p, ws_bytes=1024) == B.ERR_WORKSPACE
    bad = llama_shape()
    bad.kv_stride_tok = 130                                                       # rows not 16-byte aligned
    assert score(bad, p) == B.ERR_INVALID_ARG
    assert B.ckv_workspace_bytes(llama_shape(d=64), p) == 0
    # broadcast views (a zero stride over more than one unit or head) are refused; over an extent of one they are fine
    for field in ("q_stride_unit", "q_stride_head", "kv_stride_unit", "kv_stride_head"):
        bad = llama_shape()
        setattr(bad, field, 0)
        assert score(bad, p) == B.ERR_INVALID_ARG, field
    one = llama_shape(Nu=1)
    one.q_stride_unit = one.kv_stride_unit = 0
    assert B.ckv_workspace_bytes(one, p) > 0
    # per-call scheduling settings: -1 or a value in range
    for field, value in (("run_tiles", 0), ("run_tiles", 65), ("score_path", 3), ("l2_hints", 2), ("pdl", -2)):
        t = B.make_tuning()
        setattr(t, field, value)
        bad_t = default_params()
        bad_t.tuning = C.pointer(t)
        assert score(s, bad_t) == B.ERR_INVALID_ARG, field
    ok_t = default_params()
    ok_t.tuning = C.pointer(B.make_tuning(run_tiles=8, pdl=0))
    assert B.ckv_workspace_bytes(s, ok_t) == B.ckv_workspace_bytes(s, p)
    # the four-axis gate table: its sizes must be given, and it is one table for all units
    coords = C.cast(fake, C.c_void_p)
    gate = default_params(n_buckets=20)
    gate.gate_coords, gate.n_gate_layers, gate.n_ppl_bins, gate.n_budget_levels = coords, 32, 4, 3
    assert B.ckv_workspace_bytes(s, gate) > 0
    for field, value in (("n_gate_layers", 0), ("n_ppl_bins", 0), ("n_budget_levels", -1), ("sens_stride_unit", 20)):
        bad_gate = default_params(n_buckets=20)
        bad_gate.gate_coords, bad_gate.n_gate_layers, bad_gate.n_ppl_bins, bad_gate.n_budget_levels = coords, 32, 4, 3
        setattr(bad_gate, field, value)
        assert score(s, bad_gate) == B.ERR_INVALID_ARG, field
    assert lib.ckv_gather(C.byref(s), C.byref(p), None, fake, fake, fake, fake, fake, None) == B.ERR_INVALID_ARG
    assert lib.ckv_compress_host(C.byref(s), C.byref(p), fake, fake, fake, fake, fake, fake, fake, fake, fake, fake,
                                 fake, 16, fake, big, None) == B.ERR_WORKSPACE    # staging too small


def test_workspace_grows_with_the_problem():
    p = default_params()
    a = B.ckv_workspace_bytes(llama_shape(L=4096), p)
    b = B.ckv_workspace_bytes(llama_shape(L=32768), p)
    c = B.ckv_workspace_bytes(llama_shape(L=32768, Nu=4), p)
    assert 0 < a < b < c
    assert B.ckv_staging_bytes(llama_shape(L=4096), p) > 2 * 2 * 8 * 4096 * 128 * 2


def test_score_stage_work_space_and_the_fixed_scratch_limit():
    """ckv_score needs only the leading sections of the work space, and ckv_score_noalloc accepts what fits its
    fixed scratch by that measure: two units of the Llama shape at 32k do, three do not."""
    p = default_params()
    for Nu in (1, 2, 3):
        s = llama_shape(Nu=Nu)
        assert 0 < B.ckv_score_workspace_bytes(s, p) < B.ckv_workspace_bytes(s, p)
    assert B.ckv_score_workspace_bytes(llama_shape(Nu=2), p) <= B.NOALLOC_SCRATCH_BYTES
    assert B.ckv_score_workspace_bytes(llama_shape(Nu=3), p) > B.NOALLOC_SCRATCH_BYTES
    fake = C.c_void_p(1 << 20)   # never dereferenced: the call fails the size test first
    s3 = llama_shape(Nu=3)
    assert B.lib().ckv_score_noalloc(C.byref(s3), C.byref(p), fake, fake, fake, fake, fake, None) == B.ERR_WORKSPACE


def test_depth_map_matches_the_oracle():
    rng = np.random.default_rng(3)
    import torch
    for n_src, n_dst in ((32, 32), (32, 28), (32, 80), (4, 9), (6, 1), (1, 5)):
        table = rng.uniform(0.8, 1.0, (n_src, 20, 4, 2)).astype(np.float32)
        got = B.ckv_gate_depth_map_host(torch.from_numpy(table), n_dst).numpy()
        want = oracle.depth_map(table, n_dst)
        assert got.shape == want.shape
        np.testing.assert_allclose(got, want, rtol=1e-6, atol=0)
        if n_src == n_dst:
            np.testing.assert_array_equal(got, table)
        np.testing.assert_array_equal(got[0], table[0])
    assert B.lib().ckv_gate_depth_map_host(None, 4, 4, 8, None) == 1


def test_binding_refuses_values_laid_out_unlike_the_keys():
    """ckv_shape has one set of strides for k and v: the binding raises when v is another view."""
    import torch
    q = torch.zeros(2, 4, 8, 128, dtype=torch.bfloat16)
    k = torch.zeros(2, 2, 64, 128, dtype=torch.bfloat16)
    shape = B.make_shape(q, k)
    B._check_kv(shape, k, "k")
    B._check_kv(shape, torch.zeros_like(k), "v")
    padded = torch.zeros(2, 2, 64, 256, dtype=torch.bfloat16)[..., :128]          # other token stride
    for bad in (padded, torch.zeros(2, 2, 63, 128, dtype=torch.bfloat16), k.float(),
                torch.zeros(2, 64, 2, 128, dtype=torch.bfloat16).transpose(1, 2)):
        with pytest.raises(ValueError):
            B._check_kv(shape, bad, "v")
    with pytest.raises(ValueError):
        B._check_dense(padded, "k_out")


def test_budget_split_matches_oracle_and_brute_force():
    rng = np.random.default_rng(11)
    for Hkv in (1, 2, 3, 4, 8):
        for _ in range(300):
            n = int(rng.integers(1, 60))
            f = int(rng.integers(0, n + 1))
            P = int(rng.integers(f * Hkv, n * Hkv + 1))
            lo = max(f, 1)
            dem = rng.integers(lo, max(lo, n) + 1, Hkv)
            if rng.random() < 0.4:
                dem[:] = dem[0]                                                   # equal demands
            got = B.ckv_allocate_rows_host(n, f, P, dem)
            assert got == list(oracle.allocate(n, f, P, dem)), (n, f, P, dem)
            if Hkv <= 4:
                assert got == brute_allocate(n, f, P, dem)
    # sizes of the real workloads
    for n, f, B_, Hkv in ((32736, 1, 512, 8), (131040, 1, 2048, 8), (65472, 8, 128, 4)):
        for _ in range(50):
            dem = rng.integers(max(f, 1), n + 1, Hkv) // rng.integers(1, 2000, Hkv) + max(f, 1)
            dem = np.minimum(dem, n)
            P = Hkv * (B_ - (64 if Hkv == 4 else 32))
            got = B.ckv_allocate_rows_host(n, f, P, dem)
            assert got == list(oracle.allocate(n, f, P, dem))
            assert sum(got) == P and min(got) >= f and max(got) <= n


def test_shard_units_partitions():
    for n in (1, 7, 32, 512):
        for world in (1, 2, 3, 8):
            parts = [shard_units(n, r, world) for r in range(world)]
            assert sorted(x for p in parts for x in p) == list(range(n))
            sizes = [len(p) for p in parts]
            assert max(sizes) - min(sizes) <= 1


_GLOO_WORKER = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
from paper_2602_08686_b200.sharding import shard_units, max_over_ranks, allreduce_prompt_mass
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:" + sys.argv[2], rank=int(sys.argv[3]), world_size=2)
rank = dist.get_rank()
mine = shard_units(33, rank, 2)
t = torch.zeros(33, dtype=torch.int64); t[list(mine)] = 1
dist.all_reduce(t)
assert (t == 1).all(), t
elapsed = max_over_ranks(1.0 + rank)
assert elapsed == 2.0, elapsed
total = torch.tensor([float(len(mine))]); dist.all_reduce(total)
assert total.item() == 33.0
# prompt-global mode: 3 prompts x 8 layers, each rank holds 4 layers of every prompt; the ranks' partial
# window masses add up to the sum over all layers (what one process holding all units computes)
g = torch.Generator().manual_seed(7)
mass = torch.rand(3, 8, 50, generator=g)                     # [prompt, layer, L], the same on both ranks
mine_layers = mass[:, 4 * rank: 4 * rank + 4]
pm = mine_layers.sum(1)                                      # stands in for ckv_prompt_mass on the local units
allreduce_prompt_mass(pm)
assert torch.allclose(pm, mass.sum(1), rtol=1e-6), (pm - mass.sum(1)).abs().max()
dist.barrier(); dist.destroy_process_group()
print("rank", rank, "ok")
"""


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` outside a launcher starts two ranks itself; with --dry-run they are CPU ranks under gloo
    whose step is a sleep (rank r sleeps r + 1 ms), so the line must say two GPUs, twice the units and the slower
    rank's time."""
    import json
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--steps", "5", "--dry-run"],
                         stdout=subprocess.PIPE, stderr=subprocess.PIPE, env=env, timeout=300)
    assert res.returncode == 0, res.stderr.decode()[-2000:]
    lines = [ln for ln in res.stdout.decode().splitlines() if ln.startswith("{")]
    assert len(lines) == 1, lines
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["config"]["units_total"] == 64 and line["config"]["units_per_gpu"] == 32
    assert line["ms_per_step"] >= 2.0 and line["scaling"] == "weak"


def test_two_rank_sharding_under_gloo(tmp_path):
    """World size 2 on CPU: the ranks' shards cover every unit once and the timing reduction is a MAX."""
    script = tmp_path / "worker.py"
    script.write_text(_GLOO_WORKER)
    port = str(29000 + os.getpid() % 2000)
    procs = [subprocess.Popen([sys.executable, str(script), ROOT, port, str(r)], stdout=subprocess.PIPE,
                              stderr=subprocess.STDOUT) for r in range(2)]
    outs = [p.communicate(timeout=180)[0].decode() for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
