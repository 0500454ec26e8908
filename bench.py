#!/usr/bin/env python
"""Benchmark of the end-of-prefill KV retention pass (one JSON line on stdout).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload c2|c4|...]

A step is one call of the fused ``ckv_compress`` over one batch of synthetic units (sequence x layer
pairs) resident in HBM.  The default workload is the Llama-3-8B-shaped pass at L = 32768 (32 units,
512 rows kept per KV head).  With ``--gpus N`` above one the script starts N ranks of itself (one per GPU,
``torch.distributed.run``) unless it already runs under such a launcher; every rank runs the same number of
its own units (weak scaling, no data-path collective) and the time is the max over ranks.  On one GPU the
line also carries, under ``also``, the same measurement at L = 131072 (c4), for the batch-16 workload (c3,
when the device has the memory) and for the headline workload run back to back for at least two seconds
(the figure under the power cap), each with its own clock record.  ``--impl reference`` times the fp64 CPU
oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2602_08686_b200 import inputs as gen  # noqa: E402
from paper_2602_08686_b200.sharding import max_over_ranks  # noqa: E402

METRIC = "prefill_tokens_compressed_per_sec_per_layer"
UNIT = "tokens/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of score_tc_kernel per unit, from ncu captures of small launches of
# the workload's shape (profiles/score_tc_kernel_c2_8units.md: 8 units; 2 units for the 128k shape; all 112 of config 5).  A launch's
# traffic is this times its units (every unit streams its own K once per pass).  Each entry names the kernel source
# it was taken from (first 12 hex digits of its SHA-256): when the source has changed since, the counters no longer
# describe the kernel that is timed and the line says null.
SCAN_SOURCE = os.path.join(ROOT, "paper_2602_08686_b200", "csrc", "score_tc.cu")
SCAN_DRAM_TRAFFIC_PER_UNIT = {
    "c2": {"source": "4ebc2264eec8", "bytes": (1.019676e9 + 8.599552e6) / 8},
    "c3": {"source": "4ebc2264eec8", "bytes": (1.019676e9 + 8.599552e6) / 8},
    "c4": {"source": "4ebc2264eec8", "bytes": (1.014877952e9 + 7.403008e6) / 2},
    "c5": {"source": "4ebc2264eec8", "bytes": (1.821095936e9 + 5.0745088e7) / 112},   # the whole workload was captured
}


def scan_source_hash() -> str:
    with open(SCAN_SOURCE, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:12]


def scan_traffic(workload: str, n_units: int):
    """DRAM bytes of one scan launch from the committed ncu capture, or None if there is none for this kernel."""
    entry = SCAN_DRAM_TRAFFIC_PER_UNIT.get(workload)
    if entry is None or entry["source"] != scan_source_hash():
        return None
    return entry["bytes"] * n_units


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.thread = [], None, None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def wait_first_row(self, limit_s: float) -> None:
        t_end = time.time() + limit_s
        while self.proc is not None and not self.rows and time.time() < t_end:
            time.sleep(0.01)

    def stop(self) -> None:
        if self.proc is not None:
            self.proc.terminate()

    def window(self, t0: float, t1: float) -> dict:
        """Median SM clock and the throttle reasons seen between two wall-clock times."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        rows = [r for t, r in self.rows if t0 <= t <= t1 + 0.1] or [r for _, r in self.rows[-3:]]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            c = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(c[0]))
                smax.append(float(c[1]))
            except (ValueError, IndexError):
                continue
            for nme, val in zip(names, c[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nme)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_problem(cfg, Nu):
    import oracle
    return oracle.Problem(Nu, cfg.n_q_heads, cfg.n_kv_heads, cfg.seq_len, cfg.window, head_dim=cfg.head_dim,
                          dtype=oracle.BF16 if cfg.dtype == "bf16" else oracle.F32, pool_kind=cfg.pool_kind,
                          pool_size=cfg.pool_size, budget_per_head=cfg.budget_per_head,
                          floor_per_head=cfg.floor_per_head, n_buckets=cfg.n_buckets)


def time_oracle(cfg, batch_cpu, n_sample_units, repeats=1):
    """Seconds per run of the oracle's whole pass on the first n_sample_units units (host tensors)."""
    import oracle
    prob = oracle_problem(cfg, n_sample_units)
    args = [gen.as_numpy(batch_cpu[x][:n_sample_units]) for x in ("q", "k", "v", "head_w")]
    args.append(gen.as_numpy(batch_cpu["sens"]))
    best = float("inf")
    for _ in range(repeats):
        t = time.perf_counter()
        oracle.compress(prob, *args, want_scores=False)
        best = min(best, time.perf_counter() - t)
    return best, oracle.num_threads()


def algorithmic_bytes(cfg, n_units):
    """K read twice plus the kept K/V rows read and written (the benchmark's roofline definition)."""
    esz = 2 if cfg.dtype == "bf16" else 4
    k_bytes = n_units * cfg.n_kv_heads * cfg.seq_len * cfg.head_dim * esz
    rows = n_units * cfg.n_kv_heads * min(cfg.budget_per_head, cfg.seq_len)
    gather = 4 * rows * cfg.head_dim * esz
    return 2 * k_bytes, gather


def config_dict(cfg, n_units_per_gpu, world):
    return {"workload": cfg.name, "shape": f"{cfg.n_q_heads}q/{cfg.n_kv_heads}kv heads, d {cfg.head_dim}",
            "seq_len": cfg.seq_len, "window": cfg.window, "budget_per_head": cfg.budget_per_head,
            "pool": f"{'none max avg'.split()[cfg.pool_kind]}{cfg.pool_size}", "units_per_gpu": n_units_per_gpu,
            "units_total": n_units_per_gpu * world, "parallelism": f"dp{world} over units (no collective)",
            "l2": "inputs (K+V %.1f GB per GPU) exceed the 126 MB L2; no flush needed" %
                  (2 * n_units_per_gpu * cfg.n_kv_heads * cfg.seq_len * cfg.head_dim *
                   (2 if cfg.dtype == "bf16" else 4) / 1e9)}


def run_reference(args, cfg, rank, world):
    """The oracle, as it stands, on the host cores: each step is one unit of the workload."""
    if rank != 0:
        return
    sample_units = 1
    units = list(range(sample_units))
    batch = gen.make_batch(cfg, "cpu", units)
    for _ in range(max(args.warmup, 0)):
        time_oracle(cfg, batch, sample_units)
    t0 = time.perf_counter()
    cores = 1
    for _ in range(args.steps):
        _, cores = time_oracle(cfg, batch, sample_units)
    el = time.perf_counter() - t0
    value = args.steps * sample_units * cfg.seq_len / el
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": config_dict(cfg, sample_units, 1),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{sample_units} unit(s) of {cfg.name} per step (whole pass, fp64)"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


class Workload:
    """One workload's units resident on the device, with every buffer a fused step needs."""

    def __init__(self, B, cfg, n_units, first_unit, dev, value_norm=False):
        self.B, self.cfg, self.n_units, self.dev = B, cfg, n_units, dev
        self.batch = gen.make_batch(cfg, dev, [first_unit + u for u in range(n_units)])
        b = self.batch
        P = B.Params(pool_kind=cfg.pool_kind, pool_size=cfg.pool_size, budget_per_head=cfg.budget_per_head,
                     floor_per_head=cfg.floor_per_head, n_buckets=cfg.n_buckets, value_norm=value_norm)
        self.shape = B.make_shape(b["q"], b["k"])
        self.params = B.make_params(P, b["head_w"], b["sens"])
        self.ws = B.alloc_workspace(self.shape, self.params, dev)
        Hkv, L, n = cfg.n_kv_heads, cfg.seq_len, cfg.n
        rows = B.rows_per_unit(self.shape, self.params)
        self.k_out = torch.empty(n_units, rows, cfg.head_dim, dtype=b["k"].dtype, device=dev)
        self.v_out = torch.empty_like(self.k_out)
        self.indices = torch.empty(n_units, rows, dtype=torch.int32, device=dev)
        self.budgets = torch.empty(n_units, Hkv, dtype=torch.int32, device=dev)
        self.offsets = torch.empty(n_units, Hkv + 1, dtype=torch.int32, device=dev)
        self.scores = torch.empty(n_units, Hkv, n, dtype=torch.float32, device=dev)
        self.colmass = torch.empty(n_units, L, dtype=torch.float32, device=dev)
        self.bucket = torch.empty(n_units, dtype=torch.int32, device=dev)
        self.entropy = torch.empty(n_units, dtype=torch.float32, device=dev)

    def step(self):
        b = self.batch
        self.B.ckv_compress(self.shape, self.params, b["q"], b["k"], b["v"], b["head_w"], b["sens"], self.k_out,
                            self.v_out, self.indices, self.budgets, self.offsets, self.ws)

    def timed(self, steps, barrier=lambda: torch.cuda.synchronize(), min_seconds=0.0):
        """`steps` fused steps (or as many more as it takes to fill min_seconds) between CUDA events, with a pair of
        events around the scan kernel of every step.  Returns (ms per step, scan ms per step, steps, t0, t1, launches)."""
        B = self.B
        pairs = []

        def new_pair():
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record(), b_.record()       # a first record creates the handles
            pairs.append((a_, b_))

        for _ in range(steps):
            new_pair()
        barrier()
        launches0 = B.ckv_kernel_launches()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record()
        done = 0
        while True:
            for it in range(done, len(pairs)):
                B.ckv_set_scan_events(*pairs[it])
                self.step()
            done = len(pairs)
            if time.time() - t0 >= min_seconds:
                break
            torch.cuda.synchronize()        # the queue may run far ahead of the device: look at the clock after it drains
            if time.time() - t0 >= min_seconds:
                break
            for _ in range(steps):
                new_pair()
        e1.record()
        B.ckv_set_scan_events(None, None)
        barrier()
        t1 = time.time()
        if B.ckv_device_status(self.ws) != B.OK:
            raise SystemExit("device-side wait timed out")
        scan_ms = sum(a_.elapsed_time(b_) for a_, b_ in pairs) / len(pairs)
        return e0.elapsed_time(e1) / len(pairs), scan_ms, len(pairs), t0, t1, B.ckv_kernel_launches() - launches0

    def stage_times(self, steps, value_norm=False):
        """Per-stage times of the same kernels through the staged entry points."""
        B, b = self.B, self.batch
        names = ["score", "budget", "select", "gather"]
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
        for ev in evs:
            ev[0].record()
            B.ckv_score(self.shape, self.params, b["q"], b["k"], b["head_w"], self.scores, self.colmass, self.ws)
            ev[1].record()
            B.ckv_budget(self.shape, self.params, self.scores, self.colmass, b["sens"], self.budgets, self.offsets,
                         self.bucket, self.entropy, self.ws)
            ev[2].record()
            B.ckv_select(self.shape, self.params, self.scores, self.budgets, self.offsets, self.indices, self.ws)
            ev[3].record()
            B.ckv_gather(self.shape, self.params, b["k"], b["v"], self.indices, self.offsets, self.k_out, self.v_out)
            ev[4].record()
        torch.cuda.synchronize()
        out = {nm: sum(ev[j].elapsed_time(ev[j + 1]) for ev in evs) / steps for j, nm in enumerate(names)}
        if value_norm:   # the extra stage, timed alone: V streamed once, scores rescaled
            rho = torch.empty(self.n_units, self.cfg.n_kv_heads, self.cfg.seq_len, device=self.dev)
            va, vb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            B.ckv_vnorm(self.shape, self.params, b["v"], rho, self.scores, self.ws)
            va.record()
            for _ in range(steps):
                B.ckv_vnorm(self.shape, self.params, b["v"], rho, self.scores, self.ws)
            vb.record()
            torch.cuda.synchronize()
            out["value_norm"] = va.elapsed_time(vb) / steps
        return out


def roofline_of(cfg, n_units, ms_per_step, scan_ms, clocks, sm_count, value_norm=False):
    """The roofline object of one measurement: K-twice bytes over the scan's time against the measured copy rate,
    the whole pass beside it, and the scan's other ceiling (exponentials on the special-function unit)."""
    peak, peak_kind = measured_peaks()
    k2_bytes, gather_bytes = algorithmic_bytes(cfg, n_units)
    if value_norm:
        gather_bytes += k2_bytes // 2     # V read once: as many bytes as one pass over K
    scan_gbs = k2_bytes / (scan_ms * 1e-3) / 1e9
    whole = (k2_bytes + gather_bytes) / (ms_per_step * 1e-3)
    roofline = {"bound": "hbm", "kernel": "score_tc_kernel (window-score scan, both passes over K)",
                "achieved": scan_gbs, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                "frac": scan_gbs / peak, "traffic": scan_traffic(cfg.name, n_units),
                "algorithmic_bytes_per_launch": k2_bytes, "ms_per_launch": scan_ms,
                "whole_pass": {"algorithmic_bytes": k2_bytes + gather_bytes, "achieved": whole / 1e9,
                               "frac": whole / 1e9 / peak, "frac_of_nominal_8TBs": whole / 8e12}}
    # The scan's other ceiling: one ex2 per (query row, key) and pass on the special-function unit, 16 per clock and SM.
    n_exp = 2.0 * n_units * cfg.n_q_heads * cfg.window * cfg.seq_len
    sm_max_mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
    exp_peak = 16.0 * sm_count * sm_max_mhz * 1e6 / 1e9          # G exp/s at the maximum SM clock
    exp_rate = n_exp / (scan_ms * 1e-3) / 1e9
    alu = {"bound": "alu", "what": "ex2.approx on the special-function unit: 2*H*W*L per unit, 16 per clock and SM "
                                   "at the maximum SM clock",
           "achieved": exp_rate, "peak": exp_peak, "unit": "Gexp/s", "frac": exp_rate / exp_peak}
    if alu["frac"] > roofline["frac"]:      # many query rows per key byte: the exponentials bind, not HBM
        hbm = {k_: roofline[k_] for k_ in ("bound", "achieved", "peak", "peak_kind", "unit", "frac")}
        roofline.update({k_: alu[k_] for k_ in ("bound", "achieved", "peak", "unit", "frac")})
        roofline["peak_kind"] = "derived: 16 ex2 per clock per SM x SMs x maximum SM clock"
        roofline["what"] = alu["what"]
        roofline["hbm"] = hbm
    else:
        roofline["alu"] = alu
    return roofline


def side_record(B, cfg, n_units, steps, dev, sampler, sm_count, min_seconds=0.0, workload=None):
    """One entry of the line's `also` object: a workload measured like the headline one (device-resident, CUDA
    events, clock record), without the end-to-end and CPU legs."""
    wl = workload or Workload(B, cfg, n_units, 0, dev)
    for _ in range(3):
        wl.step()
    ms, scan_ms, n_steps, t0, t1, _ = wl.timed(steps, min_seconds=min_seconds)
    clocks = sampler.window(t0, t1) if sampler else None
    roof = roofline_of(cfg, n_units, ms, scan_ms, clocks, sm_count)
    rec = {"workload": cfg.name, "units": n_units, "seq_len": cfg.seq_len, "budget_per_head": cfg.budget_per_head,
           "steps": n_steps, "seconds": round(t1 - t0, 3), "ms_per_step": ms, "value": n_units * cfg.seq_len / (ms * 1e-3),
           "unit": UNIT, "scan_ms": scan_ms, "scan_frac": roof["hbm"]["frac"] if "hbm" in roof else roof["frac"],
           "whole_pass_frac": roof["whole_pass"]["frac"], "peak_kind": "of " + measured_peaks()[1],
           "traffic": roof["traffic"], "clocks": clocks}
    if clocks and clocks.get("sm_mhz"):
        rec["ms_times_mhz"] = ms * clocks["sm_mhz"]      # time x clock: how far the step follows the SM clock
    if workload is None:
        rec["stage_ms"] = wl.stage_times(min(steps, 10))
        del wl
        torch.cuda.empty_cache()
    return rec


def launch_ranks(n: int) -> None:
    """Starts n ranks of this script on this node (one per GPU) and leaves with their exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr",
           "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    raise SystemExit(subprocess.call(cmd))


def dry_run(args, cfg, rank, world):
    """The launcher and timing path without a GPU (gloo): every rank 'runs' its units by sleeping.  Used by the CPU test."""
    import torch.distributed as dist
    if world > 1:
        dist.init_process_group("gloo")
    n_units = args.units or cfg.n_units
    t = time.perf_counter()
    for _ in range(args.steps):
        time.sleep(0.001 * (1 + rank))
    ms_total = max_over_ranks((time.perf_counter() - t) * 1e3)
    if rank == 0:
        ms = ms_total / args.steps
        print(json.dumps({"metric": METRIC, "value": world * n_units * cfg.seq_len / (ms * 1e-3), "unit": UNIT,
                          "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
                          "higher_is_better": True, "scaling": "weak", "data": "none (dry run)",
                          "config": config_dict(cfg, n_units, world), "gpu_launches": 0}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(gen.CONFIGS))
    ap.add_argument("--units", type=int, default=0, help="units per GPU (default: the workload's)")
    ap.add_argument("--value-norm", action="store_true",
                    help="also apply Eq. 4's value-norm ratio (streams V once more; not the headline configuration)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-also", action="store_true", help="skip the 128k, batch-16 and sustained side records")
    ap.add_argument("--dry-run", action="store_true", help="launcher and timing path only, on CPU ranks (for tests)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        launch_ranks(args.gpus)          # does not return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = gen.CONFIGS[args.workload]

    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
        return
    if args.dry_run:
        dry_run(args, cfg, rank, world)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the retention pass has no CPU fallback")
    from paper_2602_08686_b200 import binding as B
    B.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    import torch.distributed as dist
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")      # the communicator's log names the ranks that joined
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        dist.init_process_group("nccl", device_id=dev)   # for the barrier and the MAX of the times only

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    n_units = args.units or cfg.n_units
    wl = Workload(B, cfg, n_units, rank * n_units, dev, value_norm=args.value_norm)
    batch, shape, params, ws = wl.batch, wl.shape, wl.params, wl.ws
    L = cfg.seq_len
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count

    # ---- device-resident timing ---------------------------------------------------------------
    # the clock sampler runs from before the warm-up (nvidia-smi takes a while to print its first row on a fresh box)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        wl.step()
    if sampler is not None:
        sampler.wait_first_row(3.0)
    ms_mine, scan_ms, _, t0, t1, launches = wl.timed(args.steps, barrier=barrier)
    ms_per_step = max_over_ranks(ms_mine)
    clocks = sampler.window(t0, t1) if sampler else None
    value = world * n_units * L / (ms_per_step * 1e-3)
    roofline = roofline_of(cfg, n_units, ms_per_step, scan_ms, clocks, sm_count, value_norm=args.value_norm)
    roofline["stage_ms"] = wl.stage_times(args.steps, value_norm=args.value_norm)

    # ---- the same step back to back for at least two seconds: the figure under the power cap ------------
    also = {}
    if world == 1 and not args.no_also:
        time.sleep(0.5)
        also[cfg.name + "_sustained"] = side_record(B, cfg, n_units, args.steps, dev, sampler, sm_count,
                                                    min_seconds=2.0, workload=wl)

    # ---- end to end through ckv_compress_host (pinned host buffers, copies inside the timed region) ----
    e2e = None
    k_out, v_out, indices, budgets, offsets = wl.k_out, wl.v_out, wl.indices, wl.budgets, wl.offsets
    if not args.no_e2e:
        pin = lambda t: t.cpu().pin_memory()
        hq, hk, hv, hw, hs = (pin(batch[x]) for x in ("q", "k", "v", "head_w", "sens"))
        hko, hvo = pin(k_out), pin(v_out)
        hidx, hbud, hoff = pin(indices), pin(budgets), pin(offsets)
        staging = torch.empty(B.ckv_staging_bytes(shape, params), dtype=torch.uint8, device=dev)
        # V is read in place when the pinned buffer is mapped: only the kept rows cross the bus (as many bytes as v_out)
        v_bytes = hvo.numel() * hvo.element_size() if B.ckv_reads_in_place(hv) and not args.value_norm else \
            hv.numel() * hv.element_size()
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hw, hs)) + v_bytes
        d2h = sum(t.numel() * t.element_size() for t in (hko, hvo, hidx, hbud, hoff))
        e2e_steps = max(1, min(args.steps, 3))

        def host_step():
            B.ckv_compress_host(shape, params, hq, hk, hv, hw, hs, hko, hvo, hidx, hbud, hoff, staging, ws)

        host_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            host_step()
        e1.record()
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1)) / e2e_steps
        e2e = {"value": world * n_units * L / (ms_e2e * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e, "steps": e2e_steps,
               "api": "ckv_compress_host (pinned host tensors)",
               "values": "kept rows read in place from the pinned host buffer" if v_bytes < hv.numel() * hv.element_size()
               else "copied whole"}
        wl.step()
        torch.cuda.synchronize()
        assert torch.equal(hidx, indices.cpu())
        del staging, hq, hk, hv, hko, hvo

    # ---- quality of the selection on this synthetic workload (Prop. 4.1's discarded mass; not timed) ----
    wl.step()
    kept = torch.empty(n_units, cfg.n_q_heads, cfg.window, device=dev)
    B.ckv_kept_mass(shape, params, batch["q"], k_out, indices, budgets, offsets, kept, ws)
    m = (1.0 - kept.double()).clamp_min(0.0)
    quality = {"mean_discarded_mass": float(m.mean()), "eps_tail": float((m ** 2).mean(-1).sqrt().mean()),
               "what": "attention mass of the window rows outside the retained set (Prop. 4.1), rank 0's units"}
    n_dec = max(1, min(4, 32 // (cfg.n_q_heads // cfg.n_kv_heads)))
    gq = torch.Generator(device=dev)
    gq.manual_seed(4242)
    q_dec = torch.randn(n_units, cfg.n_q_heads, n_dec, cfg.head_dim, generator=gq, device=dev).to(batch["q"].dtype)
    o_f = torch.empty(n_units, cfg.n_q_heads, n_dec, cfg.head_dim, device=dev)
    o_c = torch.empty_like(o_f)
    l_f = torch.empty(n_units, cfg.n_q_heads, n_dec, device=dev)
    l_c = torch.empty_like(l_f)
    B.ckv_attend(shape, params, q_dec, batch["k"], batch["v"], o_f, l_f, ws)
    B.ckv_attend(shape, params, q_dec, k_out, v_out, o_c, l_c, ws, budgets=budgets, offsets=offsets)
    quality["decode_check"] = {
        "queries_per_head": n_dec, "mean_discarded_mass": float((1.0 - torch.exp(l_c - l_f).double()).clamp_min(0).mean()),
        "mean_relative_output_error": float(((o_c - o_f).norm(dim=-1) / o_f.norm(dim=-1).clamp_min(1e-20)).mean()),
        "what": "random N(0,1) decode queries attending over the compressed cache against the full cache"}

    # ---- the oracle on the host cores, bounded sample (rank 0, single GPU only) ----------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # a first unit gives the oracle's pace; then as many units as fit in about 15 s of wall time
        host = {x: batch[x][:1].cpu() for x in ("q", "k", "v", "head_w")}
        host["sens"] = batch["sens"].cpu()
        sec1, cores = time_oracle(cfg, host, 1)
        sample = max(1, min(n_units, int(15.0 / max(sec1, 1e-3))))
        host = {x: batch[x][:sample].cpu() for x in ("q", "k", "v", "head_w")}
        host["sens"] = batch["sens"].cpu()
        sec, cores = time_oracle(cfg, host, sample)
        cpu_baseline = {"value": sample * L / sec, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"first {sample} of {n_units} units of {cfg.name}, whole pass, fp64, "
                                  f"{sec:.2f} s wall"}

    # ---- the other workloads the metric is quoted on: L = 131072 and the batch-16 serving batch ----------
    if world == 1 and not args.no_also:
        del wl, batch, kept, q_dec, o_f, o_c
        torch.cuda.empty_cache()
        for name in ("c4", "c3"):
            if name == cfg.name:
                continue
            other = gen.CONFIGS[name]
            need = 2.2 * other.n_units * other.n_kv_heads * other.seq_len * other.head_dim * 2 + 8e9
            free = torch.cuda.mem_get_info(dev)[0]
            if free < need:
                also[name] = {"skipped": f"needs {need / 1e9:.0f} GB of device memory, {free / 1e9:.0f} GB free"}
                continue
            also[name] = side_record(B, other, other.n_units, min(args.steps, 20), dev, sampler, sm_count)
    if sampler is not None:
        sampler.stop()

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if cfg.dtype == "bf16" else "f32",
                "data": "synthetic", "config": dict(config_dict(cfg, n_units, world), **({"value_norm": True} if args.value_norm else {})),
                "clocks": clocks, "e2e": e2e,
                "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu_baseline,
                "quality": quality, "also": also or None}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
