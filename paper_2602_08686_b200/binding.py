"""Thin ctypes binding over the C ABI of ``libckv.so`` (see ``include/ckv.h``).

Argument marshalling only: every step of the retention pass runs in the library's CUDA kernels.
Functions carry the names of the C entry points and take torch CUDA tensors (device memory and
streams are PyTorch's).  There is no fallback: a missing library or a non-zero status raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libckv.so")

BF16, F32 = 0, 1
POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2
OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(6)


class CkvError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class ckv_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_units", "n_q_heads", "n_kv_heads", "head_dim", "seq_len", "window",
                                         "dtype", "reserved_")] + \
               [(n, C.c_int64) for n in ("q_stride_unit", "q_stride_head", "q_stride_row",
                                         "kv_stride_unit", "kv_stride_head", "kv_stride_tok")]


class ckv_tuning(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("score_path", "run_tiles", "l2_hints", "group_fuse", "pdl", "reserved_")] + \
               [("scan_start_event", C.c_void_p), ("scan_stop_event", C.c_void_p)]


def make_tuning(score_path: int = -1, run_tiles: int = -1, l2_hints: int = -1, group_fuse: int = -1, pdl: int = -1,
                scan_events=None) -> ckv_tuning:
    """Per-call scheduling settings (-1: the process-wide default); scan_events is a pair of torch.cuda.Event objects
    (timing enabled, recorded once before) to be recorded around the tensor-core scan of the calls that carry it."""
    ev0 = ev1 = None
    if scan_events is not None:
        ev0, ev1 = (C.c_void_p(e.cuda_event) for e in scan_events)
    t = ckv_tuning(score_path, run_tiles, l2_hints, group_fuse, pdl, 0, ev0, ev1)
    t._keep = scan_events
    return t


class ckv_params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("pool_kind", "pool_size", "budget_per_head", "floor_per_head",
                                         "n_buckets", "bucket_override")] + \
               [(n, C.c_int64) for n in ("head_w_stride_unit", "sens_stride_unit")] + \
               [("value_norm", C.c_int32), ("value_norm_eps", C.c_float), ("shared_elastic", C.c_int32),
                ("global_alpha", C.c_int32), ("units_per_prompt", C.c_int32), ("reserved_", C.c_int32),
                ("n_gate_layers", C.c_int32), ("n_ppl_bins", C.c_int32), ("n_budget_levels", C.c_int32),
                ("reserved2_", C.c_int32), ("gate_coords", C.c_void_p), ("tuning", C.POINTER(ckv_tuning))]


_lib = None


def lib() -> C.CDLL:
    """Loads libckv.so; raises if it has not been built (``python -m paper_2602_08686_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_08686_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, sz, i32p, fp = C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p
        shp, prm = C.POINTER(ckv_shape), C.POINTER(ckv_params)
        L.ckv_workspace_bytes.restype = sz
        L.ckv_workspace_bytes.argtypes = [shp, prm]
        L.ckv_score_workspace_bytes.restype = sz
        L.ckv_score_workspace_bytes.argtypes = [shp, prm]
        L.ckv_staging_bytes.restype = sz
        L.ckv_staging_bytes.argtypes = [shp, prm]
        L.ckv_score.argtypes = [shp, prm, vp, vp, fp, fp, fp, vp, sz, vp]
        L.ckv_score_noalloc.argtypes = [shp, prm, vp, vp, fp, fp, fp, vp]
        L.ckv_budget.argtypes = [shp, prm, fp, fp, fp, i32p, i32p, i32p, fp, vp, sz, vp]
        L.ckv_select.argtypes = [shp, prm, fp, i32p, i32p, i32p, vp, sz, vp]
        L.ckv_vnorm.argtypes = [shp, prm, vp, fp, fp, vp, sz, vp]
        L.ckv_unit_max.argtypes = [shp, prm, fp, vp]
        L.ckv_attend.argtypes = [shp, prm, vp, C.c_int32, vp, vp, C.c_int32, i32p, i32p, fp, fp, vp, sz, vp]
        L.ckv_kept_mass.argtypes = [shp, prm, vp, vp, i32p, i32p, i32p, fp, vp, sz, vp]
        L.ckv_prompt_mass.argtypes = [shp, prm, fp, fp, vp]
        L.ckv_global_scores.argtypes = [shp, prm, fp, fp, C.c_int32, fp, fp, vp]
        L.ckv_gather.argtypes = [shp, prm, vp, vp, i32p, i32p, vp, vp, vp]
        L.ckv_compress.argtypes = [shp, prm, vp, vp, vp, fp, fp, vp, vp, i32p, i32p, i32p, fp, i32p, fp, vp, sz, vp]
        L.ckv_compress_host.argtypes = [shp, prm, vp, vp, vp, fp, fp, vp, vp, i32p, i32p, i32p, vp, sz, vp, sz, vp]
        L.ckv_device_status.argtypes = [vp, vp]
        L.ckv_gate_depth_map_host.argtypes = [fp, C.c_int, C.c_int, C.c_int64, fp]
        L.ckv_set_scan_events.argtypes = [vp, vp]
        L.ckv_set_scan_events.restype = None
        L.ckv_set_tunable.argtypes = [C.c_char_p, C.c_int]
        L.ckv_set_tunable.restype = C.c_int
        L.ckv_kernel_launches.restype = C.c_int64
        L.ckv_status_string.restype = C.c_char_p
        L.ckv_status_string.argtypes = [C.c_int]
        L.ckv_allocate_rows_host.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64, vp, vp]
        for name in ("ckv_score", "ckv_score_noalloc", "ckv_budget", "ckv_select", "ckv_vnorm", "ckv_unit_max", "ckv_kept_mass", "ckv_attend", "ckv_prompt_mass", "ckv_global_scores", "ckv_gather", "ckv_compress", "ckv_compress_host",
                     "ckv_device_status", "ckv_version", "ckv_allocate_rows_host"):
            getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().ckv_status_string(status).decode()


def ckv_version() -> int:
    return lib().ckv_version()


def ckv_set_score_path(path: int) -> int:
    """0 automatic, 1 plain kernels, 2 tensor-core kernel required; returns the previous setting."""
    return int(lib().ckv_set_score_path(int(path)))


def ckv_set_scan_events(start, stop) -> None:
    """Timing hook: torch.cuda.Event objects (timing enabled, already recorded once so that their handles
    exist) recorded around the tensor-core scan of every later call; ``None, None`` switches it off."""
    h0 = None if start is None else C.c_void_p(start.cuda_event)
    h1 = None if stop is None else C.c_void_p(stop.cuda_event)
    lib().ckv_set_scan_events(h0, h1)


def ckv_set_tunable(name: str, value: int) -> int:
    """Schedule knob of the tensor-core scan ("run_tiles", "l2_hints"); returns the previous value."""
    prev = int(lib().ckv_set_tunable(name.encode(), int(value)))
    if prev < 0:
        raise ValueError(f"unknown tunable or value out of range: {name}={value}")
    return prev


def ckv_kernel_launches() -> int:
    return int(lib().ckv_kernel_launches())


@dataclass
class Params:
    pool_kind: int = POOL_MAX
    pool_size: int = 7
    budget_per_head: int = 512
    floor_per_head: int = 1
    n_buckets: int = 16
    bucket_override: int = -1
    value_norm: bool = False
    value_norm_eps: float = 1e-6
    shared_elastic: bool = False
    global_alpha: bool = False
    units_per_prompt: int = 1
    # the four-axis gate table T_gate[layer, entropy bin, perplexity bin, budget level] (used when make_params is
    # given gate_coords); n_buckets is then the number of entropy bins
    n_gate_layers: int = 0
    n_ppl_bins: int = 1
    n_budget_levels: int = 1


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def make_shape(q: torch.Tensor, k: torch.Tensor) -> ckv_shape:
    """Shape struct from q_win [Nu,H,W,d] and k [Nu,Hkv,L,d] (last dimension contiguous)."""
    if q.dim() != 4 or k.dim() != 4 or q.stride(3) != 1 or k.stride(3) != 1:
        raise ValueError("q_win and k must be 4-D with a contiguous last dimension")
    Nu, H, W, d = q.shape
    _, Hkv, L, _ = k.shape
    return ckv_shape(Nu, H, Hkv, d, L, W, _dtype_code(k), 0, q.stride(0), q.stride(1), q.stride(2),
                     k.stride(0), k.stride(1), k.stride(2))


def make_params(p: Params, head_w: torch.Tensor | None, sens: torch.Tensor | None, H: int = 0,
                gate_coords: torch.Tensor | None = None, tuning: ckv_tuning | None = None) -> ckv_params:
    """Parameter struct.  With gate_coords ([Nu,3] int32: layer row, perplexity bin, budget level per unit; on the
    device, or on the host for ckv_compress_host) `sens` is the dense table [n_gate_layers, n_buckets, n_ppl_bins,
    n_budget_levels]; the struct keeps a reference to the tensor."""
    hw_stride = 0 if head_w is None or head_w.dim() == 1 else head_w.stride(0)
    se_stride = 0 if sens is None or sens.dim() == 1 or gate_coords is not None else sens.stride(0)
    if gate_coords is not None:
        if gate_coords.dtype != torch.int32 or not gate_coords.is_contiguous() or gate_coords.shape[-1] != 3:
            raise ValueError("gate_coords must be a contiguous int32 tensor [Nu, 3]")
        if sens is not None and (not sens.is_contiguous() or sens.numel() != p.n_gate_layers * p.n_buckets *
                                 p.n_ppl_bins * p.n_budget_levels):
            raise ValueError("the gate table must be dense [n_gate_layers, n_buckets, n_ppl_bins, n_budget_levels]")
    out = ckv_params(p.pool_kind, p.pool_size, p.budget_per_head, p.floor_per_head, p.n_buckets,
                     p.bucket_override, hw_stride, se_stride, int(p.value_norm), float(p.value_norm_eps),
                     int(p.shared_elastic), int(p.global_alpha), int(p.units_per_prompt), 0,
                     int(p.n_gate_layers) if gate_coords is not None else 0, int(p.n_ppl_bins),
                     int(p.n_budget_levels), 0, None if gate_coords is None else gate_coords.data_ptr(),
                     None if tuning is None else C.pointer(tuning))
    out._keep = (gate_coords, tuning)
    return out


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check_kv(shape: ckv_shape, t: torch.Tensor, name: str) -> None:
    """k and v share one set of strides in ckv_shape: a tensor laid out differently would be read wrongly."""
    want_shape = (shape.n_units, shape.n_kv_heads, shape.seq_len, shape.head_dim)
    if tuple(t.shape) != want_shape or _dtype_code(t) != shape.dtype or t.stride(3) != 1:
        raise ValueError(f"{name} must be {want_shape} in the dtype of the shape struct, last dimension contiguous")
    for dim, want in enumerate((shape.kv_stride_unit, shape.kv_stride_head, shape.kv_stride_tok)):
        if t.shape[dim] > 1 and t.stride(dim) != want:
            raise ValueError(f"{name} has stride {t.stride(dim)} in dimension {dim}; the shape struct says {want} "
                             "(k and v must be laid out alike)")


def _check_dense(t: torch.Tensor, name: str) -> None:
    if not t.is_contiguous():
        raise ValueError(f"{name} must be dense")


def _check(status: int, what: str):
    if status != OK:
        raise CkvError(status, what)


def ckv_workspace_bytes(shape: ckv_shape, params: ckv_params) -> int:
    return int(lib().ckv_workspace_bytes(C.byref(shape), C.byref(params)))


def ckv_score_workspace_bytes(shape: ckv_shape, params: ckv_params) -> int:
    return int(lib().ckv_score_workspace_bytes(C.byref(shape), C.byref(params)))


def ckv_reads_in_place(host_tensor: torch.Tensor) -> bool:
    """True if ckv_compress_host would read this host tensor in place (page-locked and mapped) instead of copying it."""
    lib().ckv_reads_in_place.argtypes = [C.c_void_p]
    return bool(lib().ckv_reads_in_place(_ptr(host_tensor)))


def ckv_staging_bytes(shape: ckv_shape, params: ckv_params) -> int:
    return int(lib().ckv_staging_bytes(C.byref(shape), C.byref(params)))


def alloc_workspace(shape: ckv_shape, params: ckv_params, device) -> torch.Tensor:
    nbytes = ckv_workspace_bytes(shape, params)
    if nbytes == 0:
        raise CkvError(ERR_INVALID_ARG, "ckv_workspace_bytes")
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def rows_per_unit(shape: ckv_shape, params: ckv_params) -> int:
    return shape.n_kv_heads * min(params.budget_per_head, shape.seq_len)


def ckv_score(shape, params, q_win, k, head_w, scores, colmass, ws, stream=None):
    _check(lib().ckv_score(C.byref(shape), C.byref(params), _ptr(q_win), _ptr(k), _ptr(head_w), _ptr(scores),
                           _ptr(colmass), _ptr(ws), ws.numel(), _stream(stream)), "ckv_score")


NOALLOC_SCRATCH_BYTES = 16 << 20


def ckv_score_noalloc(shape, params, q_win, k, head_w, scores, colmass, stream=None):
    """ckv_score on the library's own fixed scratch (no work space, nothing allocated); problems that need
    more than NOALLOC_SCRATCH_BYTES raise CkvError with ERR_WORKSPACE.  Calls on one device must not overlap."""
    _check(lib().ckv_score_noalloc(C.byref(shape), C.byref(params), _ptr(q_win), _ptr(k), _ptr(head_w),
                                   _ptr(scores), _ptr(colmass), _stream(stream)), "ckv_score_noalloc")


def ckv_budget(shape, params, scores, colmass, sens, budgets, offsets, bucket, entropy, ws, stream=None):
    _check(lib().ckv_budget(C.byref(shape), C.byref(params), _ptr(scores), _ptr(colmass), _ptr(sens), _ptr(budgets),
                            _ptr(offsets), _ptr(bucket), _ptr(entropy), _ptr(ws), ws.numel(), _stream(stream)),
           "ckv_budget")


def ckv_vnorm(shape, params, v, rho, scores, ws, stream=None):
    _check_kv(shape, v, "v")
    _check(lib().ckv_vnorm(C.byref(shape), C.byref(params), _ptr(v), _ptr(rho), _ptr(scores), _ptr(ws), ws.numel(),
                           _stream(stream)), "ckv_vnorm")


def ckv_prompt_mass(shape, params, colmass, pmass, stream=None):
    _check(lib().ckv_prompt_mass(C.byref(shape), C.byref(params), _ptr(colmass), _ptr(pmass), _stream(stream)),
           "ckv_prompt_mass")


def ckv_global_scores(shape, params, head_w, pmass, units_total, scores, colmass, stream=None):
    _check(lib().ckv_global_scores(C.byref(shape), C.byref(params), _ptr(head_w), _ptr(pmass), int(units_total),
                                   _ptr(scores), _ptr(colmass), _stream(stream)), "ckv_global_scores")


def ckv_kept_mass(shape, params, q_win, k_out, indices, budgets, offsets, kept, ws, stream=None):
    _check(lib().ckv_kept_mass(C.byref(shape), C.byref(params), _ptr(q_win), _ptr(k_out), _ptr(indices), _ptr(budgets),
                               _ptr(offsets), _ptr(kept), _ptr(ws), ws.numel(), _stream(stream)), "ckv_kept_mass")


def ckv_attend(shape, params, q_dec, k, v, out, lse, ws, budgets=None, offsets=None, stream=None):
    """Attention of the decode queries q_dec [Nu,H,n_dec,d] over all rows of k, v, or over the gathered rows when
    budgets and offsets are given."""
    compressed = budgets is not None
    _check_dense(q_dec, "q_dec")
    if not compressed:
        _check_kv(shape, k, "k"), _check_kv(shape, v, "v")
    else:
        _check_dense(k, "k_out"), _check_dense(v, "v_out")
    _check(lib().ckv_attend(C.byref(shape), C.byref(params), _ptr(q_dec), int(q_dec.shape[2]), _ptr(k), _ptr(v),
                            int(compressed), _ptr(budgets), _ptr(offsets), _ptr(out), _ptr(lse), _ptr(ws), ws.numel(),
                            _stream(stream)), "ckv_attend")


def ckv_unit_max(shape, params, scores, stream=None):
    _check(lib().ckv_unit_max(C.byref(shape), C.byref(params), _ptr(scores), _stream(stream)), "ckv_unit_max")


def ckv_select(shape, params, scores, budgets, offsets, indices, ws, stream=None):
    _check(lib().ckv_select(C.byref(shape), C.byref(params), _ptr(scores), _ptr(budgets), _ptr(offsets),
                            _ptr(indices), _ptr(ws), ws.numel(), _stream(stream)), "ckv_select")


def ckv_gather(shape, params, k, v, indices, offsets, k_out, v_out, stream=None):
    _check_kv(shape, k, "k"), _check_kv(shape, v, "v")
    _check_dense(k_out, "k_out"), _check_dense(v_out, "v_out")
    _check(lib().ckv_gather(C.byref(shape), C.byref(params), _ptr(k), _ptr(v), _ptr(indices), _ptr(offsets),
                            _ptr(k_out), _ptr(v_out), _stream(stream)), "ckv_gather")


def ckv_compress(shape, params, q_win, k, v, head_w, sens, k_out, v_out, indices, budgets, offsets, ws,
                 scores=None, bucket=None, entropy=None, stream=None):
    _check_kv(shape, k, "k"), _check_kv(shape, v, "v")
    _check_dense(k_out, "k_out"), _check_dense(v_out, "v_out")
    _check(lib().ckv_compress(C.byref(shape), C.byref(params), _ptr(q_win), _ptr(k), _ptr(v), _ptr(head_w),
                              _ptr(sens), _ptr(k_out), _ptr(v_out), _ptr(indices), _ptr(budgets), _ptr(offsets),
                              _ptr(scores), _ptr(bucket), _ptr(entropy), _ptr(ws), ws.numel(), _stream(stream)),
           "ckv_compress")


def ckv_compress_host(shape, params, q_win, k, v, head_w, sens, k_out, v_out, indices, budgets, offsets,
                      staging, ws, stream=None):
    """All tensor arguments except ``staging`` and ``ws`` are HOST tensors (pinned memory recommended)."""
    _check(lib().ckv_compress_host(C.byref(shape), C.byref(params), _ptr(q_win), _ptr(k), _ptr(v), _ptr(head_w),
                                   _ptr(sens), _ptr(k_out), _ptr(v_out), _ptr(indices), _ptr(budgets),
                                   _ptr(offsets), _ptr(staging), staging.numel(), _ptr(ws), ws.numel(),
                                   _stream(stream)), "ckv_compress_host")


def ckv_device_status(ws=None, stream=None) -> int:
    """What device code recorded in the work space's status word since the last such call (reading clears it);
    ``ws=None`` reads the fixed scratch of ckv_score_noalloc on the current device."""
    return int(lib().ckv_device_status(_ptr(ws), _stream(stream)))


def ckv_gate_depth_map_host(table: torch.Tensor, n_dst: int) -> torch.Tensor:
    """A host table [n_src, ...] (fp32) compiled for n_src layers, mapped to n_dst layers by relative depth."""
    src = table.detach().cpu().contiguous().float()
    n_src = src.shape[0]
    row = src[0].numel() if src.dim() > 1 else 1
    dst = torch.empty((n_dst,) + tuple(src.shape[1:]), dtype=torch.float32)
    if lib().ckv_gate_depth_map_host(_ptr(src), n_src, int(n_dst), row, _ptr(dst)) != 0:
        raise ValueError("ckv_gate_depth_map_host: invalid arguments")
    return dst


def ckv_allocate_rows_host(n: int, f: int, P: int, demands) -> list[int]:
    """Host-side run of the integer budget split used by ckv_budget (no GPU needed)."""
    hkv = len(demands)
    dem = (C.c_int64 * hkv)(*[int(x) for x in demands])
    out = (C.c_int64 * hkv)()
    rc = lib().ckv_allocate_rows_host(hkv, n, f, P, dem, out)
    if rc:
        raise ValueError(f"ckv_allocate_rows_host failed with {rc}")
    return list(out)


# ------------------------------------------------------------------------------------ convenience
def compress(q_win, k, v, head_w, sens, p: Params, want_scores: bool = False, ws=None, stream=None,
             gate_coords=None, tuning=None):
    """Allocates the outputs and the work space with torch and runs ckv_compress."""
    shape = make_shape(q_win, k)
    params = make_params(p, head_w, sens, gate_coords=gate_coords, tuning=tuning)
    dev = k.device
    Nu, Hkv = shape.n_units, shape.n_kv_heads
    rows = rows_per_unit(shape, params)
    out = dict(
        k_out=torch.empty(Nu, rows, shape.head_dim, dtype=k.dtype, device=dev),
        v_out=torch.empty(Nu, rows, shape.head_dim, dtype=v.dtype, device=dev),
        indices=torch.empty(Nu, rows, dtype=torch.int32, device=dev),
        budgets=torch.empty(Nu, Hkv, dtype=torch.int32, device=dev),
        offsets=torch.empty(Nu, Hkv + 1, dtype=torch.int32, device=dev),
        bucket=torch.empty(Nu, dtype=torch.int32, device=dev),
        entropy=torch.empty(Nu, dtype=torch.float32, device=dev),
        scores=torch.empty(Nu, Hkv, shape.seq_len - shape.window, dtype=torch.float32, device=dev)
        if want_scores else None,
    )
    ws = alloc_workspace(shape, params, dev) if ws is None else ws
    ckv_compress(shape, params, q_win, k, v, head_w, sens, out["k_out"], out["v_out"], out["indices"],
                 out["budgets"], out["offsets"], ws, scores=out["scores"], bucket=out["bucket"],
                 entropy=out["entropy"], stream=stream)
    out["ws"] = ws
    return out
