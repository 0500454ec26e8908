"""ctypes wrapper around the fp64 CPU oracle (``ckv_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
cpu-baseline leg may import this package.  It never touches the CUDA library.
All arrays are numpy arrays on the host; bf16 inputs travel as uint16 bit
patterns and are widened exactly to double inside the C code.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ckv_oracle.c")
_LIB = os.path.join(_HERE, "libckv_oracle.so")

BF16, F32 = 0, 1
POOL_NONE, POOL_MAX, POOL_AVG = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-Wall", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_units", "n_q_heads", "n_kv_heads", "head_dim", "seq_len", "window", "dtype")]


class _Params(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("pool_kind", "pool_size", "budget_per_head", "floor_per_head", "n_buckets",
                 "bucket_override", "head_w_per_unit", "sens_per_unit", "value_norm")] + \
               [("value_norm_eps", C.c_float), ("shared_elastic", C.c_int32), ("global_alpha", C.c_int32),
                ("units_per_prompt", C.c_int32), ("gate_layers", C.c_int32), ("ppl_bins", C.c_int32),
                ("budget_levels", C.c_int32), ("gate_coords", C.c_void_p)]


@dataclass
class Problem:
    """Shape and parameters of one call (the build's notation)."""
    n_units: int
    n_q_heads: int
    n_kv_heads: int
    seq_len: int
    window: int
    head_dim: int = 128
    dtype: int = BF16
    pool_kind: int = POOL_MAX
    pool_size: int = 7
    budget_per_head: int = 512
    floor_per_head: int = 1
    n_buckets: int = 16
    bucket_override: int = -1
    head_w_per_unit: bool = True
    sens_per_unit: bool = False
    value_norm: bool = False          # Eq. 4's value-norm ratio rho on (True) or off (the "u = alpha" ablation)
    value_norm_eps: float = 1e-6      # the eps of Alg. 1 (B)
    shared_elastic: bool = False      # the paper's own selection: one elastic set per unit (Eq. 6 over all heads, Eq. 8)
    global_alpha: bool = False        # Alg. 1 (A): alpha and the risk coordinate from the mean over the prompt's layers and heads
    units_per_prompt: int = 1         # layers per prompt (consecutive units) for global_alpha
    # The gate table as the paper indexes it (Sec. 4.3, Alg. 1 (D)): with gate_layers > 0 the table passed as `sens`
    # is [gate_layers, n_buckets, ppl_bins, budget_levels] and gate_coords [Nu,3] int32 gives each unit's
    # (layer row, perplexity bin, budget level).
    gate_layers: int = 0
    ppl_bins: int = 1
    budget_levels: int = 1
    gate_coords: object = None

    @property
    def n(self) -> int:
        return self.seq_len - self.window

    @property
    def rows_per_head(self) -> int:
        return min(self.budget_per_head, self.seq_len)

    def _shape(self) -> _Shape:
        return _Shape(self.n_units, self.n_q_heads, self.n_kv_heads, self.head_dim, self.seq_len,
                      self.window, self.dtype)

    def _params(self) -> _Params:
        coords = None
        if self.gate_layers > 0:
            # kept on the object so that the array outlives the C call
            self._coords = np.ascontiguousarray(self.gate_coords, np.int32).reshape(self.n_units, 3)
            coords = self._coords.ctypes.data_as(C.c_void_p)
        return _Params(self.pool_kind, self.pool_size, self.budget_per_head, self.floor_per_head,
                       self.n_buckets, self.bucket_override, int(self.head_w_per_unit),
                       int(self.sens_per_unit), int(self.value_norm), float(self.value_norm_eps),
                       int(self.shared_elastic), int(self.global_alpha), int(self.units_per_prompt),
                       int(self.gate_layers), int(self.ppl_bins), int(self.budget_levels), coords)


_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
    return _lib


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _inp(x, prob: Problem) -> np.ndarray:
    """Input tensor as a contiguous numpy array of the problem's dtype (bf16 as uint16)."""
    a = np.ascontiguousarray(x)
    want = np.uint16 if prob.dtype == BF16 else np.float32
    if a.dtype != want:
        raise TypeError(f"expected {want}, got {a.dtype}")
    return a


def _check(rc: int, what: str):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def window_attention(prob: Problem, q, k) -> np.ndarray:
    """A [Nu,H,W,L]: causal softmax rows of the window queries (O1, O2)."""
    q, k = _inp(q, prob), _inp(k, prob)
    A = np.empty((prob.n_units, prob.n_q_heads, prob.window, prob.seq_len), np.float64)
    s = prob._shape()
    _check(lib().oracle_window_attention(C.byref(s), _p(q), _p(k), _p(A)), "window_attention")
    return A


def colsum(prob: Problem, q, k) -> np.ndarray:
    """c_h[t] [Nu,H,L] (O3)."""
    q, k = _inp(q, prob), _inp(k, prob)
    c = np.empty((prob.n_units, prob.n_q_heads, prob.seq_len), np.float64)
    s = prob._shape()
    _check(lib().oracle_colsum(C.byref(s), _p(q), _p(k), _p(c)), "colsum")
    return c


def pool1d(kind: int, size: int, x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, np.float64)
    out = np.empty_like(x)
    _check(lib().oracle_pool1d(kind, size, x.shape[0], _p(x), _p(out)), "pool1d")
    return out


def vnorm(prob: Problem, v, eps: float | None = None) -> np.ndarray:
    """rho [Nu,Hkv,L] in fp64: value-row norms over their mean plus eps (O5b)."""
    v = _inp(v, prob)
    rho = np.empty((prob.n_units, prob.n_kv_heads, prob.seq_len), np.float64)
    s = prob._shape()
    fn = lib().oracle_vnorm
    fn.argtypes = [C.c_void_p, C.c_void_p, C.c_double, C.c_void_p]
    # the parameter block carries eps as fp32
    _check(fn(C.byref(s), _p(v), float(np.float32(prob.value_norm_eps)) if eps is None else float(eps), _p(rho)), "vnorm")
    return rho


def score(prob: Problem, q, k, head_w, want_csum: bool = False, v=None):
    """(scores [Nu,Hkv,n], colmass [Nu,L][, csum [Nu,H,L]]) in fp64 (O1-O6); with prob.value_norm the values
    `v` are needed for O5b."""
    q, k = _inp(q, prob), _inp(k, prob)
    head_w = np.ascontiguousarray(head_w, np.float32)
    rho = None
    if prob.value_norm:
        if v is None:
            raise ValueError("value_norm needs the values")
        rho = vnorm(prob, v)
    scores = np.empty((prob.n_units, prob.n_kv_heads, prob.n), np.float64)
    colmass = np.empty((prob.n_units, prob.seq_len), np.float64)
    csum = np.empty((prob.n_units, prob.n_q_heads, prob.seq_len), np.float64) if want_csum else None
    s, p = prob._shape(), prob._params()
    _check(lib().oracle_score(C.byref(s), C.byref(p), _p(q), _p(k), _p(head_w), _p(rho), _p(scores), _p(colmass),
                              _p(csum)), "score")
    return (scores, colmass, csum) if want_csum else (scores, colmass)


def allocate(n: int, f: int, P: int, demands) -> np.ndarray:
    """O8's integer split of P prefix rows over the heads (exposed for its pins)."""
    dem = np.ascontiguousarray(demands, np.int64)
    e = np.zeros_like(dem)
    fn = lib().oracle_allocate
    fn.argtypes = [C.c_int, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p]
    _check(fn(dem.shape[0], n, f, P, _p(dem), _p(e)), "allocate")
    return e


def budget(prob: Problem, scores, colmass, sens):
    """dict(budgets [Nu,Hkv], offsets [Nu,Hkv+1], bucket [Nu], entropy [Nu], tau [Nu], counts [Nu,Hkv]) (O7, O8)."""
    scores = np.ascontiguousarray(scores, np.float64)
    colmass = np.ascontiguousarray(colmass, np.float64)
    sens = np.ascontiguousarray(sens, np.float32)
    Nu, Hkv = prob.n_units, prob.n_kv_heads
    out = dict(budgets=np.zeros((Nu, Hkv), np.int32), offsets=np.zeros((Nu, Hkv + 1), np.int32),
               bucket=np.zeros(Nu, np.int32), entropy=np.zeros(Nu, np.float64), tau=np.zeros(Nu, np.float64),
               counts=np.zeros((Nu, Hkv), np.int32))
    s, p = prob._shape(), prob._params()
    _check(lib().oracle_budget(C.byref(s), C.byref(p), _p(scores), _p(colmass), _p(sens), _p(out["budgets"]),
                               _p(out["offsets"]), _p(out["bucket"]), _p(out["entropy"]), _p(out["tau"]),
                               _p(out["counts"])), "budget")
    return out


def select(prob: Problem, scores, budgets, offsets) -> np.ndarray:
    """indices [Nu, Hkv*B'] (O9)."""
    scores = np.ascontiguousarray(scores, np.float64)
    budgets = np.ascontiguousarray(budgets, np.int32)
    offsets = np.ascontiguousarray(offsets, np.int32)
    idx = np.full((prob.n_units, prob.n_kv_heads * prob.rows_per_head), -1, np.int32)
    s = prob._shape()
    _check(lib().oracle_select(C.byref(s), _p(scores), _p(budgets), _p(offsets), C.c_int64(idx.shape[1]), _p(idx)),
           "select")
    return idx


def gather(prob: Problem, k, v, indices, budgets, offsets):
    """(k_out, v_out) [Nu, Hkv*B', d] (O10)."""
    k, v = _inp(k, prob), _inp(v, prob)
    indices = np.ascontiguousarray(indices, np.int32)
    budgets = np.ascontiguousarray(budgets, np.int32)
    offsets = np.ascontiguousarray(offsets, np.int32)
    shape = (prob.n_units, prob.n_kv_heads * prob.rows_per_head, prob.head_dim)
    ko, vo = np.zeros(shape, k.dtype), np.zeros(shape, v.dtype)
    s = prob._shape()
    _check(lib().oracle_gather(C.byref(s), _p(k), _p(v), _p(indices), _p(budgets), _p(offsets),
                               C.c_int64(indices.shape[1]), _p(ko), _p(vo)), "gather")
    return ko, vo


def compress(prob: Problem, q, k, v, head_w, sens, want_scores: bool = True):
    """The whole pass (O1-O10); returns a dict of numpy arrays."""
    q, k, v = _inp(q, prob), _inp(k, prob), _inp(v, prob)
    head_w = np.ascontiguousarray(head_w, np.float32)
    sens = np.ascontiguousarray(sens, np.float32)
    Nu, Hkv = prob.n_units, prob.n_kv_heads
    rows = Hkv * prob.rows_per_head
    out = dict(k_out=np.zeros((Nu, rows, prob.head_dim), k.dtype), v_out=np.zeros((Nu, rows, prob.head_dim), v.dtype),
               indices=np.full((Nu, rows), -1, np.int32), budgets=np.zeros((Nu, Hkv), np.int32),
               offsets=np.zeros((Nu, Hkv + 1), np.int32), bucket=np.zeros(Nu, np.int32),
               entropy=np.zeros(Nu, np.float64),
               scores=np.empty((Nu, Hkv, prob.n), np.float64) if want_scores else None)
    s, p = prob._shape(), prob._params()
    _check(lib().oracle_compress(C.byref(s), C.byref(p), _p(q), _p(k), _p(v), _p(head_w), _p(sens), _p(out["k_out"]),
                                 _p(out["v_out"]), _p(out["indices"]), _p(out["budgets"]), _p(out["offsets"]),
                                 _p(out["bucket"]), _p(out["entropy"]), _p(out["scores"])), "compress")
    return out


def kept_mass(prob: Problem, q, k, indices, budgets, offsets) -> np.ndarray:
    """kept[u,h,i]: attention mass of window row i that lies on the retained set (Prop. 4.1's 1 - m)."""
    q, k = _inp(q, prob), _inp(k, prob)
    kept = np.empty((prob.n_units, prob.n_q_heads, prob.window), np.float64)
    s = prob._shape()
    indices = np.ascontiguousarray(indices, np.int32)
    _check(lib().oracle_kept_mass(C.byref(s), _p(q), _p(k), _p(indices), _p(np.ascontiguousarray(budgets, np.int32)),
                                  _p(np.ascontiguousarray(offsets, np.int32)), C.c_int64(indices.shape[1]),
                                  _p(kept)), "kept_mass")
    return kept


def attend(prob: Problem, q_dec, k, v, budgets=None, offsets=None):
    """(out [Nu,H,n_dec,d], lse [Nu,H,n_dec]) in fp64: attention of decode queries q_dec [Nu,H,n_dec,d] over all
    L rows of k, v, or -- when budgets and offsets are given -- over the gathered rows k_out, v_out [Nu, rows, d]."""
    q_dec, k, v = _inp(q_dec, prob), _inp(k, prob), _inp(v, prob)
    n_dec = q_dec.shape[2]
    out = np.empty(q_dec.shape, np.float64)
    lse = np.empty(q_dec.shape[:3], np.float64)
    compressed = budgets is not None
    if compressed:
        budgets = np.ascontiguousarray(budgets, np.int32)
        offsets = np.ascontiguousarray(offsets, np.int32)
    s = prob._shape()
    _check(lib().oracle_attend(C.byref(s), _p(q_dec), C.c_int(n_dec), _p(k), _p(v), C.c_int(int(compressed)),
                               _p(budgets), _p(offsets), C.c_int64(k.shape[1] if compressed else 0), _p(out), _p(lse)),
           "attend")
    return out, lse


def depth_map(table, n_dst: int) -> np.ndarray:
    """A table [n_src, ...] compiled for n_src layers, mapped to n_dst layers by relative depth (fp32)."""
    src = np.ascontiguousarray(table, np.float32)
    n_src = src.shape[0]
    row = int(np.prod(src.shape[1:])) if src.ndim > 1 else 1
    dst = np.empty((n_dst,) + src.shape[1:], np.float32)
    _check(lib().oracle_depth_map(_p(src), C.c_int(n_src), C.c_int(n_dst), C.c_int64(row), _p(dst)), "depth_map")
    return dst


def num_threads() -> int:
    return int(lib().oracle_num_threads())
