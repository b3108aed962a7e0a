"""ctypes front end of the rTop-k CPU oracle (test infrastructure only).

The oracle restates Algorithm 1 (node body and master average) and
Definitions 1-3 of the rTop-k paper as plain CPU code; see the header of
``rtopk_oracle.cpp`` for the readings it fixes.  Only tests, the smoke check
and the benchmark's CPU-baseline leg import this package; the CUDA library
never does.

All array arguments are C-contiguous numpy arrays; bfloat16 gradients are
passed as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import sys

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rtopk_oracle.cpp")
_LIB = os.path.join(_HERE, "librtopk_oracle.so")

GRAD_F32, GRAD_BF16 = 0, 1
SCALE_MEAN, SCALE_SUM, SCALE_UNBIASED, SCALE_COUNT = 0, 1, 2, 3

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler (no fast-math, no contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread", "-ffp-contract=off",
               "-fno-fast-math", "-Wall", "-Wextra", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        u32p, f32p, f64p, i64p = (C.POINTER(C.c_uint32), C.POINTER(C.c_float),
                                  C.POINTER(C.c_double), C.POINTER(C.c_int64))
        u16p = C.POINTER(C.c_uint16)
        L.oracle_set_threads.argtypes = [C.c_int]
        L.oracle_get_threads.restype = C.c_int
        L.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.oracle_scale_draw.argtypes = [C.c_uint64, C.c_uint32]
        L.oracle_scale_draw.restype = C.c_uint32
        L.oracle_draw.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32]
        L.oracle_draw.restype = C.c_uint32
        L.oracle_floyd_from_draws.argtypes = [C.c_int64, C.c_int64, u32p, u32p]
        L.oracle_sample_positions.argtypes = [C.c_int64, C.c_int64, C.c_uint64, C.c_uint32,
                                              C.c_uint32, C.c_uint32, u32p]
        L.oracle_top_r.argtypes = [f32p, C.c_int64, C.c_int64, u32p]
        L.oracle_sparsify.argtypes = [C.c_void_p, C.c_int, C.c_int64, f32p, C.c_int64, C.c_int64,
                                      C.c_int32, C.c_int32, C.c_int64, C.c_int64, C.c_uint64,
                                      C.c_uint32, u32p, f32p]
        L.oracle_sparsify_segmented.argtypes = [C.c_void_p, C.c_int, C.c_int64, f32p, C.c_int64,
                                                C.c_int64, C.c_int32, C.c_int32, C.c_int32, i64p,
                                                i64p, i64p, C.c_uint64, C.c_uint32, u32p, f32p]
        L.oracle_aggregate.argtypes = [u32p, f32p, C.c_int64, C.c_int32, C.c_int64, C.c_int,
                                       f64p, f32p]
        L.oracle_aggregate_scaled.argtypes = [u32p, f32p, C.c_int64, C.c_int32, C.c_int64, C.c_int,
                                              C.c_int64, f64p, f32p]
        L.oracle_apply_update.argtypes = [u32p, f32p, C.c_int64, C.c_int32, C.c_int64, C.c_int,
                                          C.c_int64, C.c_float, f32p]
        L.oracle_apply_momentum.argtypes = [u32p, f32p, C.c_int64, C.c_int32, C.c_int64, C.c_int, C.c_int64,
                                            C.c_float, C.c_float, f32p, f32p]
        L.oracle_tiled_spans.argtypes = [C.c_int64]
        L.oracle_tiled_spans.restype = C.c_int64
        L.oracle_encode_tiled_row.argtypes = [u32p, f32p, C.c_int64, C.c_int64, u32p, u16p, u16p, f32p]
        L.oracle_decode_tiled_row.argtypes = [u32p, u16p, u16p, C.c_int64, C.c_int64, u32p, f32p]
        L.oracle_warmup_sizes.argtypes = [C.c_int64, C.c_int32, C.c_double, C.c_double, C.c_int64, C.c_int64,
                                          i64p, i64p]
        L.oracle_index_bits.argtypes = [C.c_int64]
        L.oracle_bf16_rne.argtypes = [C.c_float]
        L.oracle_bf16_rne.restype = C.c_uint16
        L.oracle_encode_row.argtypes = [u32p, f32p, C.c_int64, C.c_int64, u32p, u16p, f32p]
        L.oracle_decode_row.argtypes = [u32p, u16p, C.c_int64, C.c_int64, u32p, f32p]
        L.oracle_sparsify_threshold.argtypes = [C.c_void_p, C.c_int, C.c_int64, f32p, C.c_int64, C.c_int64,
                                                C.c_int32, C.c_int32, C.c_float, C.c_int64, C.c_uint64,
                                                C.c_uint32, C.c_int, u32p, f32p, u32p, u32p]
        L.oracle_aggregate_threshold.argtypes = [u32p, f32p, u32p, u32p, C.c_int64, C.c_int32, C.c_int64,
                                                 f64p, f32p]
        _lib = L
    return _lib


def _p(a: np.ndarray, ty):
    return a.ctypes.data_as(C.POINTER(ty))


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"oracle: {what} rejected its arguments (code {rc})")


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    assert c.shape == (4,) and k.shape == (2,)
    out = np.zeros(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_p(c, C.c_uint32), _p(k, C.c_uint32), _p(out, C.c_uint32))
    return out


def scale_draw(u: int, n: int) -> int:
    return int(lib().oracle_scale_draw(int(u), int(n)))


def draw(seed: int, step: int, worker: int, segment: int, j: int) -> int:
    return int(lib().oracle_draw(int(seed), int(step), int(worker), int(segment), int(j)))


def floyd_from_draws(r: int, k: int, t) -> np.ndarray:
    t = np.ascontiguousarray(t, dtype=np.uint32)
    assert t.shape == (k,)
    pos = np.zeros(k, dtype=np.uint32)
    _check(lib().oracle_floyd_from_draws(r, k, _p(t, C.c_uint32), _p(pos, C.c_uint32)), "floyd")
    return pos


def sample_positions(r: int, k: int, seed: int, step: int, worker: int, segment: int = 0) -> np.ndarray:
    pos = np.zeros(k, dtype=np.uint32)
    _check(lib().oracle_sample_positions(r, k, seed, step, worker, segment, _p(pos, C.c_uint32)),
           "sample_positions")
    return pos


def top_r(a: np.ndarray, r: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    L = np.zeros(r, dtype=np.uint32)
    _check(lib().oracle_top_r(_p(a, C.c_float), a.shape[0], r, _p(L, C.c_uint32)), "top_r")
    return L


def _grad_args(grad: np.ndarray):
    assert grad.ndim == 2 and grad.flags.c_contiguous
    if grad.dtype == np.float32:
        return GRAD_F32
    if grad.dtype == np.uint16:
        return GRAD_BF16
    raise TypeError("grad must be float32 or uint16 (bfloat16 bits)")


def sparsify(grad: np.ndarray, residual: np.ndarray, d: int, r: int, k: int, seed: int, step: int,
             worker_base: int = 0):
    """Algorithm 1 node body on W rows; ``residual`` (float32, W x ld_m) is updated in place.
    Returns (msg_idx [W,k] uint32, msg_val [W,k] float32)."""
    dt = _grad_args(grad)
    assert residual.dtype == np.float32 and residual.ndim == 2 and residual.flags.c_contiguous
    W = grad.shape[0]
    assert residual.shape[0] == W
    idx = np.zeros((W, k), dtype=np.uint32)
    val = np.zeros((W, k), dtype=np.float32)
    _check(lib().oracle_sparsify(grad.ctypes.data, dt, grad.shape[1], _p(residual, C.c_float),
                                 residual.shape[1], d, W, worker_base, r, k, seed, step,
                                 _p(idx, C.c_uint32), _p(val, C.c_float)), "sparsify")
    return idx, val


def sparsify_segmented(grad: np.ndarray, residual: np.ndarray, d: int, seg_off, seg_r, seg_k,
                       seed: int, step: int, worker_base: int = 0):
    dt = _grad_args(grad)
    assert residual.dtype == np.float32 and residual.ndim == 2 and residual.flags.c_contiguous
    W = grad.shape[0]
    off = np.ascontiguousarray(seg_off, dtype=np.int64)
    rr = np.ascontiguousarray(seg_r, dtype=np.int64)
    kk = np.ascontiguousarray(seg_k, dtype=np.int64)
    S = rr.shape[0]
    assert off.shape == (S + 1,) and kk.shape == (S,)
    K = int(kk.sum())
    idx = np.zeros((W, K), dtype=np.uint32)
    val = np.zeros((W, K), dtype=np.float32)
    _check(lib().oracle_sparsify_segmented(grad.ctypes.data, dt, grad.shape[1],
                                           _p(residual, C.c_float), residual.shape[1], d, W,
                                           worker_base, S, _p(off, C.c_int64), _p(rr, C.c_int64),
                                           _p(kk, C.c_int64), seed, step, _p(idx, C.c_uint32),
                                           _p(val, C.c_float)), "sparsify_segmented")
    return idx, val


def aggregate(msg_idx: np.ndarray, msg_val: np.ndarray, d: int, scale_mode: int = SCALE_MEAN, r: int = 0):
    """Algorithm 1 master average (``r`` only for SCALE_UNBIASED).
    Returns (out64 float64 [d], out32 float32 [d])."""
    idx = np.ascontiguousarray(msg_idx, dtype=np.uint32)
    val = np.ascontiguousarray(msg_val, dtype=np.float32)
    W, k = idx.shape
    o64 = np.zeros(d, dtype=np.float64)
    o32 = np.zeros(d, dtype=np.float32)
    _check(lib().oracle_aggregate_scaled(_p(idx, C.c_uint32), _p(val, C.c_float), d, W, k, scale_mode, r,
                                         _p(o64, C.c_double), _p(o32, C.c_float)), "aggregate")
    return o64, o32


def apply_update(msg_idx: np.ndarray, msg_val: np.ndarray, d: int, eta: float, weights: np.ndarray,
                 scale_mode: int = SCALE_MEAN, r: int = 0) -> np.ndarray:
    """Algorithm 1 master update w - eta * ghat on a copy of `weights` (float32 [d])."""
    idx = np.ascontiguousarray(msg_idx, dtype=np.uint32)
    val = np.ascontiguousarray(msg_val, dtype=np.float32)
    W, k = idx.shape
    w = np.array(weights, dtype=np.float32, copy=True)
    _check(lib().oracle_apply_update(_p(idx, C.c_uint32), _p(val, C.c_float), d, W, k, scale_mode, r,
                                     C.c_float(eta), _p(w, C.c_float)), "apply_update")
    return w


def apply_momentum(msg_idx: np.ndarray, msg_val: np.ndarray, d: int, eta: float, mu: float, velocity: np.ndarray,
                   weights: np.ndarray, scale_mode: int = SCALE_MEAN, r: int = 0):
    """Heavy-ball master update v <- mu v + ghat, w <- w - eta v on copies of `velocity` and `weights`
    (float32 [d]); returns (velocity, weights)."""
    idx = np.ascontiguousarray(msg_idx, dtype=np.uint32)
    val = np.ascontiguousarray(msg_val, dtype=np.float32)
    W, k = idx.shape
    v = np.array(velocity, dtype=np.float32, copy=True)
    w = np.array(weights, dtype=np.float32, copy=True)
    _check(lib().oracle_apply_momentum(_p(idx, C.c_uint32), _p(val, C.c_float), d, W, k, scale_mode, r,
                                       C.c_float(eta), C.c_float(mu), _p(v, C.c_float), _p(w, C.c_float)),
           "apply_momentum")
    return v, w


def warmup_sizes(d: int, n: int, initial: float, final: float, warmup_steps: int, step: int):
    r, k = C.c_int64(0), C.c_int64(0)
    _check(lib().oracle_warmup_sizes(d, n, initial, final, warmup_steps, step, C.byref(r), C.byref(k)), "warmup_sizes")
    return int(r.value), int(k.value)


def index_bits(d: int) -> int:
    return int(lib().oracle_index_bits(d))


def bf16_rne(x: float) -> int:
    return int(lib().oracle_bf16_rne(C.c_float(x)))


def packed_words(d: int, k: int) -> int:
    return (k * index_bits(d) + 31) // 32


def encode(msg_idx: np.ndarray, msg_val: np.ndarray, d: int, residual: np.ndarray | None = None):
    """Packed form of W rows of k (index, value) pairs: (uint32 [W, words], uint16 [W, k]).  When
    ``residual`` (float32 [W, ld]) is given, the bfloat16 rounding error is written to the sent
    coordinates' slots in place."""
    idx = np.ascontiguousarray(msg_idx, dtype=np.uint32)
    val = np.ascontiguousarray(msg_val, dtype=np.float32)
    W, k = idx.shape
    pi = np.zeros((W, packed_words(d, k)), dtype=np.uint32)
    pv = np.zeros((W, k), dtype=np.uint16)
    for w in range(W):
        res = None if residual is None else residual[w].ctypes.data_as(C.POINTER(C.c_float))
        _check(lib().oracle_encode_row(_p(idx[w], C.c_uint32), _p(val[w], C.c_float), k, d, _p(pi[w], C.c_uint32),
                                       _p(pv[w], C.c_uint16), res), "encode_row")
    return pi, pv


def decode(packed_idx: np.ndarray, packed_val: np.ndarray, d: int, k: int):
    pi = np.ascontiguousarray(packed_idx, dtype=np.uint32)
    pv = np.ascontiguousarray(packed_val, dtype=np.uint16)
    W = pi.shape[0]
    idx = np.zeros((W, k), dtype=np.uint32)
    val = np.zeros((W, k), dtype=np.float32)
    for w in range(W):
        _check(lib().oracle_decode_row(_p(pi[w], C.c_uint32), _p(pv[w], C.c_uint16), k, d, _p(idx[w], C.c_uint32),
                                       _p(val[w], C.c_float)), "decode_row")
    return idx, val


def tiled_spans(d: int) -> int:
    return int(lib().oracle_tiled_spans(d))


def encode_tiled(msg_idx: np.ndarray, msg_val: np.ndarray, d: int, residual: np.ndarray | None = None):
    """Span-table form of W ascending rows of k (index, value) pairs: (uint32 [W, T + 1] table,
    uint16 [W, k] low index bits, uint16 [W, k] bfloat16 values).  When ``residual`` (float32 [W, ld]) is
    given, the bfloat16 rounding error is written to the sent coordinates' slots in place."""
    idx = np.ascontiguousarray(msg_idx, dtype=np.uint32)
    val = np.ascontiguousarray(msg_val, dtype=np.float32)
    W, k = idx.shape
    T = tiled_spans(d)
    tab = np.zeros((W, T + 1), dtype=np.uint32)
    low = np.zeros((W, k), dtype=np.uint16)
    qv = np.zeros((W, k), dtype=np.uint16)
    for w in range(W):
        res = None if residual is None else residual[w].ctypes.data_as(C.POINTER(C.c_float))
        _check(lib().oracle_encode_tiled_row(_p(idx[w], C.c_uint32), _p(val[w], C.c_float), k, d, _p(tab[w], C.c_uint32),
                                             _p(low[w], C.c_uint16), _p(qv[w], C.c_uint16), res), "encode_tiled_row")
    return tab, low, qv


def decode_tiled(tab: np.ndarray, low: np.ndarray, qval: np.ndarray, d: int, k: int):
    tab = np.ascontiguousarray(tab, dtype=np.uint32)
    low = np.ascontiguousarray(low, dtype=np.uint16)
    qv = np.ascontiguousarray(qval, dtype=np.uint16)
    W = tab.shape[0]
    idx = np.zeros((W, k), dtype=np.uint32)
    val = np.zeros((W, k), dtype=np.float32)
    for w in range(W):
        _check(lib().oracle_decode_tiled_row(_p(tab[w], C.c_uint32), _p(low[w], C.c_uint16), _p(qv[w], C.c_uint16), k, d,
                                             _p(idx[w], C.c_uint32), _p(val[w], C.c_float)), "decode_tiled_row")
    return idx, val


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))


def sparsify_threshold(grad: np.ndarray, residual: np.ndarray, d: int, theta: float, k: int, seed: int,
                       step: int, worker_base: int = 0, signs: bool = False):
    """Threshold-then-subsample encoder (proof of Theorem 1) on W rows; ``residual`` is updated in place.
    ``signs``: a kept coordinate carries sign(a_i) * 2 theta instead of a_i.
    Returns (msg_idx [W,k] uint32, msg_val [W,k] float32, count [W] uint32, ones [W] uint32)."""
    dt = _grad_args(grad)
    assert residual.dtype == np.float32 and residual.ndim == 2 and residual.flags.c_contiguous
    W = grad.shape[0]
    assert residual.shape[0] == W
    idx = np.zeros((W, k), dtype=np.uint32)
    val = np.zeros((W, k), dtype=np.float32)
    count = np.zeros(W, dtype=np.uint32)
    ones = np.zeros(W, dtype=np.uint32)
    _check(lib().oracle_sparsify_threshold(grad.ctypes.data, dt, grad.shape[1], _p(residual, C.c_float),
                                           residual.shape[1], d, W, worker_base, theta, k, seed, step,
                                           1 if signs else 0, _p(idx, C.c_uint32), _p(val, C.c_float), _p(count, C.c_uint32),
                                           _p(ones, C.c_uint32)), "sparsify_threshold")
    return idx, val, count, ones


def aggregate_threshold(msg_idx: np.ndarray, msg_val: np.ndarray, count: np.ndarray, ones: np.ndarray, d: int):
    """Estimator of the proof of Theorem 1: (1/n) sum_w kept_w / S_w.  Returns (out64, out32)."""
    idx = np.ascontiguousarray(msg_idx, dtype=np.uint32)
    val = np.ascontiguousarray(msg_val, dtype=np.float32)
    cnt = np.ascontiguousarray(count, dtype=np.uint32)
    one = np.ascontiguousarray(ones, dtype=np.uint32)
    W, k = idx.shape
    o64 = np.zeros(d, dtype=np.float64)
    o32 = np.zeros(d, dtype=np.float32)
    _check(lib().oracle_aggregate_threshold(_p(idx, C.c_uint32), _p(val, C.c_float), _p(cnt, C.c_uint32),
                                            _p(one, C.c_uint32), d, W, k, _p(o64, C.c_double),
                                            _p(o32, C.c_float)), "aggregate_threshold")
    return o64, o32
