"""ctypes binding of librtopk.so with the same entry-point names as include/rtopk.h.

Argument marshalling only: every step of the path runs in the library's kernels.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librtopk.so")

GRAD_F32, GRAD_BF16 = 0, 1
SCALE_MEAN, SCALE_SUM, SCALE_UNBIASED, SCALE_COUNT = 0, 1, 2, 3
OPT_SELECT_PATH, OPT_PROFILE, OPT_REUSE_THRESHOLD, OPT_THRESHOLD_SIGNS, OPT_DEVICE_STEP, OPT_FINISH_PATH = 0, 1, 2, 3, 4, 5
OPT_TEST_STREAM_GIVEUP = 6
PHASES = ("subset", "threshold", "stream", "order", "exact", "finish", "aggregate")

_vp, _i32, _i64, _u32, _u64, _int = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_int

# name -> (restype, argtypes); every symbol include/rtopk.h declares
EXPORTS = {
    "rtopk_version": (_int, []),
    "rtopk_status_string": (C.c_char_p, [_int]),
    "rtopk_last_cuda_error": (_int, [_vp]),
    "rtopk_create": (_int, [C.POINTER(_vp), _int, _i64, _i32, _i64, _i64, _i32]),
    "rtopk_destroy": (_int, [_vp]),
    "rtopk_set_option": (_int, [_vp, _int, _i64]),
    "rtopk_sparsify": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _i64, _u64, _u32,
                              _vp, _vp, _vp]),
    "rtopk_aggregate": (_int, [_vp, _vp, _vp, _i64, _i32, _i64, _int, _vp, _vp]),
    "rtopk_step": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _i64, _u64, _u32, _int,
                          _vp, _vp, _vp, _vp]),
    "rtopk_sparsify_pairs": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _i64, _u64, _u32, _vp, _vp]),
    "rtopk_aggregate_pairs": (_int, [_vp, _vp, _i64, _i32, _i64, _int, _vp, _vp]),
    "rtopk_aggregate_unbiased": (_int, [_vp, _vp, _vp, _i64, _i32, _i64, _i64, _vp, _vp]),
    "rtopk_warmup_sizes": (_int, [_i64, _i32, C.c_double, C.c_double, _i64, _i64, C.POINTER(_i64), C.POINTER(_i64)]),
    "rtopk_packed_layout": (_int, [_i64, _i64, C.POINTER(_i32), C.POINTER(_i64), C.POINTER(_i64)]),
    "rtopk_encode": (_int, [_vp, _vp, _vp, _i64, _i32, _i64, _vp, _i64, _vp, _i64, _vp, _i64, _vp]),
    "rtopk_aggregate_packed": (_int, [_vp, _vp, _i64, _vp, _i64, _i64, _i32, _i64, _int, _vp, _vp]),
    "rtopk_tiled_layout": (_int, [_i64, _i64, C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64)]),
    "rtopk_encode_tiled": (_int, [_vp, _vp, _vp, _i64, _i32, _i64, _vp, _i64, _vp, _vp, _i64, _vp, _i64, _vp]),
    "rtopk_aggregate_tiled": (_int, [_vp, _vp, _vp, _i64, _vp, _i64, _i64, _i32, _i64, _int, _vp, _vp]),
    "rtopk_apply_momentum": (_int, [_vp, _vp, _vp, _i64, _i32, _i64, _int, _i64, C.c_float, C.c_float, _vp, _vp, _vp]),
    "rtopk_step_momentum": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _i64, _u64, _u32, _int,
                                   C.c_float, C.c_float, _vp, _vp, _vp, _vp, _vp]),
    "rtopk_apply_update": (_int, [_vp, _vp, _vp, _i64, _i32, _i64, _int, C.c_float, _vp, _vp]),
    "rtopk_step_apply": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _i64, _u64, _u32, _int,
                                C.c_float, _vp, _vp, _vp, _vp]),
    "rtopk_sparsify_segmented": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i32,
                                        C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), _u64, _u32,
                                        _vp, _vp, _vp]),
    "rtopk_step_segmented": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i32,
                                    C.POINTER(_i64), C.POINTER(_i64), C.POINTER(_i64), _u64, _u32, _int,
                                    _vp, _vp, _vp, _vp]),
    "rtopk_step_host": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, _i64, _i64, _u64, _u32,
                               _int, _vp, _vp, _vp, _vp]),
    "rtopk_sparsify_threshold": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, C.c_float, _i64, _u64, _u32,
                                        _vp, _vp, _vp, _vp, _vp]),
    "rtopk_aggregate_threshold": (_int, [_vp, _vp, _vp, _vp, _vp, _i64, _i32, _i64, _vp, _vp]),
    "rtopk_step_threshold": (_int, [_vp, _vp, _int, _i64, _vp, _i64, _i64, _i32, _i32, C.c_float, _i64, _u64, _u32,
                                    _vp, _vp, _vp, _vp, _vp, _vp]),
    "rtopk_sample_positions": (_int, [_vp, _i64, _i64, _u64, _u32, _u32, _u32, _vp, _vp]),
    "rtopk_sample_positions_static": (_int, [_i64, _i64, _u64, _u32, _u32, _u32, _vp, _vp]),
    "rtopk_set_device_step": (_int, [_vp, _u32, _vp]),
    "rtopk_poll_status": (_int, [_vp, _vp]),
    "rtopk_get_phase_times": (_int, [_vp, _vp, _vp]),
    "rtopk_get_stats": (_int, [_vp, _i32, _vp, _vp]),
    "rtopk_get_launch_count": (_int, [_vp, _vp]),
}

_lib: Optional[C.CDLL] = None


class RTopKError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        self.status = status
        super().__init__(f"{what}: status {status} ({detail})")


def warmup_sizes(d: int, n_workers: int, initial_density: float, final_density: float, warmup_steps: int,
                 step: int):
    """(r, k) of round `step` under the exponential warm-up schedule with k / r = 1 / n."""
    r, k = _i64(0), _i64(0)
    rc = load_library().rtopk_warmup_sizes(d, n_workers, initial_density, final_density, warmup_steps, step,
                                           C.byref(r), C.byref(k))
    if rc != 0:
        raise RTopKError(rc, "rtopk_warmup_sizes", "invalid argument")
    return int(r.value), int(k.value)


def packed_layout(d: int, k: int):
    """(index bits, row stride in 32-bit words, row stride in 16-bit halves) of the packed format."""
    bits, lw, lh = _i32(0), _i64(0), _i64(0)
    rc = load_library().rtopk_packed_layout(d, k, C.byref(bits), C.byref(lw), C.byref(lh))
    if rc != 0:
        raise RTopKError(rc, "rtopk_packed_layout", "invalid argument")
    return int(bits.value), int(lw.value), int(lh.value)


def tiled_layout(d: int, k: int):
    """(spans, row stride of the low index halves, row stride of the value halves) of the span-table format;
    the table itself has spans + 1 words per row."""
    sp, ll, lh = _i64(0), _i64(0), _i64(0)
    rc = load_library().rtopk_tiled_layout(d, k, C.byref(sp), C.byref(ll), C.byref(lh))
    if rc != 0:
        raise RTopKError(rc, "rtopk_tiled_layout", "invalid argument")
    return int(sp.value), int(ll.value), int(lh.value)


def library_path() -> str:
    return _LIB_PATH


def load_library() -> C.CDLL:
    """Loads librtopk.so and declares every exported symbol.  Raises if it is not built."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2005_10761_b200.build` "
                               "(there is no CPU fallback)")
        lib = C.CDLL(_LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


STATIC_MAX_R = 1 << 20


def sample_positions_static(r: int, k: int, seed: int, step: int, worker: int, segment: int, pos) -> None:
    """rtopk_sample_positions_static: the k-of-r positions without a context and without any device
    allocation, for callers that must not allocate (see include/rtopk.h).  ``pos`` is a device tensor
    of k 32-bit entries on the current device.  Raises RTopKError (status 4) if r > STATIC_MAX_R."""
    lib = load_library()
    rc = lib.rtopk_sample_positions_static(r, k, seed, step, worker, segment, pos.data_ptr(), _stream())
    if rc != 0:
        raise RTopKError(rc, "rtopk_sample_positions_static", lib.rtopk_status_string(rc).decode())


class Stats(C.Structure):
    _fields_ = [("tau_key", _u32), ("tie_quota", _u32), ("n_greater", _u32), ("n_candidates", _u32),
                ("used_fallback", _u32), ("bracket_predicted", _u32), ("reserved", _u32 * 2)]


def _i64_array(xs: Sequence[int]):
    return (_i64 * len(xs))(*[int(x) for x in xs])


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class RTopK:
    """A library context on one device.  Methods mirror the C entry points; tensors must live on
    that device (except the pinned host tensors of :meth:`step_host`) and are passed by pointer."""

    def __init__(self, d_max: int, W_max: int, r_max: int, k_max: int, segments_max: int = 1,
                 device: Optional[int] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("rTop-k needs a CUDA device: there is no CPU fallback")
        self._lib = load_library()
        self.device = torch.cuda.current_device() if device is None else int(device)
        h = _vp()
        rc = self._lib.rtopk_create(C.byref(h), self.device, d_max, W_max, r_max, k_max, segments_max)
        self._h = h
        if rc != 0:
            self._h = None
            raise RTopKError(rc, "rtopk_create", self._lib.rtopk_status_string(rc).decode())

    def close(self) -> None:
        if getattr(self, "_h", None):
            self._lib.rtopk_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int, what: str) -> None:
        if rc != 0:
            detail = self._lib.rtopk_status_string(rc).decode()
            if rc == 3:
                detail += f", cudaError {self._lib.rtopk_last_cuda_error(self._h)}"
            raise RTopKError(rc, what, detail)

    @staticmethod
    def _grad_dtype(grad: torch.Tensor) -> int:
        if grad.dtype == torch.float32:
            return GRAD_F32
        if grad.dtype == torch.bfloat16:
            return GRAD_BF16
        raise TypeError("gradient must be float32 or bfloat16")

    def set_option(self, option: int, value: int) -> None:
        self._check(self._lib.rtopk_set_option(self._h, option, value), "rtopk_set_option")

    def sparsify(self, grad, residual, d, r, k, seed, step, msg_idx, msg_val, worker_base=0) -> None:
        W = grad.shape[0]
        rc = self._lib.rtopk_sparsify(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                      residual.data_ptr(), residual.stride(0), d, W, worker_base, r, k,
                                      seed, step, msg_idx.data_ptr(), msg_val.data_ptr(), _stream())
        self._check(rc, "rtopk_sparsify")

    def aggregate(self, msg_idx, msg_val, d, out, scale_mode=SCALE_MEAN) -> None:
        W, k = msg_idx.shape
        rc = self._lib.rtopk_aggregate(self._h, msg_idx.data_ptr(), msg_val.data_ptr(), d, W, k, scale_mode,
                                       out.data_ptr(), _stream())
        self._check(rc, "rtopk_aggregate")

    def step(self, grad, residual, d, r, k, seed, step, msg_idx, msg_val, out, worker_base=0,
             scale_mode=SCALE_MEAN) -> None:
        W = grad.shape[0]
        rc = self._lib.rtopk_step(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                  residual.data_ptr(), residual.stride(0), d, W, worker_base, r, k, seed, step,
                                  scale_mode, msg_idx.data_ptr(), msg_val.data_ptr(), out.data_ptr(), _stream())
        self._check(rc, "rtopk_step")

    def sparsify_pairs(self, grad, residual, d, r, k, seed, step, msg_pairs, worker_base=0) -> None:
        """msg_pairs: int64 [W, k] device tensor; entry = index | (value bits << 32)."""
        W = grad.shape[0]
        rc = self._lib.rtopk_sparsify_pairs(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                            residual.data_ptr(), residual.stride(0), d, W, worker_base, r, k,
                                            seed, step, msg_pairs.data_ptr(), _stream())
        self._check(rc, "rtopk_sparsify_pairs")

    def aggregate_pairs(self, msg_pairs, d, out, scale_mode=SCALE_MEAN) -> None:
        W, k = msg_pairs.shape
        rc = self._lib.rtopk_aggregate_pairs(self._h, msg_pairs.data_ptr(), d, W, k, scale_mode, out.data_ptr(),
                                             _stream())
        self._check(rc, "rtopk_aggregate_pairs")

    def aggregate_unbiased(self, msg_idx, msg_val, d, r, out) -> None:
        W, k = msg_idx.shape
        rc = self._lib.rtopk_aggregate_unbiased(self._h, msg_idx.data_ptr(), msg_val.data_ptr(), d, W, k, r,
                                                out.data_ptr(), _stream())
        self._check(rc, "rtopk_aggregate_unbiased")

    def encode(self, msg_idx, msg_val, d, packed_idx, packed_val, residual=None) -> None:
        """msg -> packed rows (int32 [W, ld_words], int16 [W, ld_halves]); with `residual` the
        bfloat16 rounding error goes back into the sent coordinates' slots."""
        W, k = msg_idx.shape
        rc = self._lib.rtopk_encode(self._h, msg_idx.data_ptr(), msg_val.data_ptr(), d, W, k,
                                    residual.data_ptr() if residual is not None else None,
                                    residual.stride(0) if residual is not None else 0,
                                    packed_idx.data_ptr(), packed_idx.stride(0), packed_val.data_ptr(),
                                    packed_val.stride(0), _stream())
        self._check(rc, "rtopk_encode")

    def aggregate_packed(self, packed_idx, packed_val, d, k, out, scale_mode=SCALE_MEAN) -> None:
        W = packed_idx.shape[0]
        rc = self._lib.rtopk_aggregate_packed(self._h, packed_idx.data_ptr(), packed_idx.stride(0),
                                              packed_val.data_ptr(), packed_val.stride(0), d, W, k, scale_mode,
                                              out.data_ptr(), _stream())
        self._check(rc, "rtopk_aggregate_packed")

    def encode_tiled(self, msg_idx, msg_val, d, span_tab, low_idx, packed_val, residual=None) -> None:
        """msg -> span-table rows (int32 [W, spans + 1] contiguous, int16 [W, ld_low], int16 [W, ld_halves])."""
        W, k = msg_idx.shape
        assert span_tab.is_contiguous()
        rc = self._lib.rtopk_encode_tiled(self._h, msg_idx.data_ptr(), msg_val.data_ptr(), d, W, k,
                                          residual.data_ptr() if residual is not None else None,
                                          residual.stride(0) if residual is not None else 0,
                                          span_tab.data_ptr(), low_idx.data_ptr(), low_idx.stride(0),
                                          packed_val.data_ptr(), packed_val.stride(0), _stream())
        self._check(rc, "rtopk_encode_tiled")

    def aggregate_tiled(self, span_tab, low_idx, packed_val, d, k, out, scale_mode=SCALE_MEAN) -> None:
        W = low_idx.shape[0]
        assert span_tab.is_contiguous()
        rc = self._lib.rtopk_aggregate_tiled(self._h, span_tab.data_ptr(), low_idx.data_ptr(), low_idx.stride(0),
                                             packed_val.data_ptr(), packed_val.stride(0), d, W, k, scale_mode,
                                             out.data_ptr(), _stream())
        self._check(rc, "rtopk_aggregate_tiled")

    def apply_momentum(self, msg_idx, msg_val, d, eta, mu, velocity, weights, scale_mode=SCALE_MEAN, r=0) -> None:
        W, k = msg_idx.shape
        rc = self._lib.rtopk_apply_momentum(self._h, msg_idx.data_ptr(), msg_val.data_ptr(), d, W, k, scale_mode, r,
                                            eta, mu, velocity.data_ptr(), weights.data_ptr(), _stream())
        self._check(rc, "rtopk_apply_momentum")

    def step_momentum(self, grad, residual, d, r, k, seed, step, eta, mu, msg_idx, msg_val, velocity, weights,
                      worker_base=0, scale_mode=SCALE_MEAN) -> None:
        W = grad.shape[0]
        rc = self._lib.rtopk_step_momentum(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                           residual.data_ptr(), residual.stride(0), d, W, worker_base, r, k, seed,
                                           step, scale_mode, eta, mu, msg_idx.data_ptr(), msg_val.data_ptr(),
                                           velocity.data_ptr(), weights.data_ptr(), _stream())
        self._check(rc, "rtopk_step_momentum")

    def apply_update(self, msg_idx, msg_val, d, eta, weights, scale_mode=SCALE_MEAN) -> None:
        W, k = msg_idx.shape
        rc = self._lib.rtopk_apply_update(self._h, msg_idx.data_ptr(), msg_val.data_ptr(), d, W, k, scale_mode,
                                          eta, weights.data_ptr(), _stream())
        self._check(rc, "rtopk_apply_update")

    def step_apply(self, grad, residual, d, r, k, seed, step, eta, msg_idx, msg_val, weights, worker_base=0,
                   scale_mode=SCALE_MEAN) -> None:
        W = grad.shape[0]
        rc = self._lib.rtopk_step_apply(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                        residual.data_ptr(), residual.stride(0), d, W, worker_base, r, k, seed,
                                        step, scale_mode, eta, msg_idx.data_ptr(), msg_val.data_ptr(),
                                        weights.data_ptr(), _stream())
        self._check(rc, "rtopk_step_apply")

    def sparsify_segmented(self, grad, residual, d, seg_off, seg_r, seg_k, seed, step, msg_idx, msg_val,
                           worker_base=0) -> None:
        W, S = grad.shape[0], len(seg_r)
        rc = self._lib.rtopk_sparsify_segmented(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                                residual.data_ptr(), residual.stride(0), d, W, worker_base, S,
                                                _i64_array(seg_off), _i64_array(seg_r), _i64_array(seg_k),
                                                seed, step, msg_idx.data_ptr(), msg_val.data_ptr(), _stream())
        self._check(rc, "rtopk_sparsify_segmented")

    def step_segmented(self, grad, residual, d, seg_off, seg_r, seg_k, seed, step, msg_idx, msg_val, out,
                       worker_base=0, scale_mode=SCALE_MEAN) -> None:
        W, S = grad.shape[0], len(seg_r)
        rc = self._lib.rtopk_step_segmented(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                            residual.data_ptr(), residual.stride(0), d, W, worker_base, S,
                                            _i64_array(seg_off), _i64_array(seg_r), _i64_array(seg_k), seed,
                                            step, scale_mode, msg_idx.data_ptr(), msg_val.data_ptr(),
                                            out.data_ptr(), _stream())
        self._check(rc, "rtopk_step_segmented")

    def step_host(self, h_grad, residual, d, r, k, seed, step, h_msg_idx, h_msg_val, h_out, worker_base=0,
                  scale_mode=SCALE_MEAN) -> None:
        W = h_grad.shape[0]
        rc = self._lib.rtopk_step_host(self._h, h_grad.data_ptr(), self._grad_dtype(h_grad), h_grad.stride(0),
                                       residual.data_ptr(), residual.stride(0), d, W, worker_base, r, k, seed,
                                       step, scale_mode, h_msg_idx.data_ptr(), h_msg_val.data_ptr(),
                                       h_out.data_ptr(), _stream())
        self._check(rc, "rtopk_step_host")

    def sparsify_threshold(self, grad, residual, d, theta, k, seed, step, msg_idx, msg_val, msg_count, msg_ones,
                           worker_base=0) -> None:
        """Threshold-then-subsample encoder: msg_count / msg_ones are int32 [W] device tensors."""
        W = grad.shape[0]
        rc = self._lib.rtopk_sparsify_threshold(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                                residual.data_ptr(), residual.stride(0), d, W, worker_base, theta, k,
                                                seed, step, msg_idx.data_ptr(), msg_val.data_ptr(),
                                                msg_count.data_ptr(), msg_ones.data_ptr(), _stream())
        self._check(rc, "rtopk_sparsify_threshold")

    def aggregate_threshold(self, msg_idx, msg_val, msg_count, msg_ones, d, out) -> None:
        W, k = msg_idx.shape
        rc = self._lib.rtopk_aggregate_threshold(self._h, msg_idx.data_ptr(), msg_val.data_ptr(),
                                                 msg_count.data_ptr(), msg_ones.data_ptr(), d, W, k, out.data_ptr(),
                                                 _stream())
        self._check(rc, "rtopk_aggregate_threshold")

    def step_threshold(self, grad, residual, d, theta, k, seed, step, msg_idx, msg_val, msg_count, msg_ones, out,
                       worker_base=0) -> None:
        W = grad.shape[0]
        rc = self._lib.rtopk_step_threshold(self._h, grad.data_ptr(), self._grad_dtype(grad), grad.stride(0),
                                            residual.data_ptr(), residual.stride(0), d, W, worker_base, theta, k,
                                            seed, step, msg_idx.data_ptr(), msg_val.data_ptr(),
                                            msg_count.data_ptr(), msg_ones.data_ptr(), out.data_ptr(), _stream())
        self._check(rc, "rtopk_step_threshold")

    def sample_positions(self, r, k, seed, step, worker, segment, pos) -> None:
        rc = self._lib.rtopk_sample_positions(self._h, r, k, seed, step, worker, segment, pos.data_ptr(),
                                              _stream())
        self._check(rc, "rtopk_sample_positions")

    def set_device_step(self, step: int) -> None:
        self._check(self._lib.rtopk_set_device_step(self._h, step, _stream()), "rtopk_set_device_step")

    def poll_status(self) -> None:
        self._check(self._lib.rtopk_poll_status(self._h, _stream()), "rtopk_poll_status")

    def phase_times(self) -> dict:
        ms = (C.c_float * len(PHASES))()
        self._check(self._lib.rtopk_get_phase_times(self._h, ms, _stream()), "rtopk_get_phase_times")
        return {name: float(ms[i]) for i, name in enumerate(PHASES)}

    def launch_count(self) -> int:
        n = C.c_uint64(0)
        self._check(self._lib.rtopk_get_launch_count(self._h, C.byref(n)), "rtopk_get_launch_count")
        return int(n.value)

    def stats(self, slice_index: int) -> dict:
        s = Stats()
        self._check(self._lib.rtopk_get_stats(self._h, slice_index, C.byref(s), _stream()), "rtopk_get_stats")
        return {f: getattr(s, f) for f, _ in Stats._fields_ if f != "reserved"}
