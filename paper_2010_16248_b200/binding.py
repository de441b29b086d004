"""ctypes binding of the C-ABI library (include/acc.h): argument marshalling only.

Every step of the path runs in the library's CUDA kernels.  torch is used for device
memory and streams.  There is no CPU fallback: loading fails loudly when the library
has not been built, and every call checks that its tensors live on a CUDA device.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

from . import build as _build

ACC_OK = 0
ACC_MATRIX, ACC_VECTOR = 0, 1
ACC_MAX_RANK = 4
ACC_FLAG_LAZY_RESIDUAL = 1
ACC_FLAG_PIPELINE_ALWAYS = 2
ACC_FLAG_PIPELINE_NEVER = 4
ACC_FLAG_SHARE_SMS = 8
POWERSGD, TOPK = 0, 1
ACC_TOPK_PATH_DENSE, ACC_TOPK_PATH_LIST, ACC_TOPK_PATH_LIST_PREDICTED, ACC_TOPK_PATH_STAGED, ACC_TOPK_PATH_ZERO_FILL = range(5)


class AccError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lib().acc_strerror(status).decode()} (status {status})")


class acc_layer_desc(C.Structure):
    _fields_ = [("offset", C.c_int64), ("rows", C.c_int32), ("cols", C.c_int32), ("kind", C.c_int32),
                ("reserved", C.c_int32)]


class acc_config(C.Structure):
    _fields_ = [("n_workers", C.c_int32), ("n_layers", C.c_int32), ("layers", C.POINTER(acc_layer_desc)),
                ("worker_stride", C.c_int64), ("rank_low", C.c_int32), ("rank_high", C.c_int32),
                ("topk_low_bp", C.c_int32), ("topk_high_bp", C.c_int32), ("eta", C.c_float),
                ("gs_eps", C.c_float), ("decider", C.c_int32), ("flags", C.c_int32)]


EXPORTS = ["acc_workspace_bytes", "acc_create", "acc_destroy", "acc_factor_layout", "acc_topk_layout",
           "acc_error_feedback", "acc_layer_norms", "acc_detect_regime", "acc_powersgd_step", "acc_topk_step",
           "acc_floats_sent", "acc_last_launch_count", "acc_strerror", "acc_profile_enable", "acc_profile_read",
           "acc_profile_kernel_count", "acc_profile_kernel_name", "acc_sumsq_static", "acc_powersgd_flush", "acc_device_status", "acc_topk_last_paths",
           "acc_layer_diff_norms", "acc_detect_regime_diff", "acc_sgd_nesterov", "acc_powersgd_step_sgd",
           "acc_topk_step_sgd", "acc_batch_accumulate", "acc_batch_average", "acc_detect_batch",
           "acc_exchange_layout", "acc_powersgd_phase1", "acc_powersgd_phase2", "acc_powersgd_phase3",
           "acc_topk_compress", "acc_topk_decompress", "acc_topk_flush",
           "acc_upload_grads", "acc_download_out", "acc_selftest_wait_timeout", "acc_reset_device_status",
           "acc_layer_msdr", "acc_detect_regime_lr"]

_lib = None


def lib() -> C.CDLL:
    """Loads libacc.so (built in-tree by ``build.build_library``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} not found: build it with `python -m paper_2010_16248_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(path)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    L.acc_workspace_bytes.argtypes = [C.POINTER(acc_config), C.POINTER(C.c_size_t)]
    L.acc_create.argtypes = [C.POINTER(acc_config), vp, C.c_size_t, C.POINTER(vp)]
    L.acc_destroy.argtypes = [vp]
    L.acc_factor_layout.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)]
    L.acc_topk_layout.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)]
    L.acc_error_feedback.argtypes = [vp, vp, vp, vp, vp]
    L.acc_layer_norms.argtypes = [vp, vp, i64, i32, vp, vp]
    L.acc_layer_msdr.argtypes = [vp, vp, i64, i32, vp, vp, vp]
    L.acc_detect_regime.argtypes = [vp, vp, vp, f32, f32, vp, vp, vp]
    L.acc_detect_regime_lr.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.acc_powersgd_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.acc_topk_step.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.acc_floats_sent.argtypes = [C.POINTER(acc_config), C.POINTER(C.c_uint8), i32]
    L.acc_floats_sent.restype = i64
    L.acc_last_launch_count.argtypes = [vp]
    L.acc_last_launch_count.restype = i32
    L.acc_strerror.argtypes = [C.c_int]
    L.acc_strerror.restype = C.c_char_p
    L.acc_profile_enable.argtypes = [vp, i32]
    L.acc_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i32), i32]
    L.acc_profile_kernel_count.argtypes = []
    L.acc_profile_kernel_count.restype = i32
    L.acc_profile_kernel_name.argtypes = [i32]
    L.acc_profile_kernel_name.restype = C.c_char_p
    L.acc_sumsq_static.argtypes = [vp, i64, vp, vp]
    L.acc_powersgd_flush.argtypes = [vp, vp, vp, vp, vp]
    L.acc_device_status.argtypes = [vp, C.POINTER(i32)]
    L.acc_topk_last_paths.argtypes = [vp, C.POINTER(i32), i32]
    L.acc_layer_diff_norms.argtypes = [vp, vp, vp, vp, vp]
    L.acc_detect_regime_diff.argtypes = [vp, vp, vp, vp, f32, f32, vp, vp, vp, vp]
    L.acc_sgd_nesterov.argtypes = [vp, vp, vp, vp, vp, vp]
    L.acc_powersgd_step_sgd.argtypes = [vp] * 12
    L.acc_topk_step_sgd.argtypes = [vp] * 13
    L.acc_batch_accumulate.argtypes = [vp, vp, vp, vp, i32, vp]
    L.acc_batch_average.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    L.acc_detect_batch.argtypes = [vp, vp, vp, f32, f32, i32, i32, vp, vp, vp, vp]
    L.acc_exchange_layout.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)]
    L.acc_powersgd_phase1.argtypes = [vp] * 10
    L.acc_powersgd_phase2.argtypes = [vp, vp, f32, vp, vp, vp, vp, vp]
    L.acc_powersgd_phase3.argtypes = [vp, vp, vp, vp, vp, vp, vp, f32, vp, vp, vp, vp, vp]
    L.acc_topk_compress.argtypes = [vp] * 10
    L.acc_topk_decompress.argtypes = [vp, vp, vp, vp, i32, vp, f32, vp, vp, vp, vp, vp]
    L.acc_topk_flush.argtypes = [vp, vp, vp]
    L.acc_upload_grads.argtypes = [vp, vp, vp, vp]
    L.acc_selftest_wait_timeout.argtypes = [vp, vp]
    L.acc_reset_device_status.argtypes = [vp, vp]
    L.acc_download_out.argtypes = [vp, vp, vp, vp]
    for name in EXPORTS:
        if name not in ("acc_floats_sent", "acc_last_launch_count", "acc_strerror", "acc_profile_kernel_count",
                        "acc_profile_kernel_name"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def make_config(table, n_workers, rank_low=2, rank_high=1, topk_low_bp=1000, topk_high_bp=100, eta=0.5,
                gs_eps=1e-8, decider=0, worker_stride=None, flags=0):
    """Builds an ``acc_config`` (plus the array it points to) from a workloads.LayerTable."""
    L = table.n_layers
    arr = (acc_layer_desc * L)()
    for l in range(L):
        arr[l].offset = int(table.offset[l]); arr[l].rows = int(table.rows[l]); arr[l].cols = int(table.cols[l])
        arr[l].kind = int(table.kind[l]); arr[l].reserved = 0
    cfg = acc_config(n_workers, L, arr, int(worker_stride if worker_stride is not None else table.stride),
                     rank_low, rank_high, topk_low_bp, topk_high_bp, eta, gs_eps, decider, flags)
    cfg._keepalive = arr
    return cfg


def acc_floats_sent(cfg: acc_config, level, compressor: int) -> int:
    lv = (C.c_uint8 * cfg.n_layers)(*[int(x) for x in level])
    return int(lib().acc_floats_sent(C.byref(cfg), lv, compressor))


def acc_sumsq_static(buf: torch.Tensor, n: int, norm2: torch.Tensor, stream=None) -> None:
    """Squared L2 norm of the first ``n`` floats of ``buf`` into the one-element fp64 tensor ``norm2``.

    For callers that cannot allocate device memory or supply a workspace: the reduction scratch is a
    fixed array inside the library, so this call allocates nothing (neither do these few lines).
    ``n`` is limited to 2**28 elements; calls that overlap on the GPU share the scratch and race."""
    n = int(n)
    st = lib().acc_sumsq_static(*_marshal(None, _Arg(buf, torch.float32, max(n, 0), "buf"), n,
                                          _Arg(norm2, torch.float64, 1, "norm2")), _stream(stream))
    if st != ACC_OK:
        raise AccError(st, "acc_sumsq_static")


class _Arg:
    """One tensor argument of a call with what the call requires of it."""
    __slots__ = ("t", "dtype", "min_numel", "what")

    def __init__(self, t, dtype, min_numel, what):
        self.t, self.dtype, self.min_numel, self.what = t, dtype, int(min_numel), what


def _marshal(device, *items):
    """Turns the ``_Arg`` items into device addresses (other items pass through) after checking what the C ABI
    cannot see.  First every tensor's dtype, contiguity and length -- the kernels index by the context's layout, so
    a short tensor would be an out-of-bounds device access, not an exception -- then that every tensor lives on
    the GPU the call runs on (there is no CPU path)."""
    for a in items:
        if not isinstance(a, _Arg) or a.t is None:
            continue
        t = a.t
        if not isinstance(t, torch.Tensor):
            raise ValueError(f"{a.what}: expected a torch tensor")
        if t.dtype != a.dtype:
            raise ValueError(f"{a.what}: expected dtype {a.dtype}, got {t.dtype}")
        if not t.is_contiguous():
            raise ValueError(f"{a.what}: expected a contiguous tensor")
        if t.numel() < a.min_numel:
            raise ValueError(f"{a.what}: {t.numel()} elements, the call needs at least {a.min_numel}")
    out = []
    for a in items:
        if not isinstance(a, _Arg):
            out.append(a)
            continue
        if a.t is None:
            out.append(None)
            continue
        if not a.t.is_cuda:
            raise ValueError(f"{a.what}: expected a CUDA tensor (the library has no CPU path)")
        if device is not None and device.index is not None and a.t.device.index != device.index:
            raise ValueError(f"{a.what}: lives on {a.t.device}, the context on {device}")
        out.append(a.t.data_ptr())
    return out


def _stream(stream) -> Optional[int]:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


class Context:
    """Owns the workspace tensor and the ``acc_ctx``; methods mirror the C entry points."""

    def __init__(self, table, n_workers, device="cuda", **cfg_kwargs):
        self.table = table
        self.device = torch.device(device)
        if self.device.type == "cuda" and self.device.index is None:
            self.device = torch.device("cuda", torch.cuda.current_device())
        self.cfg = make_config(table, n_workers, **cfg_kwargs)
        self.n_workers, self.n_layers, self.stride = n_workers, table.n_layers, int(self.cfg.worker_stride)
        # elements of one worker's slice that the layer table reaches (<= worker_stride)
        self.extent = int(max(int(table.offset[l]) + int(table.rows[l]) * int(table.cols[l])
                              for l in range(table.n_layers)))
        L = lib()
        nbytes = C.c_size_t(0)
        st = L.acc_workspace_bytes(C.byref(self.cfg), C.byref(nbytes))
        if st != ACC_OK:
            raise AccError(st, "acc_workspace_bytes")
        self.workspace_bytes = int(nbytes.value)
        with torch.cuda.device(self.device):
            self.workspace = torch.zeros(max(self.workspace_bytes, 256), dtype=torch.uint8, device=self.device)
            h = C.c_void_p()
            st = L.acc_create(C.byref(self.cfg), self.workspace.data_ptr(), self.workspace_bytes, C.byref(h))
        if st != ACC_OK:
            raise AccError(st, "acc_create")
        self._h = h
        n = self.n_layers
        qr, pr = (C.c_int64 * n)(), (C.c_int64 * n)()
        qn, pn = C.c_int64(), C.c_int64()
        L.acc_factor_layout(self._h, qr, pr, C.byref(qn), C.byref(pn))
        self.q_row, self.p_row = np.array(qr[:], np.int64), np.array(pr[:], np.int64)
        self.q_rows, self.p_rows = int(qn.value), int(pn.value)
        so, kl, kh, cap = (C.c_int64 * n)(), (C.c_int64 * n)(), (C.c_int64 * n)(), C.c_int64()
        L.acc_topk_layout(self._h, so, kl, kh, C.byref(cap))
        self.seg_offset, self.k_low, self.k_high = (np.array(a[:], np.int64) for a in (so, kl, kh))
        self.capacity = int(cap.value)
        x1, x2, vf = C.c_int64(), C.c_int64(), C.c_int64()
        L.acc_exchange_layout(self._h, C.byref(x1), C.byref(x2), C.byref(vf))
        self.x1_floats, self.x2_floats, self.vec_floats = int(x1.value), int(x2.value), int(vf.value)

    def close(self):
        if getattr(self, "_h", None):
            lib().acc_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st, where):
        if st != ACC_OK:
            raise AccError(st, where)

    def _call(self, name, *items, stream=None):
        """Checks and marshals the tensor arguments, then calls entry point ``name`` on this context."""
        self._check(getattr(lib(), name)(self._h, *_marshal(self.device, *items), _stream(stream)), name)

    # --- argument checks: every device buffer must hold what the context's layout will index -----------------
    def _f(self, t, n, what):
        return _Arg(t, torch.float32, n, what)

    def _d(self, t, n, what):
        return _Arg(t, torch.float64, n, what)

    def _i(self, t, n, what):
        return _Arg(t, torch.int32, n, what)

    def _lv(self, t):
        return _Arg(t, torch.uint8, self.n_layers, "level")

    @property
    def _wn(self):  # elements of a [W][worker_stride] buffer
        return self.n_workers * self.stride

    def _tail(self, params, mom, hyper):
        if params is None:
            return None, None, None
        if mom is None or hyper is None:
            raise ValueError("the optimiser tail needs params, mom and hyper together")
        return self._f(params, self.stride, "params"), self._f(mom, self.stride, "mom"), self._f(hyper, 3, "hyper")

    # --- entry points -------------------------------------------------------------------------
    def acc_error_feedback(self, grads, err, delta=None, stream=None):
        self._call("acc_error_feedback", self._f(grads, self._wn, "grads"), self._f(err, self._wn, "err"),
                   self._f(delta, self.stride, "delta"), stream=stream)

    def acc_layer_norms(self, buf, n_bufs, norm2, buf_stride=None, stream=None):
        stride = int(buf_stride if buf_stride is not None else self.stride)
        n_bufs = int(n_bufs)
        need = (n_bufs - 1) * stride + self.extent if n_bufs >= 1 else 0
        self._call("acc_layer_norms", self._f(buf, need, "buf"), stride, n_bufs,
                   self._d(norm2, max(n_bufs, 0) * self.n_layers, "norm2"), stream=stream)

    def acc_layer_msdr(self, buf, n_bufs, moments, msdr, buf_stride=None, stream=None):
        stride = int(buf_stride if buf_stride is not None else self.stride)
        n_bufs = int(n_bufs)
        need = (n_bufs - 1) * stride + self.extent if n_bufs >= 1 else 0
        self._call("acc_layer_msdr", self._f(buf, need, "buf"), stride, n_bufs,
                   self._d(moments, 2 * max(n_bufs, 0) * self.n_layers, "moments"),
                   self._d(msdr, max(n_bufs, 0) * self.n_layers, "msdr"), stream=stream)

    def acc_detect_regime(self, norm2_curr, norm2_prev, lr_curr, lr_next, level, delta=None, stream=None):
        L = self.n_layers
        self._call("acc_detect_regime", self._d(norm2_curr, L, "norm2_curr"),
                   self._d(norm2_prev, L, "norm2_prev"), float(lr_curr), float(lr_next), self._lv(level),
                   self._f(delta, self.stride, "delta"), stream=stream)

    def acc_detect_regime_lr(self, norm2_curr, norm2_prev, lr_pair, level, delta=None, stream=None):
        L = self.n_layers
        self._call("acc_detect_regime_lr", self._d(norm2_curr, L, "norm2_curr"), self._d(norm2_prev, L, "norm2_prev"),
                   self._f(lr_pair, 2, "lr_pair"), self._lv(level), self._f(delta, self.stride, "delta"),
                   stream=stream)

    def acc_layer_diff_norms(self, a, b, norm2, stream=None):
        self._call("acc_layer_diff_norms", self._f(a, self.extent, "a"), self._f(b, self.extent, "b"),
                   self._d(norm2, self.n_layers, "norm2"), stream=stream)

    def acc_detect_regime_diff(self, norm2_diff, norm2_curr, norm2_prev, lr_curr, lr_next, level, delta, delta_prev,
                               stream=None):
        L = self.n_layers
        self._call("acc_detect_regime_diff", self._d(norm2_diff, L, "norm2_diff"),
                   self._d(norm2_curr, L, "norm2_curr"), self._d(norm2_prev, L, "norm2_prev"), float(lr_curr),
                   float(lr_next), self._lv(level), self._f(delta, self.stride, "delta"),
                   self._f(delta_prev, self.stride, "delta_prev"), stream=stream)

    def _psgd_args(self, grads, err, q, p_hat, level, out, delta):
        return (self._f(grads, self._wn, "grads"), self._f(err, self._wn, "err"), self._f(q, 4 * self.q_rows, "q"),
                self._f(p_hat, 4 * self.p_rows, "p_hat"), self._lv(level), self._f(out, self.stride, "out"),
                self._f(delta, self.stride, "delta"))

    def _topk_args(self, grads, err, level, vals, idx, counts):
        cap = self.n_workers * self.capacity
        return (self._f(grads, self._wn, "grads"), self._f(err, self._wn, "err"), self._lv(level),
                self._f(vals, cap, "vals"), self._i(idx, cap, "idx"),
                self._i(counts, self.n_workers * self.n_layers, "counts"))

    def acc_powersgd_step(self, grads, err, q, p_hat, level, out, delta=None, stream=None):
        self._call("acc_powersgd_step", *self._psgd_args(grads, err, q, p_hat, level, out, delta),
                   stream=stream)

    def acc_powersgd_flush(self, err, q, p_hat, stream=None):
        self._call("acc_powersgd_flush", self._f(err, self._wn, "err"), self._f(q, 4 * self.q_rows, "q"),
                   self._f(p_hat, 4 * self.p_rows, "p_hat"), stream=stream)

    def acc_topk_step(self, grads, err, level, vals, idx, counts, out, delta=None, stream=None):
        self._call("acc_topk_step", *self._topk_args(grads, err, level, vals, idx, counts),
                   self._f(out, self.stride, "out"), self._f(delta, self.stride, "delta"), stream=stream)

    def acc_sgd_nesterov(self, d, params, mom, hyper, stream=None):
        self._call("acc_sgd_nesterov", self._f(d, self.stride, "d"), *self._tail(params, mom, hyper),
                   stream=stream)

    def acc_powersgd_step_sgd(self, grads, err, q, p_hat, level, out, delta, params, mom, hyper, stream=None):
        self._call("acc_powersgd_step_sgd", *self._psgd_args(grads, err, q, p_hat, level, out, delta),
                   *self._tail(params, mom, hyper), stream=stream)

    def acc_topk_step_sgd(self, grads, err, level, vals, idx, counts, out, delta, params, mom, hyper, stream=None):
        self._call("acc_topk_step_sgd", *self._topk_args(grads, err, level, vals, idx, counts),
                   self._f(out, self.stride, "out"), self._f(delta, self.stride, "delta"),
                   *self._tail(params, mom, hyper), stream=stream)

    def acc_batch_accumulate(self, grads, acc, delta=None, first=False, stream=None):
        self._call("acc_batch_accumulate", self._f(grads, self._wn, "grads"), self._f(acc, self._wn, "acc"),
                   self._f(delta, self.stride, "delta"), int(bool(first)), stream=stream)

    def acc_batch_average(self, acc, n_accum, out, params=None, mom=None, hyper=None, stream=None):
        self._call("acc_batch_average", self._f(acc, self._wn, "acc"), int(n_accum),
                   self._f(out, self.stride, "out"), *self._tail(params, mom, hyper), stream=stream)

    def acc_detect_batch(self, norm2_layers, norm2_prev, lr_curr, lr_next, b_low, b_high, batch, lr_scale,
                         delta=None, stream=None):
        self._call("acc_detect_batch", self._d(norm2_layers, self.n_layers, "norm2_layers"),
                   self._d(norm2_prev, 1, "norm2_prev"), float(lr_curr), float(lr_next), int(b_low), int(b_high),
                   self._i(batch, 1, "batch"), self._f(lr_scale, 1, "lr_scale"),
                   self._f(delta, self.stride, "delta"), stream=stream)

    def acc_powersgd_phase1(self, grads, err, q, p_hat, level, out, delta, x1, stream=None):
        self._call("acc_powersgd_phase1", *self._psgd_args(grads, err, q, p_hat, level, out, delta),
                   self._f(x1, self.x1_floats, "x1"), stream=stream)

    def acc_powersgd_phase2(self, x1, scale, p_hat, level, out, x2, stream=None):
        self._call("acc_powersgd_phase2", self._f(x1, self.x1_floats, "x1"), float(scale),
                   self._f(p_hat, 4 * self.p_rows, "p_hat"), self._lv(level), self._f(out, self.stride, "out"),
                   self._f(x2, self.x2_floats, "x2"), stream=stream)

    def acc_powersgd_phase3(self, err, q, p_hat, level, x1, x2, scale, out, params=None, mom=None, hyper=None,
                            stream=None):
        self._call("acc_powersgd_phase3", self._f(err, self._wn, "err"), self._f(q, 4 * self.q_rows, "q"),
                   self._f(p_hat, 4 * self.p_rows, "p_hat"), self._lv(level), self._f(x1, self.x1_floats, "x1"),
                   self._f(x2, self.x2_floats, "x2"), float(scale), self._f(out, self.stride, "out"),
                   *self._tail(params, mom, hyper), stream=stream)

    def acc_topk_compress(self, grads, err, level, vals, idx, counts, delta, vec_packed, stream=None):
        self._call("acc_topk_compress", *self._topk_args(grads, err, level, vals, idx, counts),
                   self._f(delta, self.stride, "delta"), self._f(vec_packed, self.vec_floats, "vec_packed"),
                   stream=stream)

    def acc_topk_decompress(self, vals_all, idx_all, counts_all, n_sets, vec_packed, vec_scale, out, params=None,
                            mom=None, hyper=None, stream=None):
        n_sets = int(n_sets)
        cap = max(n_sets, 0) * self.capacity
        self._call("acc_topk_decompress", self._f(vals_all, cap, "vals_all"), self._i(idx_all, cap, "idx_all"),
                   self._i(counts_all, max(n_sets, 0) * self.n_layers, "counts_all"), n_sets,
                   self._f(vec_packed, self.vec_floats, "vec_packed"), float(vec_scale),
                   self._f(out, self.stride, "out"), *self._tail(params, mom, hyper), stream=stream)

    def acc_topk_flush(self, err, stream=None):
        self._call("acc_topk_flush", self._f(err, self._wn, "err"), stream=stream)

    def acc_upload_grads(self, grads_host, grads_dev, stream=None):
        """``grads_host``: CPU float32 tensor [W, stride] (pinned for an asynchronous copy)."""
        if grads_host.is_cuda or grads_host.dtype != torch.float32 or not grads_host.is_contiguous():
            raise ValueError("expected a contiguous float32 CPU tensor")
        if grads_host.numel() != self._wn or grads_dev.numel() != grads_host.numel():
            raise ValueError("expected [n_workers, worker_stride] elements")
        self._call("acc_upload_grads", grads_host.data_ptr(), self._f(grads_dev, self._wn, "grads_dev"),
                   stream=stream)

    def acc_download_out(self, out_dev, out_host, stream=None):
        if out_host.is_cuda or out_host.dtype != torch.float32 or not out_host.is_contiguous():
            raise ValueError("expected a contiguous float32 CPU tensor")
        if out_host.numel() != self.stride or out_dev.numel() != self.stride:
            raise ValueError("expected worker_stride elements")
        self._call("acc_download_out", self._f(out_dev, self.stride, "out_dev"), out_host.data_ptr(),
                   stream=stream)

    def acc_profile_enable(self, enable: bool):
        self._check(lib().acc_profile_enable(self._h, int(bool(enable))), "acc_profile_enable")

    def acc_profile_read(self):
        """{kernel name: (milliseconds, launches)} since the last read; waits for the recorded kernels."""
        n = int(lib().acc_profile_kernel_count())
        ms, cnt = (C.c_double * n)(), (C.c_int32 * n)()
        self._check(lib().acc_profile_read(self._h, ms, cnt, n), "acc_profile_read")
        return {lib().acc_profile_kernel_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i]}

    def acc_topk_last_paths(self) -> np.ndarray:
        """Selection path (0 dense, 1 list, 2 predicted list, 3 staged) per (worker, MATRIX layer) of the last TopK step."""
        n = self.n_workers * int((self.q_row >= 0).sum())
        buf = (C.c_int32 * max(n, 1))()
        self._check(lib().acc_topk_last_paths(self._h, buf, n), "acc_topk_last_paths")
        return np.array(buf[:n], np.int32).reshape(self.n_workers, -1)

    def acc_device_status(self) -> int:
        """Device-side status word (0 = fine); waits for the queued work of this device."""
        v = C.c_int32(0)
        self._check(lib().acc_device_status(self._h, C.byref(v)), "acc_device_status")
        return int(v.value)

    def acc_selftest_wait_timeout(self, stream=None):
        self._check(lib().acc_selftest_wait_timeout(self._h, _stream(stream)), "acc_selftest_wait_timeout")

    def acc_reset_device_status(self, stream=None):
        self._check(lib().acc_reset_device_status(self._h, _stream(stream)), "acc_reset_device_status")

    def last_launch_count(self) -> int:
        return int(lib().acc_last_launch_count(self._h))

    # --- buffer helpers (allocation and layout conversion only) -------------------------------
    def new_q(self, q_list=None):
        """Device q buffer ``[q_rows, 4]``; filled from per-layer ``[m, r]`` tensors when given."""
        # (at least one row, so that a table without MATRIX layers still has a buffer to point at)
        q = torch.zeros(max(self.q_rows, 1), ACC_MAX_RANK, dtype=torch.float32, device=self.device)
        if q_list is not None:
            for l, ql in enumerate(q_list):
                if ql is not None:
                    r0 = int(self.q_row[l])
                    q[r0:r0 + ql.shape[0], :ql.shape[1]] = ql.to(self.device)
        return q

    def new_p(self):
        return torch.zeros(max(self.p_rows, 1), ACC_MAX_RANK, dtype=torch.float32, device=self.device)

    def new_topk_buffers(self):
        W = self.n_workers
        vals = torch.zeros(max(W * self.capacity, 4), dtype=torch.float32, device=self.device)
        idx = torch.zeros(max(W * self.capacity, 4), dtype=torch.int32, device=self.device)
        counts = torch.zeros(W * self.n_layers, dtype=torch.int32, device=self.device)
        return vals, idx, counts
