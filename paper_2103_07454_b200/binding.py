"""Thin ctypes binding of the C ABI in ``include/eventgrad.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  PyTorch is used
for device memory and streams.  There is no fallback — if ``libeventgrad.so`` has not been
built (``python -m paper_2103_07454_b200.build``) the first use raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libeventgrad.so")

EG_OK = 0
TOPO_RING = 0
THRESH_ADAPTIVE = 0
THRESH_FIXED = 1

EXPORTS = [
    "eg_create", "eg_layout", "eg_step", "eg_step_host", "eg_set_carry_norm", "eg_stats",
    "eg_event_count", "eg_last_decisions", "eg_thresholds", "eg_last_outbox", "eg_topk_count",
    "eg_read_mailboxes", "eg_average_model", "eg_export_state", "eg_import_state", "eg_reset",
    "eg_destroy", "eg_strerror", "eg_last_cuda_error", "eg_last_launch_count",
    "eg_set_timing", "eg_kernel_times", "eg_set_fused_kernel", "eg_change_norms_static", "eg_set_variant", "eg_set_threshold_cap",
    "eg_enable_delivery_masks", "eg_step_masked", "eg_read_received", "eg_delivery_status",
    "eg_selftest_wait_timeout", "eg_set_momentum", "eg_read_velocity", "eg_write_velocity",
    "eg_debug_fail_allocation", "eg_status_of_error_word", "eg_debug_build",
    "eg_topk_repeat_count",
    "eg_set_quantisation",
    "eg_last_quantised",
]
STATIC_MAX_TENSORS = 192
STATIC_MAX_PARTIALS = 524288
FUSED_PIPELINED = 0
FUSED_REGISTER = 1
FUSED_AUTO = 2
KERNEL_GROUPS = ("norm", "decide", "topk", "fused")


class ThresholdParams(C.Structure):
    _fields_ = [("mode", C.c_int), ("horizon", C.c_double), ("history_len", C.c_int),
                ("delta_init", C.c_double), ("delta_fixed", C.c_double),
                ("force_first_event", C.c_int)]


class TopkParams(C.Structure):
    _fields_ = [("enabled", C.c_int), ("k_num", C.c_uint32), ("k_den", C.c_uint32)]


class EventGradError(RuntimeError):
    pass


_lib = None


def load_library() -> C.CDLL:
    """Loads the CUDA library; raises if it is missing (there is no CPU path)."""
    global _lib
    if _lib is not None:
        return _lib
    # EG_LIBRARY names another build of the same library (the bounds-checked one, for instance)
    path = os.environ.get("EG_LIBRARY") or LIB_PATH
    if not os.path.exists(path):
        raise EventGradError(
            f"{path} not found: build it with `python -m paper_2103_07454_b200.build`; "
            "this package has no CPU fallback")
    lib = C.CDLL(path)
    vp, i64p, u64p = C.c_void_p, C.POINTER(C.c_int64), C.POINTER(C.c_uint64)
    lib.eg_create.argtypes = [C.POINTER(vp), C.c_int, C.c_int, i64p, C.c_int,
                              C.POINTER(ThresholdParams), C.POINTER(TopkParams)]
    lib.eg_layout.argtypes = [vp, i64p, i64p]
    lib.eg_step.argtypes = [vp, vp, vp, C.c_float, vp]
    lib.eg_step_host.argtypes = [vp, vp, vp, C.c_float]
    lib.eg_set_carry_norm.argtypes = [vp, C.c_int]
    lib.eg_stats.argtypes = [vp, u64p, u64p]
    lib.eg_event_count.argtypes = [vp, u64p]
    lib.eg_last_decisions.argtypes = [vp, vp, vp, vp]
    lib.eg_thresholds.argtypes = [vp, vp, vp]
    lib.eg_last_outbox.argtypes = [vp, C.c_int, C.c_int, vp, vp, C.POINTER(C.c_int32)]
    lib.eg_topk_count.argtypes = [vp, C.c_int, i64p]
    lib.eg_read_mailboxes.argtypes = [vp, vp]
    lib.eg_average_model.argtypes = [vp, vp, vp, C.POINTER(C.c_double), vp]
    lib.eg_export_state.argtypes = [vp, vp, C.POINTER(C.c_size_t)]
    lib.eg_import_state.argtypes = [vp, vp, C.c_size_t]
    lib.eg_reset.argtypes = [vp]
    lib.eg_set_timing.argtypes = [vp, C.c_int]
    lib.eg_set_fused_kernel.argtypes = [vp, C.c_int]
    lib.eg_set_variant.argtypes = [vp, C.c_int, C.c_int]
    lib.eg_set_threshold_cap.argtypes = [vp, C.c_double, C.c_double]
    lib.eg_set_momentum.argtypes = [vp, C.c_int, C.c_double]
    lib.eg_read_velocity.argtypes = [vp, vp]
    lib.eg_write_velocity.argtypes = [vp, vp]
    lib.eg_enable_delivery_masks.argtypes = [vp]
    lib.eg_selftest_wait_timeout.argtypes = [vp, vp]
    lib.eg_step_masked.argtypes = [vp, vp, vp, C.c_float, vp, vp]
    lib.eg_read_received.argtypes = [vp, vp]
    lib.eg_delivery_status.argtypes = [vp, vp, u64p]
    lib.eg_change_norms_static.argtypes = [vp, vp, C.c_int, C.c_int64, i64p, i64p, C.c_int, vp, vp]
    lib.eg_kernel_times.argtypes = [vp, C.POINTER(C.c_double), u64p]
    lib.eg_debug_fail_allocation.argtypes = [C.c_int]
    lib.eg_debug_fail_allocation.restype = None
    lib.eg_destroy.argtypes = [vp]
    lib.eg_destroy.restype = None
    lib.eg_strerror.argtypes = [C.c_int]
    lib.eg_strerror.restype = C.c_char_p
    lib.eg_status_of_error_word.argtypes = [C.c_uint]
    lib.eg_debug_build.argtypes = []
    lib.eg_topk_repeat_count.argtypes = [vp, u64p]
    lib.eg_set_quantisation.argtypes = [vp, C.c_int]
    lib.eg_last_quantised.argtypes = [vp, vp, vp]
    lib.eg_last_cuda_error.argtypes = [vp]
    lib.eg_last_launch_count.argtypes = [vp]
    _lib = lib
    return lib


def _check(lib, status: int, ctx=None, what: str = ""):
    if status != EG_OK:
        msg = lib.eg_strerror(status).decode()
        extra = f" (cudaError {lib.eg_last_cuda_error(ctx)})" if ctx else ""
        raise EventGradError(f"{what}: {msg}{extra}")


class EventGrad:
    """One ring of ``P`` replicas held on the current CUDA device (``eg_create``)."""

    def __init__(self, P: int, layer_numel: Sequence[int], *, mode: int = THRESH_ADAPTIVE,
                 horizon: float = 1.0, history_len: int = 1, delta_init: float = 0.0,
                 delta_fixed: float = 0.0, force_first_event: bool = True,
                 topk: Optional[tuple] = None, device: Optional[int] = None, hops: int = 1):
        self._h = None
        lib = load_library()
        self._lib = lib
        if not torch.cuda.is_available():
            raise EventGradError("no CUDA device: this library has no CPU path")
        self.device = torch.device("cuda", torch.cuda.current_device() if device is None else device)
        self.P, self.T = int(P), len(layer_numel)
        self.numel = [int(n) for n in layer_numel]
        thr = ThresholdParams(mode, horizon, history_len, delta_init, delta_fixed,
                              int(force_first_event))
        tk = TopkParams(1, topk[0], topk[1]) if topk else None
        arr = (C.c_int64 * self.T)(*self.numel)
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            st = lib.eg_create(C.byref(h), TOPO_RING + int(hops) - 1, self.P, arr, self.T, C.byref(thr),
                               C.byref(tk) if tk else None)
        _check(lib, st, None, "eg_create")
        self._h = h
        offs = (C.c_int64 * self.T)()
        stride = C.c_int64()
        _check(lib, lib.eg_layout(h, offs, C.byref(stride)), h, "eg_layout")
        self.tensor_offset = list(offs)
        self.replica_stride = int(stride.value)
        self.has_topk = topk is not None

    # ------------------------------------------------------------------ lifetime
    def close(self):
        if getattr(self, "_h", None):
            self._lib.eg_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ buffers
    def empty_params(self) -> torch.Tensor:
        """A zeroed ``[P, replica_stride]`` fp32 device tensor in the library's layout."""
        return torch.zeros((self.P, self.replica_stride), dtype=torch.float32, device=self.device)

    def pack_into(self, dst: torch.Tensor, packed: torch.Tensor) -> torch.Tensor:
        """Copies a packed ``[P, N]`` tensor into the padded layout ``dst``."""
        off = 0
        for t, n in enumerate(self.numel):
            o = self.tensor_offset[t]
            dst[:, o:o + n].copy_(packed[:, off:off + n])
            off += n
        return dst

    def to_layout(self, packed: torch.Tensor) -> torch.Tensor:
        return self.pack_into(self.empty_params(), packed.to(self.device))

    def from_layout(self, padded: torch.Tensor) -> torch.Tensor:
        """Packed ``[P, N]`` copy of a tensor in the library's layout."""
        return torch.cat([padded[:, o:o + n] for o, n in zip(self.tensor_offset, self.numel)], dim=1)

    # ------------------------------------------------------------------ the step
    def step(self, params: torch.Tensor, grads: torch.Tensor, lr: float,
             stream: Optional[torch.cuda.Stream] = None):
        """``eg_step``: one iteration on ``stream`` (default: torch's current stream)."""
        assert params.is_cuda and grads.is_cuda and params.dtype == grads.dtype == torch.float32
        assert params.is_contiguous() and grads.is_contiguous()
        assert params.shape == grads.shape == (self.P, self.replica_stride)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        st = self._lib.eg_step(self._h, params.data_ptr(), grads.data_ptr(), C.c_float(lr),
                               C.c_void_p(s.cuda_stream))
        _check(self._lib, st, self._h, "eg_step")

    def enable_delivery_masks(self):
        _check(self._lib, self._lib.eg_enable_delivery_masks(self._h), self._h,
               "eg_enable_delivery_masks")

    def step_masked(self, params: torch.Tensor, grads: torch.Tensor, lr: float,
                    deliver: Optional[torch.Tensor], stream: Optional[torch.cuda.Stream] = None):
        """``eg_step_masked``: ``deliver`` is a uint8 device tensor of ``P*T`` entries or None."""
        assert params.shape == grads.shape == (self.P, self.replica_stride)
        if deliver is not None:
            assert deliver.is_cuda and deliver.dtype == torch.uint8 and deliver.is_contiguous()
            assert deliver.numel() == self.P * self.T
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        st = self._lib.eg_step_masked(self._h, params.data_ptr(), grads.data_ptr(), C.c_float(lr),
                                      deliver.data_ptr() if deliver is not None else None,
                                      C.c_void_p(s.cuda_stream))
        _check(self._lib, st, self._h, "eg_step_masked")

    def received(self) -> torch.Tensor:
        out = torch.empty((self.P, self.replica_stride), dtype=torch.float32)
        _check(self._lib, self._lib.eg_read_received(self._h, out.data_ptr()), self._h,
               "eg_read_received")
        return out

    def delivery_status(self):
        pend = np.empty(self.P * self.T, np.uint8)
        arr = C.c_uint64()
        _check(self._lib, self._lib.eg_delivery_status(self._h, pend.ctypes.data, C.byref(arr)),
               self._h, "eg_delivery_status")
        return pend.reshape(self.P, self.T), int(arr.value)

    def step_host(self, params_host: torch.Tensor, grads_host: torch.Tensor, lr: float):
        """``eg_step_host``: the same iteration with host-resident buffers."""
        assert not params_host.is_cuda and not grads_host.is_cuda
        assert params_host.is_contiguous() and grads_host.is_contiguous()
        assert params_host.shape == grads_host.shape == (self.P, self.replica_stride)
        st = self._lib.eg_step_host(self._h, params_host.data_ptr(), grads_host.data_ptr(),
                                    C.c_float(lr))
        _check(self._lib, st, self._h, "eg_step_host")

    def set_carry_norm(self, enabled: bool):
        _check(self._lib, self._lib.eg_set_carry_norm(self._h, int(enabled)), self._h,
               "eg_set_carry_norm")

    # ------------------------------------------------------------------ readers
    def stats(self) -> dict:
        m, b, e = C.c_uint64(), C.c_uint64(), C.c_uint64()
        _check(self._lib, self._lib.eg_stats(self._h, C.byref(m), C.byref(b)), self._h, "eg_stats")
        _check(self._lib, self._lib.eg_event_count(self._h, C.byref(e)), self._h, "eg_event_count")
        return {"messages": m.value, "bytes": b.value, "events": e.value}

    def last_decisions(self):
        S = self.P * self.T
        f, d, thr = np.empty(S, np.uint8), np.empty(S, np.float64), np.empty(S, np.float64)
        _check(self._lib, self._lib.eg_last_decisions(self._h, f.ctypes.data, d.ctypes.data,
                                                      thr.ctypes.data), self._h, "eg_last_decisions")
        shape = (self.P, self.T)
        return f.reshape(shape), d.reshape(shape), thr.reshape(shape)

    def thresholds(self):
        S = self.P * self.T
        d, ev = np.empty(S, np.float64), np.empty(S, np.uint64)
        _check(self._lib, self._lib.eg_thresholds(self._h, d.ctypes.data, ev.ctypes.data),
               self._h, "eg_thresholds")
        return d.reshape(self.P, self.T), ev.reshape(self.P, self.T)

    def topk_count(self, t: int) -> int:
        k = C.c_int64()
        _check(self._lib, self._lib.eg_topk_count(self._h, t, C.byref(k)), self._h, "eg_topk_count")
        return int(k.value)

    def topk_repeat_count(self) -> int:
        """Sparse messages whose guessed bin failed and that were selected again exactly."""
        n = C.c_uint64()
        _check(self._lib, self._lib.eg_topk_repeat_count(self._h, C.byref(n)), self._h, "eg_topk_repeat_count")
        return int(n.value)

    def set_quantisation(self, bits: int):
        """Quantised messages of ``bits`` bits per element (2..16; 0 or 32: full precision)."""
        _check(self._lib, self._lib.eg_set_quantisation(self._h, int(bits)), self._h, "eg_set_quantisation")

    def last_quantised(self):
        """(which, exponents) of the last step, ``[P, T]`` uint8 / int32 host arrays."""
        q = np.zeros((self.P, self.T), dtype=np.uint8)
        e = np.zeros((self.P, self.T), dtype=np.int32)
        _check(self._lib, self._lib.eg_last_quantised(self._h, q.ctypes.data, e.ctypes.data), self._h,
               "eg_last_quantised")
        return q, e

    def last_outbox(self, i: int, t: int):
        cap = max(1, self.topk_count(t))
        idx, val = np.empty(cap, np.int32), np.empty(cap, np.float32)
        n = C.c_int32()
        _check(self._lib, self._lib.eg_last_outbox(self._h, i, t, idx.ctypes.data, val.ctypes.data,
                                                   C.byref(n)), self._h, "eg_last_outbox")
        return idx[:n.value].copy(), val[:n.value].copy()

    def mailboxes(self, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Host copy of x_hat in the library's layout ``[P, replica_stride]`` (into ``out``, a
        contiguous fp32 host tensor of that shape, when given)."""
        if out is None:
            out = torch.empty((self.P, self.replica_stride), dtype=torch.float32)
        assert (not out.is_cuda and out.dtype == torch.float32 and out.is_contiguous()
                and out.shape == (self.P, self.replica_stride))
        _check(self._lib, self._lib.eg_read_mailboxes(self._h, out.data_ptr()), self._h,
               "eg_read_mailboxes")
        return out

    def average_model(self, params: torch.Tensor, consensus: bool = False,
                      stream: Optional[torch.cuda.Stream] = None):
        avg = torch.zeros(self.replica_stride, dtype=torch.float32, device=self.device)
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        c = C.c_double()
        st = self._lib.eg_average_model(self._h, params.data_ptr(), avg.data_ptr(),
                                        C.byref(c) if consensus else None,
                                        C.c_void_p(s.cuda_stream))
        _check(self._lib, st, self._h, "eg_average_model")
        return (avg, c.value) if consensus else avg

    def export_state(self) -> bytes:
        n = C.c_size_t()
        _check(self._lib, self._lib.eg_export_state(self._h, None, C.byref(n)), self._h,
               "eg_export_state")
        buf = C.create_string_buffer(n.value)
        _check(self._lib, self._lib.eg_export_state(self._h, buf, C.byref(n)), self._h,
               "eg_export_state")
        return buf.raw

    def import_state(self, blob: bytes):
        _check(self._lib, self._lib.eg_import_state(self._h, blob, len(blob)), self._h,
               "eg_import_state")

    def set_variant(self, own_last_sent: bool = False, change_of_norm: bool = False):
        """``eg_set_variant``: alternative readings of the own term / the tested quantity."""
        _check(self._lib, self._lib.eg_set_variant(self._h, int(own_last_sent), int(change_of_norm)),
               self._h, "eg_set_variant")

    def set_threshold_cap(self, alpha: float, beta: float):
        """``eg_set_threshold_cap``: thresholds bounded by sqrt(alpha * beta**k)."""
        _check(self._lib, self._lib.eg_set_threshold_cap(self._h, float(alpha), float(beta)),
               self._h, "eg_set_threshold_cap")

    def set_momentum(self, mu: Optional[float]):
        """``eg_set_momentum``: heavy-ball momentum with coefficient ``mu``; ``None`` turns it off."""
        with torch.cuda.device(self.device):
            st = self._lib.eg_set_momentum(self._h, int(mu is not None), float(mu or 0.0))
        _check(self._lib, st, self._h, "eg_set_momentum")

    def velocity(self) -> torch.Tensor:
        """Host copy of the velocities in the library's layout ``[P, replica_stride]``."""
        out = torch.empty((self.P, self.replica_stride), dtype=torch.float32)
        _check(self._lib, self._lib.eg_read_velocity(self._h, out.data_ptr()), self._h,
               "eg_read_velocity")
        return out

    def write_velocity(self, v: torch.Tensor):
        assert v.dtype == torch.float32 and v.is_contiguous() and not v.is_cuda
        assert tuple(v.shape) == (self.P, self.replica_stride)
        _check(self._lib, self._lib.eg_write_velocity(self._h, v.data_ptr()), self._h,
               "eg_write_velocity")

    def set_fused_kernel(self, kind: int):
        _check(self._lib, self._lib.eg_set_fused_kernel(self._h, int(kind)), self._h,
               "eg_set_fused_kernel")

    def set_timing(self, enabled: bool):
        _check(self._lib, self._lib.eg_set_timing(self._h, int(enabled)), self._h, "eg_set_timing")

    def kernel_times(self) -> dict:
        """{group: (total ms, timed sections)} since the last call (``eg_kernel_times``)."""
        ms = (C.c_double * len(KERNEL_GROUPS))()
        n = (C.c_uint64 * len(KERNEL_GROUPS))()
        _check(self._lib, self._lib.eg_kernel_times(self._h, ms, n), self._h, "eg_kernel_times")
        return {g: (ms[q], int(n[q])) for q, g in enumerate(KERNEL_GROUPS)}

    def selftest_wait_timeout(self) -> int:
        """``eg_selftest_wait_timeout``; returns the raw status (0 = the wait gave up as designed)."""
        s = torch.cuda.current_stream(self.device)
        return int(self._lib.eg_selftest_wait_timeout(self._h, C.c_void_p(s.cuda_stream)))

    def reset(self):
        _check(self._lib, self._lib.eg_reset(self._h), self._h, "eg_reset")

    @property
    def last_launch_count(self) -> int:
        return int(self._lib.eg_last_launch_count(self._h))


def change_norms_static(x: torch.Tensor, xhat: torch.Tensor, tensor_offset: Sequence[int],
                        layer_numel: Sequence[int], out: torch.Tensor,
                        stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """``eg_change_norms_static``: || x - x_hat || of every (replica, tensor) into ``out``
    (float64 device tensor of ``P*T`` entries) without allocating anything.  ``x`` and ``xhat``
    are ``[P, replica_stride]`` fp32 device tensors.  Raises EventGradError if the sizes exceed
    the library's fixed scratch."""
    lib = load_library()
    assert x.is_cuda and xhat.is_cuda and out.is_cuda and out.dtype == torch.float64
    assert x.dtype == xhat.dtype == torch.float32 and x.shape == xhat.shape and x.dim() == 2
    assert x.is_contiguous() and xhat.is_contiguous() and out.is_contiguous()
    T = len(layer_numel)
    assert out.numel() == x.shape[0] * T
    offs = (C.c_int64 * T)(*[int(o) for o in tensor_offset])
    nums = (C.c_int64 * T)(*[int(n) for n in layer_numel])
    s = stream if stream is not None else torch.cuda.current_stream(x.device)
    with torch.cuda.device(x.device):
        st = lib.eg_change_norms_static(x.data_ptr(), xhat.data_ptr(), int(x.shape[0]),
                                        int(x.shape[1]), offs, nums, T, out.data_ptr(),
                                        C.c_void_p(s.cuda_stream))
    _check(lib, st, None, "eg_change_norms_static")
    return out


def from_workload(wl, **overrides) -> EventGrad:
    """Context configured with a workload's threshold and Top-K recipe."""
    kw = dict(horizon=wl.horizon, history_len=wl.history_len, delta_init=wl.delta_init,
              topk=wl.topk)
    kw.update(overrides)
    return EventGrad(wl.P, wl.numel, **kw)
