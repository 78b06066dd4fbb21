"""ctypes front end of the CPU oracle (``eg_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The arithmetic lives in the C file; this module builds it with
gcc and marshals numpy arrays.  Nothing here is shared with, or imported by, the CUDA path.
"""
from __future__ import annotations

import ctypes as C
import math
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "eg_oracle.c")
_LIB = os.path.join(_HERE, "libeg_oracle.so")

ADAPTIVE = 0
FIXED = 1


def build(force: bool = False) -> str:
    """Compile the oracle (no contraction of a*b+c, OpenMP over independent segments)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp",
               "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = C.CDLL(build())
        lib.ego_create.restype = C.c_void_p
        lib.ego_create.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_int64), C.c_int, C.c_double,
                                   C.c_int, C.c_double, C.c_double, C.c_int, C.c_int,
                                   C.c_uint32, C.c_uint32]
        lib.ego_destroy.argtypes = [C.c_void_p]
        lib.ego_reset.argtypes = [C.c_void_p]
        lib.ego_set_threads.argtypes = [C.c_void_p, C.c_int]
        lib.ego_set_variant.argtypes = [C.c_void_p, C.c_int, C.c_int]
        lib.ego_set_hops.argtypes = [C.c_void_p, C.c_int]
        lib.ego_set_threshold_cap.argtypes = [C.c_void_p, C.c_double, C.c_double]
        lib.ego_set_momentum.restype = C.c_int
        lib.ego_set_momentum.argtypes = [C.c_void_p, C.c_double]
        lib.ego_velocity.restype = C.c_void_p
        lib.ego_velocity.argtypes = [C.c_void_p]
        lib.ego_set_quantisation.restype = C.c_int
        lib.ego_set_quantisation.argtypes = [C.c_void_p, C.c_int]
        for name in ("ego_quant_exponents", "ego_quantised"):
            getattr(lib, name).restype = C.c_void_p
            getattr(lib, name).argtypes = [C.c_void_p]
        lib.ego_threads_available.restype = C.c_int
        lib.ego_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float]
        lib.ego_step_masked.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p]
        lib.ego_enable_delivery_masks.argtypes = [C.c_void_p]
        lib.ego_received.restype = C.c_void_p
        lib.ego_received.argtypes = [C.c_void_p]
        lib.ego_pending.restype = C.c_void_p
        lib.ego_pending.argtypes = [C.c_void_p]
        lib.ego_received_once.restype = C.c_void_p
        lib.ego_received_once.argtypes = [C.c_void_p]
        lib.ego_arrivals.restype = C.c_uint64
        lib.ego_arrivals.argtypes = [C.c_void_p]
        lib.ego_stats.argtypes = [C.c_void_p] + [C.POINTER(C.c_uint64)] * 3
        lib.ego_iteration.restype = C.c_int64
        lib.ego_iteration.argtypes = [C.c_void_p]
        for name in ("ego_flags", "ego_norms", "ego_thresholds_used", "ego_thresholds",
                     "ego_valid", "ego_last_event_iteration", "ego_segment_events", "ego_xhat",
                     "ego_history", "ego_history_len", "ego_sent_norms"):
            getattr(lib, name).restype = C.c_void_p
            getattr(lib, name).argtypes = [C.c_void_p]
        lib.ego_topk_count.restype = C.c_int64
        lib.ego_topk_count.argtypes = [C.c_void_p, C.c_int]
        lib.ego_outbox.restype = C.c_int32
        lib.ego_outbox.argtypes = [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_void_p),
                                   C.POINTER(C.c_void_p)]
        lib.ego_average_model.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        lib.ego_consensus_distance.restype = C.c_double
        lib.ego_consensus_distance.argtypes = [C.c_void_p, C.c_void_p]
        _lib = lib
    return _lib


def threads_available() -> int:
    return int(_load().ego_threads_available())


def _view(ptr, dtype, count):
    buf = (C.c_char * (count * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype, count=count)


class Oracle:
    """One ring of ``P`` replicas of ``T`` tensors; ``step`` is one iteration of Algorithm B.

    Arrays are packed ``[P, N]`` float32 numpy arrays (C-contiguous); ``x`` is updated in place.
    """

    def __init__(self, P: int, numel: Sequence[int], *, mode: int = ADAPTIVE,
                 horizon: float = 1.0, history_len: int = 1, delta_init: float = 0.0,
                 delta_fixed: float = 0.0, force_first_event: bool = True,
                 topk: Optional[tuple] = None, threads: int = 1,
                 own_last_sent: bool = False, change_of_norm: bool = False, hops: int = 1,
                 threshold_cap: Optional[tuple] = None, momentum: Optional[float] = None,
                 quant_bits: Optional[int] = None):
        lib = _load()
        self._lib = lib
        self.P, self.T = int(P), len(numel)
        self.numel = [int(n) for n in numel]
        self.N = sum(self.numel)
        arr = (C.c_int64 * self.T)(*self.numel)
        k_num, k_den = (topk if topk else (0, 1))
        self._h = lib.ego_create(self.P, self.T, arr, mode, float(horizon), int(history_len),
                                 float(delta_init), float(delta_fixed), int(force_first_event),
                                 int(topk is not None), int(k_num), int(k_den))
        if not self._h:
            raise ValueError("ego_create rejected the arguments")
        lib.ego_set_threads(self._h, int(threads))
        lib.ego_set_variant(self._h, int(own_last_sent), int(change_of_norm))
        if lib.ego_set_hops(self._h, int(hops)):
            raise ValueError("hops out of range")
        if threshold_cap:
            lib.ego_set_threshold_cap(self._h, float(threshold_cap[0]), float(threshold_cap[1]))
        if momentum is not None and lib.ego_set_momentum(self._h, float(momentum)):
            raise ValueError("momentum must be in [0, 1)")
        if quant_bits is not None and lib.ego_set_quantisation(self._h, int(quant_bits)):
            raise ValueError("quantisation: 2..16 bits (or 32 for none), and not together with Top-K")
        self.S = self.P * self.T
        self.history_len = int(history_len)

    def close(self):
        if getattr(self, "_h", None):
            self._lib.ego_destroy(self._h)
            self._h = None

    __del__ = close

    def reset(self):
        self._lib.ego_reset(self._h)

    def set_threshold_cap(self, alpha: float, beta: float):
        """Bound sqrt(alpha * beta^k) on the thresholds from the current iteration on."""
        self._lib.ego_set_threshold_cap(self._h, float(alpha), float(beta))

    def set_threads(self, n: int):
        self._lib.ego_set_threads(self._h, int(n))

    def step(self, x: np.ndarray, g: np.ndarray, lr: float, deliver: Optional[np.ndarray] = None):
        """One iteration; ``deliver`` ([P, T] uint8, optional) says whose outstanding messages
        arrive in this iteration (default: all, i.e. synchronous delivery)."""
        assert x.dtype == np.float32 and g.dtype == np.float32
        assert x.flags.c_contiguous and g.flags.c_contiguous
        assert x.shape == (self.P, self.N) and g.shape == (self.P, self.N)
        if deliver is None:
            self._lib.ego_step(self._h, x.ctypes.data, g.ctypes.data, C.c_float(lr))
        else:
            d = np.ascontiguousarray(deliver, dtype=np.uint8)
            assert d.size == self.S
            self._lib.ego_step_masked(self._h, x.ctypes.data, g.ctypes.data, C.c_float(lr), d.ctypes.data)

    def enable_delivery_masks(self):
        self._lib.ego_enable_delivery_masks(self._h)

    def received(self) -> np.ndarray:
        """Copy of what the neighbours hold of every replica (== xhat() under synchronous delivery)."""
        return _view(self._lib.ego_received(self._h), np.float32, self.P * self.N).reshape(
            self.P, self.N).copy()

    def pending(self):
        p = self._lib.ego_pending(self._h)
        if not p:
            return np.zeros((self.P, self.T), np.uint8)
        return _view(p, np.uint8, self.S).reshape(self.P, self.T).copy()

    def received_once(self):
        """Per (replica, tensor): the neighbours have received this tensor at least once."""
        return _view(self._lib.ego_received_once(self._h), np.uint8, self.S).reshape(self.P, self.T).copy()

    @property
    def arrivals(self) -> int:
        return int(self._lib.ego_arrivals(self._h))

    @property
    def iteration(self) -> int:
        return int(self._lib.ego_iteration(self._h))

    def stats(self):
        m, b, e = C.c_uint64(), C.c_uint64(), C.c_uint64()
        self._lib.ego_stats(self._h, C.byref(m), C.byref(b), C.byref(e))
        return {"messages": m.value, "bytes": b.value, "events": e.value}

    def _seg(self, fn, dtype):
        return _view(getattr(self._lib, fn)(self._h), dtype, self.S).reshape(self.P, self.T).copy()

    def flags(self):
        return self._seg("ego_flags", np.uint8)

    def norms(self):
        return self._seg("ego_norms", np.float64)

    def thresholds_used(self):
        """Threshold each (replica, tensor) was tested against in the last step."""
        return self._seg("ego_thresholds_used", np.float64)

    def thresholds(self):
        """Threshold in force after the last step."""
        return self._seg("ego_thresholds", np.float64)

    def sent_norms(self):
        """||x|| of every (replica, tensor) at its last event (change-of-norm variant)."""
        return self._seg("ego_sent_norms", np.float64)

    def valid(self):
        return self._seg("ego_valid", np.uint8)

    def last_event_iteration(self):
        return self._seg("ego_last_event_iteration", np.int64)

    def segment_events(self):
        return self._seg("ego_segment_events", np.uint64)

    def history(self):
        """(slopes [P, T, H] oldest first, number of slopes kept [P, T])."""
        H = self.history_len
        h = _view(self._lib.ego_history(self._h), np.float64, self.S * H).reshape(
            self.P, self.T, H).copy()
        return h, self._seg("ego_history_len", np.int32)

    def xhat(self) -> np.ndarray:
        """Copy of the mailboxes (last communicated values), packed ``[P, N]``."""
        return _view(self._lib.ego_xhat(self._h), np.float32, self.P * self.N).reshape(
            self.P, self.N).copy()

    def velocity(self) -> Optional[np.ndarray]:
        """Copy of the momentum buffers, packed ``[P, N]`` (None when momentum is off)."""
        p = self._lib.ego_velocity(self._h)
        if not p:
            return None
        return _view(p, np.float32, self.P * self.N).reshape(self.P, self.N).copy()

    def quant_exponents(self) -> Optional[np.ndarray]:
        """Scale exponents E of the last step's quantised messages, ``[P, T]`` int32 (None when
        quantisation is off); only meaningful where ``quantised()`` is set."""
        p = self._lib.ego_quant_exponents(self._h)
        if not p:
            return None
        return _view(p, np.int32, self.S).reshape(self.P, self.T).copy()

    def quantised(self) -> Optional[np.ndarray]:
        """Which (replica, tensor) pairs sent a quantised message in the last step."""
        p = self._lib.ego_quantised(self._h)
        if not p:
            return None
        return _view(p, np.uint8, self.S).reshape(self.P, self.T).copy()

    def topk_count(self, t: int) -> int:
        return int(self._lib.ego_topk_count(self._h, t))

    def outbox(self, i: int, t: int):
        """(indices, values) of the sparse message tensor ``t`` of replica ``i`` sent in the
        last step; empty arrays if it sent none."""
        pi, pv = C.c_void_p(), C.c_void_p()
        n = self._lib.ego_outbox(self._h, i, t, C.byref(pi), C.byref(pv))
        if n <= 0:
            return np.zeros(0, np.int32), np.zeros(0, np.float32)
        return _view(pi.value, np.int32, n).copy(), _view(pv.value, np.float32, n).copy()

    def average_model(self, x: np.ndarray) -> np.ndarray:
        out = np.empty(self.N, np.float32)
        self._lib.ego_average_model(self._h, x.ctypes.data, out.ctypes.data)
        return out

    def consensus_distance(self, x: np.ndarray) -> float:
        return float(self._lib.ego_consensus_distance(self._h, x.ctypes.data))


def from_workload(wl, *, threads: int = 1, **overrides) -> Oracle:
    """Oracle configured with a workload's threshold and Top-K recipe."""
    kw = dict(horizon=wl.horizon, history_len=wl.history_len, delta_init=wl.delta_init,
              topk=wl.topk, threads=threads)
    kw.update(overrides)
    return Oracle(wl.P, wl.numel, **kw)
