"""Seeded synthetic workloads for the event-triggered communication step.

This module only produces *inputs*: parameter-set shapes, initial parameters and
per-step gradients.  It holds none of the method's arithmetic (no norm, trigger,
averaging or update) and imports neither the CUDA binding nor the CPU oracle, so
both can be fed from it.

The parameter sets stand in for the ResNet-18/CIFAR-10 training tensors of the
paper's experiments (Section 7 "Results"): only the shapes, sizes and value
scales are reproduced; the data set and trained weights are not needed.

Random numbers come from a counter-based generator written with integer tensor
operations only, so the very same code yields identical bits on a CPU tensor
and on a CUDA tensor:

* bits: SplitMix64 (Steele, Lea & Flood, "Fast splittable pseudorandom number
  generators", OOPSLA 2014): ``state += GAMMA; out = finalise(state)``.
* one approximately normal deviate per element: the sum of eight 16-bit fields
  of two consecutive outputs (an Irwin-Hall(8) variate), centred in integers,
  converted exactly to fp32 and multiplied once by an fp32 scale.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import torch

MASTER_SEED = 20210307
STREAM_INIT = 1
STREAM_GRAD = 2
STREAM_LAYER_SCALE = 3

_M64 = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

#: mean and standard deviation of the sum of eight independent uniform draws from
#: {0, ..., 65535}
IH8_MEAN = 4 * 65535
IH8_STD = math.sqrt(8.0 * (65536.0 ** 2 - 1.0) / 12.0)


# --------------------------------------------------------------------------------------
# integer generator: pure-Python definition (for scalars) and tensor form (for arrays)
# --------------------------------------------------------------------------------------
def _finalise_py(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def stream_base(seed: int, stream: int, *counters: int) -> int:
    """64-bit starting state for the element stream named by (seed, stream, counters)."""
    z = _finalise_py(seed ^ (stream * _GAMMA))
    for c in counters:
        z = _finalise_py((z + (int(c) + 1) * _GAMMA) & _M64)
    return z


def _signed(c: int) -> int:
    c &= _M64
    return c - (1 << 64) if c >= (1 << 63) else c


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of an int64 tensor holding 64 raw bits."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _finalise_t(z: torch.Tensor) -> torch.Tensor:
    z = (z ^ _lsr(z, 30)) * _signed(_C1)
    z = (z ^ _lsr(z, 27)) * _signed(_C2)
    return z ^ _lsr(z, 31)


def _fields16(h: torch.Tensor) -> torch.Tensor:
    return (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + _lsr(h, 48)


def ih8_integers(base: int, start: int, count: int, device) -> torch.Tensor:
    """Centred Irwin-Hall(8) integers for elements ``start .. start+count-1`` of a stream.

    Element ``e`` uses SplitMix64 outputs number ``2e+1`` and ``2e+2`` of the stream
    whose state starts at ``base``.  Returns int64 values in ``[-262140, 262140]``.
    """
    e = torch.arange(start, start + count, dtype=torch.int64, device=device)
    s1 = (2 * e + 1) * _signed(_GAMMA) + _signed(base)
    s2 = s1 + _signed(_GAMMA)
    total = _fields16(_finalise_t(s1)) + _fields16(_finalise_t(s2))
    return total - IH8_MEAN


def ih8_integers_py(base: int, e: int) -> int:
    """Pure-Python restatement of :func:`ih8_integers` for one element (test pin)."""
    def f16(h):
        return (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + (h >> 48)
    s1 = (base + (2 * e + 1) * _GAMMA) & _M64
    s2 = (s1 + _GAMMA) & _M64
    return f16(_finalise_py(s1)) + f16(_finalise_py(s2)) - IH8_MEAN


def uniform01_py(base: int, e: int) -> float:
    """One uniform double in [0, 1) for element ``e`` of a stream (53 random bits)."""
    s1 = (base + (2 * e + 1) * _GAMMA) & _M64
    return (_finalise_py(s1) >> 11) / float(1 << 53)


# --------------------------------------------------------------------------------------
# parameter sets
# --------------------------------------------------------------------------------------
@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: tuple
    kind: str  # "weight" | "bn_scale" | "bn_shift" | "bias"

    @property
    def numel(self) -> int:
        n = 1
        for s in self.shape:
            n *= s
        return n

    @property
    def fan_in(self) -> int:
        n = 1
        for s in self.shape[1:]:
            n *= s
        return n


def _conv_bn(name, cout, cin, k) -> List[TensorSpec]:
    return [TensorSpec(f"{name}.conv", (cout, cin, k, k), "weight"),
            TensorSpec(f"{name}.bn.scale", (cout,), "bn_scale"),
            TensorSpec(f"{name}.bn.shift", (cout,), "bn_shift")]


def mlp_tensors() -> List[TensorSpec]:
    dims = [784, 64, 32, 10]
    out = []
    for l in range(3):
        # stored as (out, in) so fan_in is the input width
        out.append(TensorSpec(f"fc{l}.weight", (dims[l + 1], dims[l]), "weight"))
        out.append(TensorSpec(f"fc{l}.bias", (dims[l + 1],), "bias"))
    return out


def resnet20_tensors() -> List[TensorSpec]:
    out = _conv_bn("stem", 16, 3, 3)
    cin = 16
    for s, w in enumerate((16, 32, 64)):
        for b in range(3):
            out += _conv_bn(f"s{s}.b{b}.c1", w, cin, 3)
            out += _conv_bn(f"s{s}.b{b}.c2", w, w, 3)
            cin = w
    out.append(TensorSpec("fc.weight", (10, 64), "weight"))
    out.append(TensorSpec("fc.bias", (10,), "bias"))
    return out


def resnet18_cifar_tensors() -> List[TensorSpec]:
    out = _conv_bn("stem", 64, 3, 3)
    cin = 64
    for s, w in enumerate((64, 128, 256, 512)):
        for b in range(2):
            out += _conv_bn(f"s{s}.b{b}.c1", w, cin, 3)
            out += _conv_bn(f"s{s}.b{b}.c2", w, w, 3)
            if b == 0 and cin != w:
                out += _conv_bn(f"s{s}.b{b}.proj", w, cin, 1)
            cin = w
    out.append(TensorSpec("fc.weight", (10, 512), "weight"))
    out.append(TensorSpec("fc.bias", (10,), "bias"))
    return out


def resnet50_tensors() -> List[TensorSpec]:
    out = _conv_bn("stem", 64, 3, 7)
    cin = 64
    for s, (w, nb) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3))):
        for b in range(nb):
            out += _conv_bn(f"s{s}.b{b}.c1", w, cin, 1)
            out += _conv_bn(f"s{s}.b{b}.c2", w, w, 3)
            out += _conv_bn(f"s{s}.b{b}.c3", 4 * w, w, 1)
            if b == 0:
                out += _conv_bn(f"s{s}.b{b}.proj", 4 * w, cin, 1)
            cin = 4 * w
    out.append(TensorSpec("fc.weight", (1000, 2048), "weight"))
    out.append(TensorSpec("fc.bias", (1000,), "bias"))
    return out


@dataclass
class Workload:
    """One configuration: a ring of ``P`` replicas of a parameter set plus the run recipe."""
    name: str
    P: int
    tensors: List[TensorSpec]
    steps: int
    lr: float
    grad_law: str               # "inv_sqrt" | "per_layer_uniform" | "boosted_tenth" | "const"
    grad_sigma: float
    init_law: str = "kaiming"   # "kaiming" | "normal_all"
    init_sigma: float = 0.05
    topk: Optional[tuple] = None  # (k_num, k_den) or None for dense messages
    seed: int = MASTER_SEED
    # adaptive threshold recipe of the paper's experiments: horizon 1 (Section 7)
    horizon: float = 1.0
    history_len: int = 1
    delta_init: float = 0.0
    _layer_scale: Optional[List[float]] = field(default=None, repr=False)

    @property
    def T(self) -> int:
        return len(self.tensors)

    @property
    def numel(self) -> List[int]:
        return [t.numel for t in self.tensors]

    @property
    def N(self) -> int:
        return sum(self.numel)

    # ---------------------------------------------------------------- scales
    def layer_scale(self) -> List[float]:
        """Per-tensor multiplier u_t ~ U(0.5, 2), drawn once (law "per_layer_uniform")."""
        if self._layer_scale is None:
            base = stream_base(self.seed, STREAM_LAYER_SCALE)
            self._layer_scale = [0.5 + 1.5 * uniform01_py(base, t) for t in range(self.T)]
        return self._layer_scale

    def grad_sigmas(self, k: int) -> List[float]:
        """Standard deviation of the step-``k`` gradient of every tensor."""
        if self.grad_law == "inv_sqrt":
            s = self.grad_sigma / math.sqrt(k + 1.0)
            return [s] * self.T
        if self.grad_law == "per_layer_uniform":
            return [self.grad_sigma * u for u in self.layer_scale()]
        if self.grad_law == "boosted_tenth":
            return [self.grad_sigma * (10.0 if t % 10 == 0 else 1.0) for t in range(self.T)]
        if self.grad_law == "const":
            return [self.grad_sigma] * self.T
        raise ValueError(self.grad_law)

    def init_sigmas(self) -> List[Optional[float]]:
        """Std-dev of the initial value of every tensor; ``None`` marks a constant fill."""
        out = []
        for t in self.tensors:
            if self.init_law == "normal_all":
                out.append(self.init_sigma)
            elif t.kind == "weight":
                out.append(math.sqrt(2.0 / t.fan_in))
            else:
                out.append(None)
        return out

    # ---------------------------------------------------------------- tensors
    def _scale_vector(self, sigmas: Sequence[Optional[float]], device) -> torch.Tensor:
        per_tensor = torch.tensor(
            [0.0 if s is None else s / IH8_STD for s in sigmas], dtype=torch.float64
        ).to(torch.float32)
        counts = torch.tensor(self.numel, dtype=torch.int64)
        return torch.repeat_interleave(per_tensor, counts).to(device)

    def init_params(self, device="cpu") -> torch.Tensor:
        """Initial parameters, packed ``[P, N]`` fp32; every replica starts from the same
        values (the usual data-parallel start)."""
        base = stream_base(self.seed, STREAM_INIT)
        z = ih8_integers(base, 0, self.N, device).to(torch.float32)
        row = z * self._scale_vector(self.init_sigmas(), device)
        off = 0
        for t in self.tensors:
            if self.init_law != "normal_all" and t.kind == "bn_scale":
                row[off:off + t.numel] = 1.0
            off += t.numel
        return row.unsqueeze(0).repeat(self.P, 1).contiguous()

    def grads(self, k: int, device="cpu", out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Gradients of step ``k``, packed ``[P, N]`` fp32."""
        if out is None:
            out = torch.empty((self.P, self.N), dtype=torch.float32, device=device)
        scale = self._scale_vector(self.grad_sigmas(k), device)
        for i in range(self.P):
            base = stream_base(self.seed, STREAM_GRAD, k, i)
            z = ih8_integers(base, 0, self.N, device).to(torch.float32)
            torch.mul(z, scale, out=out[i])
        return out


def config(index: int) -> List[Workload]:
    """The run(s) of configuration ``index`` (1-based).  Configurations 4 and 5 hold more
    than one run (two Top-K fractions; dense and Top-K)."""
    if index == 1:
        return [Workload("mlp_p4_dense", 4, mlp_tensors(), steps=20, lr=0.1,
                         grad_law="inv_sqrt", grad_sigma=0.01,
                         init_law="normal_all", init_sigma=0.05)]
    if index == 2:
        return [Workload("resnet20_p8_dense", 8, resnet20_tensors(), steps=200, lr=0.1,
                         grad_law="per_layer_uniform", grad_sigma=1e-3)]
    if index == 3:
        return [Workload("resnet18_p16_dense", 16, resnet18_cifar_tensors(), steps=100, lr=0.05,
                         grad_law="inv_sqrt", grad_sigma=1e-3)]
    if index == 4:
        return [Workload(f"resnet18_p8_top{pct}pct", 8, resnet18_cifar_tensors(), steps=100,
                         lr=0.05, grad_law="inv_sqrt", grad_sigma=1e-3, topk=(pct, 100))
                for pct in (1, 10)]
    if index == 5:
        return [Workload("resnet50_p64_dense", 64, resnet50_tensors(), steps=50, lr=0.05,
                         grad_law="boosted_tenth", grad_sigma=5e-4),
                Workload("resnet50_p64_top1pct", 64, resnet50_tensors(), steps=50, lr=0.05,
                         grad_law="boosted_tenth", grad_sigma=5e-4, topk=(1, 100))]
    raise ValueError(f"no configuration {index}")


def synthetic(P: int, numel: Sequence[int], steps: int = 8, lr: float = 0.05,
              grad_sigma: float = 1e-3, topk: Optional[tuple] = None, seed: int = 1234,
              grad_law: str = "inv_sqrt", history_len: int = 1,
              horizon: float = 1.0) -> Workload:
    """A small ragged parameter set for unit tests: tensor ``t`` has ``numel[t]`` elements."""
    tensors = [TensorSpec(f"t{t}", (n,), "weight") for t, n in enumerate(numel)]
    return Workload(f"synthetic_p{P}", P, tensors, steps=steps, lr=lr, grad_law=grad_law,
                    grad_sigma=grad_sigma, init_law="normal_all", init_sigma=0.05, topk=topk,
                    seed=seed, history_len=history_len, horizon=horizon)


def distinct_init_params(wl: Workload, device="cpu") -> torch.Tensor:
    """Initial parameters that differ between replicas (for invariant tests)."""
    out = torch.empty((wl.P, wl.N), dtype=torch.float32, device=device)
    scale = wl._scale_vector([wl.init_sigma] * wl.T, device)
    for i in range(wl.P):
        base = stream_base(wl.seed, STREAM_INIT, i)
        out[i] = ih8_integers(base, 0, wl.N, device).to(torch.float32) * scale
    return out
