"""Lock-step comparison of the CUDA library (through its C ABI) with the CPU oracle.

Both sides are fed the same seeded inputs, step by step.  Compared every step:
trigger flags (bit-exact, except decisions whose norm lies within 1e-6 relative of the
threshold, which are reported and followed by a re-synchronisation), change norms and
thresholds (1e-12 relative: only the summation order differs), message / byte / event
counters (exact), Top-K messages (exact index sets and values), mailboxes, parameters and,
with momentum, the velocities.

Tensors never interact with each other in the method, so at sizes where the oracle would be
too slow it is run on a subset of the tensors (``tensors=[...]``) while the CUDA library runs
the whole configuration.
"""
from __future__ import annotations

import os
import time
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

from oracle import eg_oracle as eo
from paper_2103_07454_b200 import binding as B
from paper_2103_07454_b200 import workload as W

PARAM_RTOL = 1e-5      # parameters: 1e-5 relative in fp32
NEAR_BAND = 1e-6       # decisions this close to the threshold are reported, not failed
UNIT_ROUNDOFF = 2.0 ** -53


def norm_rtol(numel) -> np.ndarray:
    """Tolerance on || x - x_hat ||: the oracle adds the n squares one after the other, the
    kernels add them as a tree; each is within (n-1)*u relative of the exact sum of these
    non-negative terms (standard bound for recursive summation), so the two norms (square
    roots halve the error) agree within n*u.  Floor: a few roundings."""
    return np.maximum(np.asarray(numel, dtype=np.float64) * UNIT_ROUNDOFF, 8 * UNIT_ROUNDOFF)


@dataclass
class Report:
    steps: int = 0
    events: int = 0
    sparse_checked: int = 0
    near_threshold: List[tuple] = field(default_factory=list)
    max_param_rel: float = 0.0
    max_norm_rel: float = 0.0
    params_bit_exact: bool = True
    launches: int = 0
    topk_repeats: int = 0
    quantised_checked: int = 0
    seconds: dict = field(default_factory=lambda: {"inputs": 0.0, "oracle": 0.0, "compare": 0.0})


def oracle_threads() -> int:
    return max(1, min(eo.threads_available(), int(os.environ.get("EG_ORACLE_THREADS", "64"))))


def _columns(numel: Sequence[int], tensors: Sequence[int]) -> np.ndarray:
    off = np.concatenate([[0], np.cumsum(numel)])
    return np.concatenate([np.arange(off[t], off[t] + numel[t]) for t in tensors])


def _counters_from_events(events: np.ndarray, numel, k_t, degree: int, quant_bits: int = 0) -> dict:
    """Message, byte and event totals implied by the number of events of every (replica,
    tensor): `degree` messages per event, 4 n_t bytes for a dense message, 8 K_t for a Top-K
    message, 4 + ceil(n_t b / 8) for a quantised one and 4 + 4 K_t + ceil(K_t b / 8) for a quantised
    Top-K one (finite changes), the first message of a tensor always being dense."""
    ev = np.asarray(events, dtype=np.int64)
    n = np.asarray(numel, dtype=np.int64)[None, :]
    if quant_bits and k_t is not None:
        kt = np.asarray(k_t, dtype=np.int64)[None, :]
        payload = np.where(ev > 0, 4 * n + (4 + 4 * kt + (kt * quant_bits + 7) // 8) * (ev - 1), 0)
    elif quant_bits:
        payload = np.where(ev > 0, 4 * n + (4 + (n * quant_bits + 7) // 8) * (ev - 1), 0)
    elif k_t is None:
        payload = 4 * n * ev
    else:
        kt = np.asarray(k_t, dtype=np.int64)[None, :]
        payload = np.where(ev > 0, 4 * n + 8 * kt * (ev - 1), 0)
    return {"messages": int(degree * ev.sum()), "bytes": int(degree * payload.sum()), "events": int(ev.sum())}


# Checkpoint header, 8-byte words: magic, P, T, H, stride, N, topk, k_num, k_den, variant, step,
# 3 counters, hops, mode, force_first, delivery, velocity, 6 doubles (horizon, delta_init,
# delta_fixed, bound alpha / beta, mu), arrivals, bits of a quantised message.
HEADER_WORDS = 27


def resynchronise(eg: B.EventGrad, o: eo.Oracle, x_dev: torch.Tensor, x_host: np.ndarray, delivery: bool = False):
    """After a reported near-threshold disagreement: overwrite the CUDA context's state and
    parameters with the oracle's (through the checkpoint interface) so the comparison of the
    following steps stays meaningful."""
    blob = bytearray(eg.export_state())
    S, H = eg.P * eg.T, o.history_len
    head = np.frombuffer(blob, dtype=np.int64, count=HEADER_WORDS)
    st = o.stats()
    head[10] = o.iteration
    head[11:14] = [st["messages"], st["bytes"], st["events"]]
    head[25] = o.arrivals
    pos = HEADER_WORDS * 8

    def put(arr, dtype):
        nonlocal pos
        raw = np.ascontiguousarray(arr, dtype=dtype).tobytes()
        blob[pos:pos + len(raw)] = raw
        pos += len(raw)

    def put_layout(packed):
        padded = torch.zeros((eg.P, eg.replica_stride), dtype=torch.float32)
        eg.pack_into(padded, torch.from_numpy(packed))
        put(padded.numpy(), np.float32)

    hist, hist_len = o.history()
    put(o.thresholds(), np.float64)
    put(o.last_event_iteration(), np.int64)
    put(hist_len, np.int32)
    put(o.valid(), np.uint8)
    put(o.segment_events(), np.uint64)
    put(hist, np.float64)
    put(o.sent_norms(), np.float64)
    put_layout(o.xhat())
    if delivery:
        put_layout(o.received())
        put(o.pending(), np.uint8)
        put(o.received_once(), np.uint8)
    if o.velocity() is not None:
        put_layout(o.velocity())
    assert pos == len(blob)
    eg.import_state(bytes(blob))
    eg.pack_into(x_dev, torch.from_numpy(x_host).to(x_dev.device))


def lockstep(wl: W.Workload, *, steps: Optional[int] = None, init: str = "workload",
             gen_device: str = "cuda", tensors: Optional[Sequence[int]] = None,
             carry: bool = False, check_every: int = 1, oracle_kw: Optional[dict] = None,
             eg_kw: Optional[dict] = None, outbox_samples: int = 8, grad_hook=None,
             fused_kernel: int = B.FUSED_PIPELINED, deliver_fn=None) -> Report:
    steps = wl.steps if steps is None else steps
    dev = torch.device("cuda")
    full = tensors is None
    tensors = list(range(wl.T)) if full else list(tensors)
    sub_numel = [wl.numel[t] for t in tensors]
    cols = None if full else torch.from_numpy(_columns(wl.numel, tensors)).to(dev)

    okw = dict(horizon=wl.horizon, history_len=wl.history_len, delta_init=wl.delta_init,
               topk=wl.topk, threads=oracle_threads())
    okw.update(oracle_kw or {})
    o = eo.Oracle(wl.P, sub_numel, **okw)
    ekw = dict(eg_kw or {})
    cap = okw.get("threshold_cap")
    if "hops" in okw:
        ekw.setdefault("hops", okw["hops"])
    ekw.pop("threshold_cap", None)
    ekw.pop("own_last_sent", None)
    ekw.pop("change_of_norm", None)
    ekw.pop("momentum", None)
    ekw.pop("quant_bits", None)
    for key in ("mode", "delta_fixed", "force_first_event", "horizon", "history_len", "delta_init"):
        if key in okw and key not in ekw:
            ekw[key] = okw[key]
    eg = B.from_workload(wl, **ekw)
    eg.set_carry_norm(carry)
    eg.set_fused_kernel(fused_kernel)
    if deliver_fn is not None:
        eg.enable_delivery_masks()
        o.enable_delivery_masks()
    eg.set_variant(bool(okw.get("own_last_sent")), bool(okw.get("change_of_norm")))
    if cap:
        eg.set_threshold_cap(*cap)
    if okw.get("momentum") is not None:
        eg.set_momentum(okw["momentum"])
    if okw.get("quant_bits") is not None:
        eg.set_quantisation(okw["quant_bits"])

    x0 = (W.distinct_init_params(wl, gen_device) if init == "distinct" else wl.init_params(gen_device)).to(dev)
    x_dev = eg.to_layout(x0)
    x_host = (x0 if full else x0[:, cols]).cpu().numpy().copy()
    del x0
    ncol = x_host.shape[1]
    # Large runs move their data between device and host through page-locked buffers, and the
    # inputs of iteration k+1 are produced on the device while the oracle works on iteration k.
    big = wl.P * ncol >= (1 << 24)
    g_devs = [eg.empty_params(), eg.empty_params()]
    g_pins = [torch.empty((wl.P, ncol), dtype=torch.float32, pin_memory=big) for _ in range(2)]
    chk_pin = torch.empty((wl.P, ncol), dtype=torch.float32, pin_memory=True) if big else None
    box_pin = torch.empty((wl.P, eg.replica_stride), dtype=torch.float32, pin_memory=True) if big else None
    rep = Report()
    sub_off = np.concatenate([[0], np.cumsum(sub_numel)])
    degree = min(2 * int(okw.get("hops", 1)), wl.P - 1)
    all_kt = [eg.topk_count(t) for t in range(wl.T)] if wl.topk else None
    sub_kt = [all_kt[t] for t in tensors] if wl.topk else None
    rng = np.random.default_rng(7)

    def gpu_sub(padded: torch.Tensor) -> np.ndarray:
        """The oracle's tensors of a device array in the library's layout, packed, on the host."""
        parts = [padded[:, eg.tensor_offset[t]:eg.tensor_offset[t] + wl.numel[t]] for t in tensors]
        packed = torch.cat(parts, dim=1)
        if chk_pin is None:
            return packed.cpu().numpy()
        chk_pin.copy_(packed)
        return chk_pin.numpy()

    def host_sub(padded: np.ndarray, packed: np.ndarray) -> bool:
        """Bit equality of the oracle's tensors of a host array in the library's layout with a packed array."""
        return all(np.array_equal(padded[:, eg.tensor_offset[t]:eg.tensor_offset[t] + wl.numel[t]].view(np.uint32),
                                  packed[:, sub_off[q]:sub_off[q + 1]].view(np.uint32))
                   for q, t in enumerate(tensors))

    def produce(k):
        """Inputs of iteration k: gradients in the library's layout on the device, and the
        oracle's columns of them on the host (ready once the returned event has completed)."""
        slot = k & 1
        g = wl.grads(k, gen_device)
        if grad_hook is not None:
            g = grad_hook(k, g)
        g = g.to(dev)
        eg.pack_into(g_devs[slot], g)
        g_pins[slot].copy_(g if full else g[:, cols], non_blocking=True)
        ready = torch.cuda.Event()
        ready.record()
        return g_devs[slot], g_pins[slot].numpy(), ready

    t_mark = time.perf_counter()

    def lap(name):
        nonlocal t_mark
        now = time.perf_counter()
        rep.seconds[name] += now - t_mark
        t_mark = now

    ahead = produce(0)
    for k in range(steps):
        g_dev, g_host, ready = ahead
        ready.synchronize()
        sent_pre = o.sent_norms() if okw.get("change_of_norm") else None
        mask = None if deliver_fn is None else deliver_fn(k)          # [P, T] uint8 or None
        if deliver_fn is None:
            eg.step(x_dev, g_dev, wl.lr)
        else:
            eg.step_masked(x_dev, g_dev, wl.lr,
                           None if mask is None else torch.from_numpy(np.ascontiguousarray(mask)).to(dev))
        if k + 1 < steps:
            ahead = produce(k + 1)          # enqueued behind the step; runs while the oracle works
        lap("inputs")
        o.step(x_host, g_host, wl.lr,
               deliver=None if mask is None else np.ascontiguousarray(mask[:, tensors]))
        lap("oracle")
        rep.launches += eg.last_launch_count
        rep.steps += 1
        if (k % check_every) and k != steps - 1 and k >= 8:
            continue        # the first steps (where most events happen) are always checked
        # (what follows synchronises with the device; its time is booked under "compare")

        f_g, d_g, thr_g = eg.last_decisions()
        f_g, d_g, thr_g = f_g[:, tensors], d_g[:, tensors], thr_g[:, tensors]
        f_o, d_o, thr_o = o.flags(), o.norms(), o.thresholds_used()
        tol = 2 * norm_rtol(sub_numel)[None, :]     # thresholds are norms divided by integers
        if sent_pre is not None:
            # d = | ||x|| - ||x sent|| | cancels: its error is that of the two norms, so the
            # relative tolerance grows by their size over d (also for the thresholds made of d)
            tol = np.maximum(tol, 1e-9)
        fin = np.isfinite(thr_o)
        assert np.array_equal(fin, np.isfinite(thr_g)) and np.array_equal(thr_g[~fin], thr_o[~fin])
        tol = np.broadcast_to(tol, thr_o.shape)
        assert np.all(np.abs(thr_g[fin] - thr_o[fin]) <= tol[fin] * np.abs(thr_o[fin])), f"thresholds, step {k}"
        scale = np.abs(d_o) if sent_pre is None else np.abs(d_o) + 2 * sent_pre + 2 * np.abs(d_o)
        rel = np.abs(d_g - d_o) / np.maximum(scale, 1e-300) / norm_rtol(sub_numel)[None, :]
        rep.max_norm_rel = max(rep.max_norm_rel, float(rel.max()))
        assert rel.max() <= 1.0, (
            f"norms, step {k}: {rel.max():.3e} x tolerance at {np.unravel_index(rel.argmax(), rel.shape)} "
            f"cuda {d_g.flat[rel.argmax()]!r} oracle {d_o.flat[rel.argmax()]!r}")
        bad = f_g != f_o
        if bad.any():
            near = np.abs(d_o - thr_o) <= NEAR_BAND * np.abs(thr_o)
            assert near[bad].all(), f"trigger flags differ away from the threshold, step {k}"
            rep.near_threshold += [(k, int(i), int(tensors[t])) for i, t in zip(*np.nonzero(bad))]
            assert full, "near-threshold disagreement in a tensor-subset run cannot be re-synchronised"
            resynchronise(eg, o, x_dev, x_host, delivery=deliver_fn is not None)
            continue
        rep.events += int(f_o.sum())

        if full:
            so, sg = o.stats(), eg.stats()
            assert so == sg, f"counters, step {k}: oracle {so} cuda {sg}"
        _, ev_g = eg.thresholds()
        assert np.array_equal(ev_g[:, tensors], o.segment_events()), f"per-tensor events, step {k}"
        if not full:
            # The oracle's counters cover its tensors only.  Both totals follow from the events
            # per (replica, tensor) -- every event is one message per distinct neighbour, the
            # first message of a tensor is dense, later ones carry K_t pairs under Top-K -- so
            # the oracle's counters must equal that sum over its tensors and the library's the
            # same sum over all tensors, the per-tensor events of the sample being equal.
            so, sg = o.stats(), eg.stats()
            qb = okw.get("quant_bits") or 0
            qb = 0 if qb == 32 else qb
            assert so == _counters_from_events(o.segment_events(), sub_numel, sub_kt, degree, qb), f"step {k}"
            assert sg == _counters_from_events(ev_g, wl.numel, all_kt, degree, qb), f"counters, step {k}"
        dl_g, _ = eg.thresholds()
        dl_g, dl_o = dl_g[:, tensors], o.thresholds()
        fin = np.isfinite(dl_o)
        assert np.all(np.abs(dl_g[fin] - dl_o[fin]) <= tol[fin] * np.abs(dl_o[fin])), f"delta, step {k}"

        if wl.topk:
            valid_events = np.argwhere(f_o.astype(bool))
            if len(valid_events) > outbox_samples:
                valid_events = valid_events[rng.choice(len(valid_events), outbox_samples, replace=False)]
            for i, ts in valid_events:
                idx_o, val_o = o.outbox(int(i), int(ts))
                idx_g, val_g = eg.last_outbox(int(i), int(tensors[ts]))
                assert np.array_equal(idx_o, idx_g), f"Top-K index set, step {k}, replica {i}, tensor {tensors[ts]}"
                assert np.array_equal(val_o.view(np.uint32), val_g.view(np.uint32)), "Top-K values"
                rep.sparse_checked += int(len(idx_o) > 0)

        x_g = gpu_sub(x_dev)
        same = np.array_equal(x_g.view(np.uint32), x_host.view(np.uint32))
        rep.params_bit_exact &= bool(same)
        if not same:
            err = np.abs(x_g.astype(np.float64) - x_host) / np.maximum(np.abs(x_host), 1e-30)
            rep.max_param_rel = max(rep.max_param_rel, float(err.max()))
            assert rep.max_param_rel <= PARAM_RTOL, f"parameters, step {k}: rel err {rep.max_param_rel}"
        if box_pin is None:
            xh_g = gpu_sub(eg.mailboxes().to(dev))
            assert np.array_equal(xh_g.view(np.uint32), o.xhat().view(np.uint32)), f"mailboxes, step {k}"
        else:
            assert host_sub(eg.mailboxes(out=box_pin).numpy(), o.xhat()), f"mailboxes, step {k}"
        if okw.get("quant_bits") not in (None, 0, 32):
            q_g, e_g = eg.last_quantised()
            q_o, e_o = o.quantised(), o.quant_exponents()
            # (the library tells a message that went out in full because its change was not finite
            #  from one that was never a candidate; the oracle marks both 0)
            assert np.array_equal(q_g[:, tensors] == 1, q_o == 1), f"which messages are quantised, step {k}"
            assert np.array_equal(e_g[:, tensors][q_o == 1], e_o[q_o == 1]), f"scale exponents, step {k}"
            rep.quantised_checked += int((q_o == 1).sum())
        if okw.get("momentum") is not None:
            v_g = gpu_sub(eg.velocity().to(dev))
            assert np.array_equal(v_g.view(np.uint32), o.velocity().view(np.uint32)), f"velocity, step {k}"
        if deliver_fn is not None:
            rc_g = gpu_sub(eg.received().to(dev))
            assert np.array_equal(rc_g.view(np.uint32), o.received().view(np.uint32)), f"received, step {k}"
            pend, arrivals = eg.delivery_status()
            assert np.array_equal(pend[:, tensors], o.pending()), f"in flight, step {k}"
            if full:
                assert arrivals == o.arrivals, f"arrivals, step {k}"
        lap("compare")

    rep.topk_repeats = eg.topk_repeat_count()
    eg.close()
    o.close()
    return rep
