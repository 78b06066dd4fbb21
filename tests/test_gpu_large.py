"""Largest supported tensor (2^31 - 1 elements) and element offsets beyond 2^31.

The oracle follows the small tensors that sit behind the large one (their offsets inside a
replica exceed 32 bits); the large tensor itself is checked through properties that hold at any
size and are computed with torch's own fp64 routines on the GPU: the SGD update of a lone
replica (Algorithm B with no neighbours: x <- x - lr g, rounded once), the change norm
|| x - x_hat ||, and for Top-K the size, order, values and threshold property of the message.
"""
import numpy as np
import pytest
import torch

from oracle import eg_oracle as eo
from paper_2103_07454_b200 import binding as B
from paper_2103_07454_b200 import workload as W

pytestmark = pytest.mark.gpu

N0 = 2 ** 31 - 1
NUMEL = [N0, 5000, 37]
CHUNK = 1 << 26
SEED = 4242
LR = 0.05
NEED_BYTES = 70 << 30


def _chunks(n):
    for s in range(0, n, CHUNK):
        yield s, min(CHUNK, n - s)


def _fill(eg, out, stream, scale):
    """Seeded values for every tensor, written at the library's offsets, chunk by chunk."""
    for t, n in enumerate(NUMEL):
        base = W.stream_base(SEED, stream, t)
        o = int(eg.tensor_offset[t])
        for s, c in _chunks(n):
            out[0, o + s:o + s + c] = W.ih8_integers(base, s, c, "cuda").to(torch.float32) * scale


def _small(stream, scale):
    """The same values for the small tensors, made on the CPU, packed [1, 5037]."""
    parts = [W.ih8_integers(W.stream_base(SEED, stream, t), 0, NUMEL[t], "cpu").to(torch.float32) * scale
             for t in (1, 2)]
    return torch.cat(parts).unsqueeze(0).numpy().copy()


def _sq_norm(a, b):
    """fp64 sum over the fp32 differences a - b (1-D views), chunked."""
    acc = 0.0
    for s, c in _chunks(a.numel()):
        d = (a[s:s + c] - b[s:s + c]).double()
        acc += float((d * d).sum())
    return acc


def _check_update(x_new, x_old, g, lr32):
    for s, c in _chunks(x_new.numel()):
        want = (x_old[s:s + c].double() + (-lr32) * g[s:s + c].double()).float()
        assert torch.equal(want, x_new[s:s + c]), f"update, elements {s}..{s + c}"


def _enough_memory():
    free, _ = torch.cuda.mem_get_info()
    return free >= NEED_BYTES


@pytest.mark.parametrize("carry", [False, True])
def test_largest_tensor_dense(carry):
    if not _enough_memory():
        pytest.skip("needs about 70 GB of free device memory")
    wl = W.synthetic(1, NUMEL, steps=3, lr=LR)
    eg = B.from_workload(wl)
    eg.set_carry_norm(carry)
    assert eg.tensor_offset[1] >= 2 ** 31 and eg.replica_stride > 2 ** 31
    o = eo.Oracle(1, NUMEL[1:], horizon=1.0, history_len=1, delta_init=0.0, threads=1)
    lr32 = float(np.float32(LR))
    x = torch.zeros((1, eg.replica_stride), dtype=torch.float32, device="cuda")
    g = torch.zeros_like(x)
    _fill(eg, x, 1, 0.05 / W.IH8_STD)
    xs = _small(1, 0.05 / W.IH8_STD)
    big = slice(int(eg.tensor_offset[0]), int(eg.tensor_offset[0]) + N0)
    xhat = torch.zeros(N0, dtype=torch.float32, device="cuda")     # what the large tensor last sent
    events = 0
    for k in range(3):
        _fill(eg, g, 10 + k, 1e-3 / W.IH8_STD)
        gs = _small(10 + k, 1e-3 / W.IH8_STD)
        x_old = x[0, big].clone()
        eg.step(x, g, LR)
        o.step(xs, gs, LR)
        f, d, thr = eg.last_decisions()
        # the small tensors behind the 2^31 boundary, against the oracle
        assert np.array_equal(f[:, 1:], o.flags())
        assert np.allclose(d[:, 1:], o.norms(), rtol=1e-12, atol=0)
        for t in (1, 2):
            lo = int(eg.tensor_offset[t])
            got = x[0, lo:lo + NUMEL[t]].cpu().numpy()
            first = 0 if t == 1 else NUMEL[1]
            assert np.array_equal(got.view(np.uint32), xs[0, first:first + NUMEL[t]].view(np.uint32))
        # the large tensor: norm, decision, update
        want_d = float(np.sqrt(_sq_norm(x_old, xhat)))
        assert abs(d[0, 0] - want_d) <= 1e-10 * want_d, (k, d[0, 0], want_d)
        assert bool(f[0, 0]) == (k == 0 or d[0, 0] >= thr[0, 0])
        if f[0, 0]:
            xhat.copy_(x_old)
            events += 1
        _check_update(x[0, big], x_old, g[0, big], lr32)
        del x_old
    _, ev = eg.thresholds()
    assert int(ev[0, 0]) == events and events >= 2
    assert eg.stats()["messages"] == 0          # a lone replica has nobody to send to
    eg.close()
    o.close()


def test_largest_tensor_topk():
    if not _enough_memory():
        pytest.skip("needs about 70 GB of free device memory")
    wl = W.synthetic(1, NUMEL, steps=3, lr=LR, topk=(1, 100))
    eg = B.from_workload(wl)
    o = eo.Oracle(1, NUMEL[1:], horizon=1.0, history_len=1, delta_init=0.0, topk=(1, 100), threads=1)
    k0 = eg.topk_count(0)
    assert k0 == -(-N0 // 100)
    lr32 = float(np.float32(LR))
    x = torch.zeros((1, eg.replica_stride), dtype=torch.float32, device="cuda")
    g = torch.zeros_like(x)
    _fill(eg, x, 1, 0.05 / W.IH8_STD)
    xs = _small(1, 0.05 / W.IH8_STD)
    big = slice(int(eg.tensor_offset[0]), int(eg.tensor_offset[0]) + N0)
    xhat = torch.zeros(N0, dtype=torch.float32, device="cuda")
    sparse_seen = 0
    for k in range(3):
        _fill(eg, g, 10 + k, 1e-3 / W.IH8_STD)
        gs = _small(10 + k, 1e-3 / W.IH8_STD)
        x_old = x[0, big].clone()
        eg.step(x, g, LR)
        o.step(xs, gs, LR)
        f, d, thr = eg.last_decisions()
        assert np.array_equal(f[:, 1:], o.flags())
        for ts, t in enumerate((1, 2)):
            if o.flags()[0, ts]:
                idx_o, val_o = o.outbox(0, ts)
                idx_g, val_g = eg.last_outbox(0, t)
                assert np.array_equal(idx_o, idx_g) and np.array_equal(val_o.view(np.uint32), val_g.view(np.uint32))
        want_d = float(np.sqrt(_sq_norm(x_old, xhat)))
        assert abs(d[0, 0] - want_d) <= 1e-10 * want_d, (k, d[0, 0], want_d)
        if f[0, 0] and k == 0:
            xhat.copy_(x_old)                               # the first message is dense
        elif f[0, 0]:
            idx, val = eg.last_outbox(0, 0)
            assert len(idx) == k0
            idx_d = torch.from_numpy(idx).cuda().long()
            val_d = torch.from_numpy(val).cuda()
            assert bool((idx_d[1:] > idx_d[:-1]).all()) and int(idx_d[0]) >= 0 and int(idx_d[-1]) < N0
            assert torch.equal(x_old[idx_d], val_d)
            sel = torch.zeros(N0, dtype=torch.bool, device="cuda")
            sel[idx_d] = True
            lowest_sent, highest_kept = float("inf"), 0.0
            for s, c in _chunks(N0):
                mag = (x_old[s:s + c] - xhat[s:s + c]).abs()
                m = sel[s:s + c]
                if bool(m.any()):
                    lowest_sent = min(lowest_sent, float(mag[m].min()))
                if not bool(m.all()):
                    highest_kept = max(highest_kept, float(mag[~m].max()))
            assert lowest_sent >= highest_kept
            xhat[idx_d] = val_d                              # delivery; checked by the next step's norm
            del sel, idx_d, val_d
            sparse_seen += 1
        _check_update(x[0, big], x_old, g[0, big], lr32)
        del x_old
    assert sparse_seen >= 1
    eg.close()
    o.close()
