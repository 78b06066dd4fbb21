"""The allocation-free norm entry point (eg_change_norms_static) against the norm pass of
eg_step.

Collected last on purpose (file name): a run that stops at the first failure has then already
run every other test.  The entry point serves callers that cannot allocate device memory when
they need the norms (during stream capture, inside a memory pool that forbids raw cudaMalloc,
in a latency-bound loop); it keeps its scratch in a fixed array inside the library, so the
test also checks that a second call, which reuses that array, is not disturbed by the first.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2103_07454_b200 import binding as B
from paper_2103_07454_b200 import workload as W

pytestmark = pytest.mark.gpu

from parity_harness import norm_rtol  # noqa: E402

NUMEL = [1, 3, 4, 5, 31, 32, 33, 1023, 1024, 1025, 4095, 4096, 4097, 10000, (1 << 18) + 1]


def test_static_norms_match_eg_step_on_two_calls_in_a_row():
    wl = W.synthetic(5, NUMEL, steps=6, lr=0.1, grad_sigma=0.01)
    eg = B.from_workload(wl)
    x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
    out = torch.full((wl.P * wl.T,), -1.0, dtype=torch.float64, device="cuda")
    tol = norm_rtol(wl.numel)[None, :]
    checked = 0
    for k in range(wl.steps):
        g = eg.to_layout(wl.grads(k, "cuda"))
        xhat = eg.mailboxes().cuda()                 # x_hat as eg_step is about to see it
        for _ in range(2):                           # two calls in a row share the scratch
            out.fill_(-1.0)
            B.change_norms_static(x, xhat, eg.tensor_offset, eg.numel, out)
            got = out.cpu().numpy().reshape(wl.P, wl.T)
            if checked == 0:
                first = got.copy()
            checked += 1
        eg.step(x, g, wl.lr)
        _, want, _ = eg.last_decisions()             # the norms eg_step computed from the same data
        assert np.all(np.abs(got - want) <= tol * np.abs(want)), f"step {k}"
        assert np.array_equal(got, want), "same tiles and summation order: expected the same bits"
    assert checked == 2 * wl.steps and np.all(first >= 0)
    eg.close()


def test_static_norms_unpadded_layout_and_limits():
    P, numel = 3, [5, 4099, 64]
    offs = [0, 8, 8 + 4100]                          # multiples of 4, no 128-byte padding
    stride = 8 + 4100 + 64
    gen = torch.Generator(device="cuda").manual_seed(3)
    x = torch.randn((P, stride), device="cuda", generator=gen)
    h = torch.randn((P, stride), device="cuda", generator=gen)
    out = torch.empty(P * 3, dtype=torch.float64, device="cuda")
    B.change_norms_static(x, h, offs, numel, out)
    got = out.cpu().numpy().reshape(P, 3)
    for t, (o, n) in enumerate(zip(offs, numel)):
        d = (x[:, o:o + n] - h[:, o:o + n]).double()
        want = d.pow(2).sum(dim=1).sqrt().cpu().numpy()
        assert np.allclose(got[:, t], want, rtol=1e-13, atol=0)

    lib = B.load_library()
    i64 = ctypes.c_int64
    too_many = B.STATIC_MAX_TENSORS + 1
    offs_c = (i64 * too_many)(*[4 * t for t in range(too_many)])
    nums_c = (i64 * too_many)(*([4] * too_many))
    args = (x.data_ptr(), h.data_ptr(), 1, 4 * too_many, offs_c, nums_c, too_many, out.data_ptr(), None)
    assert lib.eg_change_norms_static(*args) == 1                     # too many tensors
    big = (B.STATIC_MAX_PARTIALS // 2 + 1) * 4096                     # 2 replicas exceed the scratch
    offs_c, nums_c = (i64 * 1)(0), (i64 * 1)(big)
    assert lib.eg_change_norms_static(x.data_ptr(), h.data_ptr(), 2, big, offs_c, nums_c, 1,
                                      out.data_ptr(), None) == 1
    assert lib.eg_change_norms_static(None, h.data_ptr(), 1, 8, offs_c, (i64 * 1)(8), 1,
                                      out.data_ptr(), None) == 1      # NULL input
    # more replicas than a grid dimension holds: refused before anything is launched
    assert lib.eg_change_norms_static(x.data_ptr(), h.data_ptr(), 65536, 4, offs_c, (i64 * 1)(4), 1,
                                      out.data_ptr(), None) == 1
    # an offset that would overflow the bounds check
    assert lib.eg_change_norms_static(x.data_ptr(), h.data_ptr(), 1, 8, (i64 * 1)(2 ** 63 - 4), (i64 * 1)(8), 1,
                                      out.data_ptr(), None) == 1
    torch.cuda.synchronize()
