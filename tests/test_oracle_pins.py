"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests re-types the oracle's own loop: each compares it with a closed form, a
dense matrix product, a brute-force sort, an invariant, or a sequence worked by hand and
stored under tests/golden/.
"""
import math
import os

import numpy as np
import pytest

from oracle import eg_oracle as eo
from paper_2103_07454_b200 import workload as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
INF = float("inf")


def ring_matrix(P, hops=1):
    """Mixing matrix of Section 3: W_ij = 1/(N_i + 1) over the PE itself and its distinct
    ring neighbours (the `hops` nearest on each side)."""
    Wm = np.zeros((P, P))
    for i in range(P):
        nb = {i} | {(i + d) % P for d in range(-hops, hops + 1)}
        for j in nb:
            Wm[i, j] = 1.0 / len(nb)
    return Wm


def ulp32(a):
    return np.spacing(np.abs(a).astype(np.float32)).astype(np.float64)


def small(P=5, numel=(7, 1, 33, 128, 5), **kw):
    return W.synthetic(P, numel, **kw)


# ---------------------------------------------------------------------------------------
# delta = 0  ==  regular D-PSGD,  X_{k+1} = X_k W - gamma G   (Eq. (dist_sgd_neigh); remark
# after Corollary 1: "a threshold of 0 reduces to the regular algorithm")
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("P", [1, 2, 3, 4, 7])
def test_zero_threshold_is_dpsgd(P):
    wl = small(P=P, steps=6, lr=0.1, grad_sigma=0.01)
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=0.0, force_first_event=False)
    x = W.distinct_init_params(wl).numpy().copy()
    Wm = ring_matrix(P)
    deg = 0 if P == 1 else (1 if P == 2 else 2)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        ref = Wm @ x.astype(np.float64) - np.float64(np.float32(wl.lr)) * g.astype(np.float64)
        o.step(x, g, wl.lr)
        assert o.flags().all()
        assert np.all(np.abs(x.astype(np.float64) - ref) <= 0.5000001 * ulp32(ref) + 1e-300)
        st = o.stats()
        assert st["messages"] == P * wl.T * deg * (k + 1)
        assert st["bytes"] == 4 * wl.N * P * deg * (k + 1)
        assert st["events"] == P * wl.T * (k + 1)


@pytest.mark.parametrize("P,hops", [(2, 2), (3, 2), (4, 2), (5, 2), (7, 3), (9, 2), (16, 4)])
def test_more_neighbours_zero_threshold_is_xw(P, hops):
    """More neighbours per PE (Section 7): W stays symmetric doubly stochastic with
    W_ij = 1/(N_i + 1); threshold 0 still gives X W - gamma G, and the message count follows
    the number of distinct neighbours."""
    wl = small(P=P, steps=4, lr=0.1, grad_sigma=0.01)
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=0.0, hops=hops)
    x = W.distinct_init_params(wl).numpy().copy()
    Wm = ring_matrix(P, hops)
    assert np.allclose(Wm.sum(0), 1) and np.allclose(Wm.sum(1), 1) and np.allclose(Wm, Wm.T)
    deg = min(2 * hops, P - 1)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        ref = Wm @ x.astype(np.float64) - np.float64(np.float32(wl.lr)) * g.astype(np.float64)
        o.step(x, g, wl.lr)
        assert np.all(np.abs(x.astype(np.float64) - ref) <= 0.5000001 * ulp32(ref) + 1e-300)
        assert o.stats()["messages"] == P * wl.T * deg * (k + 1)


def test_more_neighbours_eigenmode_decay():
    """Circulant W with 2 neighbours per side: eigenvalue (1 + 2cos(a) + 2cos(2a)) / 5, a = 2 pi m / P."""
    P, m, hops = 12, 1, 2
    o = eo.Oracle(P, [3], mode=eo.FIXED, delta_fixed=0.0, hops=hops)
    mode = np.cos(2 * np.pi * m * np.arange(P) / P)
    amp = np.array([1.0, -2.0, 0.5])
    x = (mode[:, None] * amp[None, :]).astype(np.float32)
    x_init = x.astype(np.float64)
    a = 2 * math.pi * m / P
    lam = (1 + 2 * math.cos(a) + 2 * math.cos(2 * a)) / 5
    lam1 = (1 + 2 * math.cos(a)) / 3
    assert lam < lam1                                   # information flows sooner
    for s_ in range(1, 9):
        o.step(x, np.zeros_like(x), 0.1)
        assert np.all(np.abs(x - lam ** s_ * x_init) <= 3e-7 * np.abs(amp)[None, :] * s_ + 1e-12)


# ---------------------------------------------------------------------------------------
# delta = infinity: no messages, every replica runs plain SGD on its own
# ---------------------------------------------------------------------------------------
def test_infinite_threshold_is_independent_sgd():
    wl = small(P=4, steps=5, lr=0.25, grad_sigma=0.02)
    o = eo.Oracle(4, wl.numel, mode=eo.FIXED, delta_fixed=INF, force_first_event=False)
    x0 = W.distinct_init_params(wl).numpy().copy()
    x = x0.copy()
    ref = x0.astype(np.float64)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        o.step(x, g, wl.lr)
        ref = (ref - np.float64(np.float32(wl.lr)) * g.astype(np.float64)).astype(np.float32).astype(np.float64)
        assert not o.flags().any()
        assert np.all(np.abs(x - ref) <= ulp32(ref))
    assert o.stats() == {"messages": 0, "bytes": 0, "events": 0}
    assert not o.valid().any()
    assert np.all(o.xhat() == 0)


def test_only_forced_event_then_frozen_mailboxes():
    """With an infinite threshold but the forced event at k = 0 (Section 4), neighbours keep
    averaging with the value received at k = 0 ("the last received version") while the own
    term follows the replica's current parameters."""
    P = 5
    wl = small(P=P, steps=4, lr=0.1, grad_sigma=0.05)
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=INF, force_first_event=True)
    x0 = W.distinct_init_params(wl).numpy().copy()
    x = x0.copy()
    frozen = x0.astype(np.float64)
    ref = x0.astype(np.float64)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        o.step(x, g, wl.lr)
        assert o.flags().all() == (k == 0) and o.flags().any() == (k == 0)
        left, right = np.roll(frozen, 1, axis=0), np.roll(frozen, -1, axis=0)
        ref = (ref + left + right) / 3.0 - np.float64(np.float32(wl.lr)) * g.astype(np.float64)
        ref = ref.astype(np.float32).astype(np.float64)
        assert np.all(np.abs(x - ref) <= ulp32(ref))
    assert np.array_equal(o.xhat(), x0)
    assert o.stats()["messages"] == P * wl.T * 2


# ---------------------------------------------------------------------------------------
# W doubly stochastic: replica mean preserved; circulant eigen-modes of the ring
# ---------------------------------------------------------------------------------------
def test_mean_preserved_with_zero_gradients():
    P = 6
    wl = small(P=P, steps=25)
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=0.0)
    x = W.distinct_init_params(wl).numpy().copy()
    mean0 = x.astype(np.float64).mean(axis=0)
    g = np.zeros_like(x)
    d_prev = o.consensus_distance(x)
    for _ in range(wl.steps):
        o.step(x, g, 0.1)
        mean = x.astype(np.float64).mean(axis=0)
        assert np.all(np.abs(mean - mean0) <= 4 * wl.steps * ulp32(np.abs(x).max(axis=0)))
        d = o.consensus_distance(x)
        assert d < d_prev  # contraction towards the mean on a connected ring
        d_prev = d
    assert d_prev < 1e-6 * o.consensus_distance(W.distinct_init_params(wl).numpy())


@pytest.mark.parametrize("P,m", [(4, 1), (5, 1), (5, 2), (8, 3), (16, 1)])
def test_ring_eigenmode_decay(P, m):
    """The ring W is circulant with eigenvalues (1 + 2 cos(2 pi m / P)) / 3 (all of modulus
    < 1 for m != 0: the spectral-gap assumption); a cosine mode decays geometrically."""
    n = 4
    steps = 12
    o = eo.Oracle(P, [n], mode=eo.FIXED, delta_fixed=0.0)
    mode = np.cos(2 * np.pi * m * np.arange(P) / P)
    amp = np.array([1.0, -2.5, 0.125, 3.0])
    x = (mode[:, None] * amp[None, :]).astype(np.float32)
    x_init = x.astype(np.float64)
    lam = (1 + 2 * math.cos(2 * math.pi * m / P)) / 3
    g = np.zeros_like(x)
    for s in range(1, steps + 1):
        o.step(x, g, 0.3)
        ref = lam ** s * x_init
        assert np.all(np.abs(x - ref) <= 2e-7 * np.abs(amp)[None, :] * s + 1e-12)


# ---------------------------------------------------------------------------------------
# forced first event, error bound, accounting
# ---------------------------------------------------------------------------------------
def seg_norms(a, b, numel):
    """||a - b|| per (replica, tensor) with fp32 differences, computed by numpy."""
    P = a.shape[0]
    out = np.zeros((P, len(numel)))
    off = 0
    for t, n in enumerate(numel):
        d = (a[:, off:off + n] - b[:, off:off + n]).astype(np.float32).astype(np.float64)
        out[:, t] = np.sqrt((d * d).sum(axis=1))
        off += n
    return out


@pytest.mark.parametrize("hist", [1, 3])
def test_error_bound_and_forced_first_event(hist):
    P = 4
    wl = small(P=P, steps=30, lr=0.1, grad_sigma=0.01, history_len=hist)
    o = eo.from_workload(wl)
    x = W.distinct_init_params(wl).numpy().copy()
    total_events = 0
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        x_pre = x.copy()
        xhat_pre = o.xhat()
        o.step(x, g, wl.lr)
        f = o.flags().astype(bool)
        if k == 0:
            assert f.all()                      # forced event at k = 0
            assert np.all(o.thresholds_used() == 0.0)
        d_np = seg_norms(x_pre, xhat_pre, wl.numel)
        assert np.allclose(o.norms(), d_np, rtol=1e-13, atol=0)
        # the decision is the displayed inequality
        if k > 0:
            differs = f != (d_np >= o.thresholds_used())
            assert np.all(np.abs(d_np - o.thresholds_used())[differs] <= 1e-12 * d_np[differs])
        # error bound of Section 5: after communicating, ||x_hat - x|| is 0 for the tensors
        # sent and stays below the threshold for the others
        e_post = seg_norms(x_pre, o.xhat(), wl.numel)
        assert np.all(e_post[f] == 0.0)
        assert np.all(e_post[~f] < o.thresholds_used()[~f])
        total_events += int(f.sum())
        assert np.array_equal(o.last_event_iteration()[f], np.full(f.sum(), k))
    st = o.stats()
    assert st["events"] == total_events
    assert st["messages"] == 2 * total_events
    assert 0 < total_events < P * wl.T * wl.steps  # some, not all: the trigger does select
    assert o.segment_events().sum() == total_events


@pytest.mark.parametrize("P,deg", [(1, 0), (2, 1), (3, 2)])
def test_message_accounting_and_neighbour_dedup(P, deg):
    numel = [3, 10]
    o = eo.Oracle(P, numel, mode=eo.FIXED, delta_fixed=0.0)
    x = np.arange(P * 13, dtype=np.float32).reshape(P, 13) / 8
    x0 = x.astype(np.float64)
    o.step(x, np.zeros_like(x), 0.0)
    st = o.stats()
    assert st["events"] == 2 * P and st["messages"] == 2 * P * deg
    assert st["bytes"] == deg * P * 4 * 13
    assert np.allclose(x, ring_matrix(P) @ x0, rtol=0, atol=1e-6)


# ---------------------------------------------------------------------------------------
# adaptive threshold: hand-worked sequences
# ---------------------------------------------------------------------------------------
def load_threshold_cases():
    cases, cur = [], None
    with open(os.path.join(GOLDEN, "threshold_sequence.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("case"):
                _, name, H, h, *rest = line.split()
                cur = {"name": name, "H": int(H[2:]), "h": float(h[2:]), "rows": [],
                       "change_of_norm": "metric=change_of_norm" in rest}
                cases.append(cur)
            else:
                cur["rows"].append([float(v) for v in line.split()])
    return cases


@pytest.mark.parametrize("case", load_threshold_cases(), ids=lambda c: c["name"])
def test_hand_worked_threshold_sequence(case):
    rows = case["rows"]
    o = eo.Oracle(1, [2], horizon=case["h"], history_len=case["H"], delta_init=0.0,
                  change_of_norm=case["change_of_norm"])
    x = np.array([[rows[0][1], rows[0][2]]], dtype=np.float32)
    for r, row in enumerate(rows):
        k, x0, x1, flag, d, thr_tested, thr_after = row
        assert o.iteration == int(k)
        assert x[0, 0] == x0 and x[0, 1] == x1
        nxt = rows[r + 1] if r + 1 < len(rows) else row
        g = np.array([[x0 - nxt[1], x1 - nxt[2]]], dtype=np.float32)
        o.step(x, g, 1.0)
        assert int(o.flags()[0, 0]) == int(flag), f"k={k}"
        assert o.norms()[0, 0] == pytest.approx(d, rel=1e-15, abs=0)
        assert o.thresholds_used()[0, 0] == pytest.approx(thr_tested, rel=1e-15, abs=0)
        assert o.thresholds()[0, 0] == pytest.approx(thr_after, rel=1e-15, abs=0)


def test_geometric_bound_on_the_threshold():
    """Assumption 1 with g(k) = alpha beta^k (Corollary 2): the threshold in force is
    min(delta, sqrt(g(k))).  alpha = 16, beta = 1/4: sqrt(g) = 4, 2, 1, 1/2, 1/4 (exact).
    x moves along u = (0.75, 1), |u| = 1.25, by 1, 1, 1, 1/2, 1/4 units; fixed delta = 2."""
    o = eo.Oracle(1, [2], mode=eo.FIXED, delta_fixed=2.0, force_first_event=False,
                  threshold_cap=(16.0, 0.25))
    steps_u = [1.0, 1.0, 1.0, 0.5, 0.25]
    x = np.zeros((1, 2), np.float32)
    pos = 0.0
    want = [(0, 1.25, 2.0), (1, 2.5, 2.0), (1, 1.25, 1.0), (1, 0.625, 0.5), (1, 0.3125, 0.25)]
    for k, du in enumerate(steps_u):
        pos += du
        x[0] = [0.75 * pos, pos]
        o.step(x, np.zeros_like(x), 1.0)
        flag, d, thr = want[k]
        assert int(o.flags()[0, 0]) == flag and o.norms()[0, 0] == d
        assert o.thresholds_used()[0, 0] == thr and o.thresholds()[0, 0] == 2.0
    # without the bound: k = 1 fires (d = 2.5), then d = 1.25, 1.875, 2.1875 -> k = 4 fires again
    o = eo.Oracle(1, [2], mode=eo.FIXED, delta_fixed=2.0, force_first_event=False)
    x[:] = 0
    pos, fired = 0.0, []
    for du in steps_u:
        pos += du
        x[0] = [0.75 * pos, pos]
        o.step(x, np.zeros_like(x), 1.0)
        fired.append(int(o.flags()[0, 0]))
    assert fired == [0, 1, 0, 0, 1]


def test_geometric_bound_stays_on_the_exact_sequence():
    """The bound is carried as the geometric sequence it is, g(0) = alpha, g(k+1) = beta g(k), one
    rounding per term.  Against alpha * beta^k in exact rational arithmetic (a double is a dyadic
    rational) the k-th term is off by at most k roundings; the tested threshold is its square
    root.  A bound that is set at iteration k0 continues with the k0-th term of the sequence."""
    from fractions import Fraction
    alpha, beta, steps = 3.7, 0.93, 60
    o = eo.Oracle(1, [2], mode=eo.FIXED, delta_fixed=float("inf"), force_first_event=False,
                  threshold_cap=(alpha, beta))
    late = eo.Oracle(1, [2], mode=eo.FIXED, delta_fixed=float("inf"), force_first_event=False)
    x = np.ones((1, 2), np.float32)
    exact = Fraction(alpha)
    for k in range(steps):
        if k == 17:
            late.set_threshold_cap(alpha, beta)
        o.step(x, np.zeros_like(x), 1.0)
        late.step(x.copy(), np.zeros_like(x), 1.0)
        thr = o.thresholds_used()[0, 0]
        rel = abs(Fraction(thr) ** 2 / exact - 1)
        assert rel <= (k + 2) * 2.0 ** -52, (k, float(rel))
        if k >= 17:
            assert late.thresholds_used()[0, 0] == thr
        else:
            assert late.thresholds_used()[0, 0] == float("inf")
        exact *= Fraction(beta)
    o.reset()
    o.step(x, np.zeros_like(x), 1.0)
    assert o.thresholds_used()[0, 0] == np.sqrt(alpha)


def test_fixed_threshold_never_adapts():
    o = eo.Oracle(1, [2], mode=eo.FIXED, delta_fixed=2.0, force_first_event=False)
    x = np.zeros((1, 2), np.float32)
    fired = []
    for k in range(6):
        o.step(x, np.array([[-0.6, -0.8]], np.float32), 1.0)  # |x| grows by 1 per step
        fired.append(int(o.flags()[0, 0]))
        assert o.thresholds()[0, 0] == 2.0
    # x_k = k*(0.6,0.8): k=0,1 below 2; k=2 fires (d~2, x_hat<-x_2); k=3 d~1; k=4 fires; ...
    assert fired[:2] == [0, 0] and sum(fired) >= 1


# ---------------------------------------------------------------------------------------
# variants: own term read literally from Eq. (dist_sgd_event); change-of-norm trigger
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("own,con", [(True, False), (False, True), (True, True)])
def test_variants_reduce_to_dpsgd_at_zero_threshold(own, con):
    P = 5
    wl = small(P=P, steps=5, lr=0.1, grad_sigma=0.01)
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=0.0, own_last_sent=own, change_of_norm=con)
    x = W.distinct_init_params(wl).numpy().copy()
    Wm = ring_matrix(P)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        ref = Wm @ x.astype(np.float64) - np.float64(np.float32(wl.lr)) * g.astype(np.float64)
        o.step(x, g, wl.lr)
        assert o.flags().all()
        assert np.all(np.abs(x.astype(np.float64) - ref) <= 0.5000001 * ulp32(ref) + 1e-300)


def test_literal_own_term_uses_the_last_sent_value():
    """X_{k+1} = X_hat_k W - gamma G read literally: with mailboxes frozen at x_0 (forced first
    event, infinite threshold afterwards) nothing accumulates, x_{k+1} = W x_0 - gamma g_k;
    and a replica that never sent anything averages with X_0 = 0."""
    P = 5
    wl = small(P=P, steps=4, lr=0.1, grad_sigma=0.05)
    lr64 = np.float64(np.float32(wl.lr))
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=INF, force_first_event=True, own_last_sent=True)
    x0 = W.distinct_init_params(wl).numpy().copy()
    x = x0.copy()
    base = ring_matrix(P) @ x0.astype(np.float64)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        o.step(x, g, wl.lr)
        ref = base - lr64 * g.astype(np.float64)
        assert np.all(np.abs(x - ref) <= ulp32(ref))
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=INF, force_first_event=False, own_last_sent=True)
    x = x0.copy()
    g = wl.grads(0).numpy()
    o.step(x, g, wl.lr)
    assert np.all(np.abs(x - (-lr64 * g.astype(np.float64))) <= ulp32(lr64 * g))


def test_change_of_norm_ignores_rotations():
    """A vector that turns without changing its length triggers the norm-of-change test but
    not the change-of-norm test."""
    fired = {}
    for con in (False, True):
        o = eo.Oracle(1, [2], mode=eo.FIXED, delta_fixed=0.5, force_first_event=True, change_of_norm=con)
        x = np.array([[3.0, 4.0]], np.float32)
        o.step(x, np.array([[-5.0, 2.0]], np.float32), 1.0)      # x becomes (8, 2)... any value
        x[:] = [[4.0, 3.0]]                                         # same length as (3, 4), turned
        o.step(x, np.zeros((1, 2), np.float32), 1.0)
        fired[con] = int(o.flags()[0, 0])
        if con:
            assert o.norms()[0, 0] == 0.0 and o.sent_norms()[0, 0] == 5.0
        else:
            assert o.norms()[0, 0] == pytest.approx(math.sqrt(2.0), rel=1e-15)
    assert fired == {False: 1, True: 0}


# ---------------------------------------------------------------------------------------
# intermittent delivery (messages that stay in flight)
# ---------------------------------------------------------------------------------------
def test_delivering_everything_is_synchronous_delivery():
    wl = small(P=4, steps=12, lr=0.1, grad_sigma=0.01, topk=(1, 4))
    a, b = eo.from_workload(wl), eo.from_workload(wl)
    xa = W.distinct_init_params(wl).numpy().copy()
    xb = xa.copy()
    ones = np.ones((wl.P, wl.T), np.uint8)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        a.step(xa, g, wl.lr)
        b.step(xb, g, wl.lr, deliver=ones)
        assert np.array_equal(xa, xb) and np.array_equal(a.flags(), b.flags())
        assert np.array_equal(b.received(), b.xhat()) and not b.pending().any()
    assert a.stats() == b.stats() and b.arrivals == b.stats()["events"]


def test_nothing_ever_delivered_is_independent_sgd_although_events_happen():
    wl = small(P=4, steps=6, lr=0.25, grad_sigma=0.02)
    o = eo.from_workload(wl)
    x0 = W.distinct_init_params(wl).numpy().copy()
    x = x0.copy()
    ref = x0.astype(np.float64)
    none = np.zeros((wl.P, wl.T), np.uint8)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        o.step(x, g, wl.lr, deliver=none)
        ref = (ref - np.float64(np.float32(wl.lr)) * g.astype(np.float64)).astype(np.float32).astype(np.float64)
        assert np.all(np.abs(x - ref) <= ulp32(ref))
    assert o.stats()["events"] >= wl.P * wl.T and o.arrivals == 0
    assert o.pending().all() and np.all(o.received() == 0)


def test_links_that_are_up_every_other_step():
    """Threshold 0 (everything is sent every step); links deliver on even steps only.  On an even
    step neighbours average with x_k, on an odd step with the stale x_{k-1}."""
    P = 5
    wl = small(P=P, steps=6, lr=0.1, grad_sigma=0.02)
    lr64 = np.float64(np.float32(wl.lr))
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=0.0)
    x = W.distinct_init_params(wl).numpy().copy()
    stale = None
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        up = k % 2 == 0
        cur = x.astype(np.float64)
        box = cur if up else stale
        ref = (cur + np.roll(box, 1, axis=0) + np.roll(box, -1, axis=0)) / 3.0 - lr64 * g.astype(np.float64)
        o.step(x, g, wl.lr, deliver=np.full((P, wl.T), int(up), np.uint8))
        assert np.all(np.abs(x - ref) <= ulp32(ref))
        if up:
            stale = cur
        assert o.pending().all() == (not up) and np.array_equal(o.received(), stale.astype(np.float32))
    assert o.arrivals == P * wl.T * 3


def test_outstanding_sparse_messages_arrive_together():
    """A delivery hands over everything outstanding: afterwards the receivers' copy equals
    the sender's record, before it is untouched."""
    wl = small(P=3, numel=(40, 300), steps=10, lr=0.1, grad_sigma=0.02, topk=(1, 10))
    o = eo.Oracle(3, wl.numel, mode=eo.FIXED, delta_fixed=0.0, topk=wl.topk)
    x = W.distinct_init_params(wl).numpy().copy()
    rng = np.random.default_rng(0)
    for k in range(wl.steps):
        mask = (rng.random((3, wl.T)) < 0.4).astype(np.uint8)
        before = o.received() if k else np.zeros_like(x)
        o.step(x, wl.grads(k).numpy(), wl.lr, deliver=mask)
        sent, got = o.xhat(), o.received()
        off = 0
        for t, n in enumerate(wl.numel):
            for i in range(3):
                seg = slice(off, off + n)
                if mask[i, t]:
                    assert np.array_equal(got[i, seg], sent[i, seg])
                else:
                    assert np.array_equal(got[i, seg], before[i, seg])
            off += n


# ---------------------------------------------------------------------------------------
# Top-K
# ---------------------------------------------------------------------------------------
def brute_force_topk(x_row, xhat_row, K):
    d = (x_row - xhat_row).astype(np.float32)
    key = np.abs(d).view(np.uint32).astype(np.int64)
    order = np.lexsort((np.arange(len(d)), -key))  # key descending, index ascending
    return np.sort(order[:K]).astype(np.int32)


@pytest.mark.parametrize("frac", [(1, 100), (10, 100), (1, 3), (1, 1)])
def test_topk_against_brute_force(frac):
    P = 3
    numel = [1, 2, 17, 100, 1000, 4097]
    wl = W.synthetic(P, numel, steps=24, lr=0.1, grad_sigma=0.01, topk=frac)
    o = eo.from_workload(wl)
    x = W.distinct_init_params(wl).numpy().copy()
    rng = np.random.default_rng(5)
    sparse_seen = 0
    bytes_expected = 0
    for k in range(wl.steps):
        g = wl.grads(k).numpy().copy()
        # engineered ties: quantise some gradients so many |delta| coincide, and zero some
        g[:, 1200:1600] = np.round(g[:, 1200:1600] * 64) / 64
        g[:, 3000:3100] = 0.0
        x_pre = x.copy()
        xhat_pre = o.xhat()
        valid_pre = o.valid().astype(bool)
        o.step(x, g, wl.lr)
        f = o.flags().astype(bool)
        xhat_post = o.xhat()
        off = 0
        for t, n in enumerate(numel):
            K = max(1, -(-n * frac[0] // frac[1]))
            assert o.topk_count(t) == K
            for i in range(P):
                idx, val = o.outbox(i, t)
                seg_pre = xhat_pre[i, off:off + n]
                seg_post = xhat_post[i, off:off + n]
                if f[i, t] and valid_pre[i, t]:
                    want = brute_force_topk(x_pre[i, off:off + n], seg_pre, K)
                    assert np.array_equal(idx, want)
                    assert np.array_equal(val, x_pre[i, off:off + n][want])
                    expect = seg_pre.copy()
                    expect[want] = x_pre[i, off:off + n][want]
                    assert np.array_equal(seg_post, expect)
                    sparse_seen += 1
                    bytes_expected += 2 * 8 * K          # "2K percent" of a dense message
                elif f[i, t]:
                    assert len(idx) == 0                    # first message of a tensor is dense
                    assert np.array_equal(seg_post, x_pre[i, off:off + n])
                    bytes_expected += 2 * 4 * n
                else:
                    assert len(idx) == 0
                    assert np.array_equal(seg_post, seg_pre)
            off += n
    assert sparse_seen > 12
    assert o.stats()["bytes"] == bytes_expected


def test_topk_tie_break_prefers_lower_index():
    o = eo.Oracle(1, [8], mode=eo.FIXED, delta_fixed=0.0, topk=(3, 8))
    x = np.zeros((1, 8), np.float32)
    z = np.zeros_like(x)
    o.step(x, z, 0.0)                                   # first message: dense
    x[0] = [1, -2, 2, 0.5, -2, 2, -0.0, 1]              # |delta| = 1 2 2 .5 2 2 0 1
    o.step(x, z, 0.0)
    idx, val = o.outbox(0, 0)
    assert idx.tolist() == [1, 2, 4]                    # four ties at 2: lowest three indices
    assert val.tolist() == [-2.0, 2.0, -2.0]
    assert o.xhat()[0].tolist() == [0, -2, 2, 0, -2, 0, 0, 0]


def test_topk_with_k_equal_n_is_dense():
    P = 4
    wl_d = small(P=P, steps=15, lr=0.1, grad_sigma=0.01)
    wl_s = small(P=P, steps=15, lr=0.1, grad_sigma=0.01, topk=(1, 1))
    od, os_ = eo.from_workload(wl_d), eo.from_workload(wl_s)
    xd = W.distinct_init_params(wl_d).numpy().copy()
    xs = xd.copy()
    for k in range(wl_d.steps):
        g = wl_d.grads(k).numpy()
        od.step(xd, g, wl_d.lr)
        os_.step(xs, g, wl_s.lr)
        assert np.array_equal(od.flags(), os_.flags())
        assert np.array_equal(xd, xs)
        assert np.array_equal(od.xhat(), os_.xhat())
    sd, ss = od.stats(), os_.stats()
    assert sd["messages"] == ss["messages"]
    first = 2 * 4 * wl_d.N * P                         # the dense first messages
    assert ss["bytes"] - first == 2 * (sd["bytes"] - first)  # index + value: twice the size


def test_topk_counts_of_the_resnet18_tensors():
    o = eo.Oracle(1, [10, 64, 1728, 2359296], topk=(1, 100))
    assert [o.topk_count(t) for t in range(4)] == [1, 1, 18, 23593]
    o = eo.Oracle(1, [10, 64, 1728, 2359296], topk=(10, 100))
    assert [o.topk_count(t) for t in range(4)] == [1, 7, 173, 235930]


# ---------------------------------------------------------------------------------------
# Heavy-ball momentum (the Introduction names other training algorithms as extensions and
# gives none; the oracle takes v <- mu v + g, x <- average - gamma v, velocities local)
# ---------------------------------------------------------------------------------------
def test_momentum_zero_is_the_plain_update():
    wl = small(P=5, steps=7, lr=0.1, grad_sigma=0.01)
    a = eo.from_workload(wl)
    b = eo.from_workload(wl, momentum=0.0)
    xa = W.distinct_init_params(wl).numpy().copy()
    xb = xa.copy()
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        a.step(xa, g, wl.lr)
        b.step(xb, g, wl.lr)
        assert np.array_equal(xa, xb) and np.array_equal(a.flags(), b.flags())
        assert np.array_equal(b.velocity(), g)          # mu = 0: the velocity is the gradient
    assert a.stats() == b.stats()
    assert a.velocity() is None


def test_momentum_matches_torch_sgd_on_independent_replicas():
    """No messages (infinite threshold): every replica is torch.optim.SGD(momentum=mu) on its
    own parameters.  torch runs in fp64 with an fp64 velocity; the oracle stores both in fp32,
    so the two drift apart by roundings only."""
    import torch
    mu, lr, steps = 0.9, 0.05, 12
    wl = small(P=3, steps=steps, lr=lr, grad_sigma=0.02)
    o = eo.Oracle(3, wl.numel, mode=eo.FIXED, delta_fixed=INF, force_first_event=False, momentum=mu)
    x = W.distinct_init_params(wl).numpy().copy()
    p = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([p], lr=float(np.float32(lr)), momentum=mu)
    vmax = 0.0
    for k in range(steps):
        g = wl.grads(k).numpy()
        o.step(x, g, lr)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        ref = p.detach().numpy()
        buf = opt.state[p]["momentum_buffer"].numpy()
        vmax = max(vmax, float(np.abs(buf).max()))
        assert np.max(np.abs(o.velocity() - buf)) <= (k + 1) * 2.0 ** -23 * vmax
        assert np.max(np.abs(x - ref)) <= (k + 1) * 2.0 ** -23 * (float(np.abs(ref).max()) + vmax)
    assert o.stats()["messages"] == 0
    # a wrong sign or a velocity that is not accumulated is far outside those bounds
    plain = W.distinct_init_params(wl).numpy().astype(np.float64)
    for k in range(steps):
        plain -= float(np.float32(lr)) * wl.grads(k).numpy()
    assert np.max(np.abs(plain - p.detach().numpy())) > 1e-3


def test_momentum_closed_form_with_a_constant_gradient():
    """mu = 1/2, g = 1, gamma = 1/4, one replica: v_k = 2 - 2^(1-k) and
    x_k = x_0 - gamma * sum_{j<=k} v_j = x_0 - (2k - 2 + 2^(1-k)) / 4, all exact in fp32."""
    o = eo.Oracle(1, [4], mode=eo.FIXED, delta_fixed=INF, force_first_event=False, momentum=0.5)
    x = np.full((1, 4), 3.0, np.float32)
    g = np.ones((1, 4), np.float32)
    for k in range(1, 11):
        o.step(x, g, 0.25)
        assert np.all(o.velocity() == np.float32(2.0 - 2.0 ** (1 - k)))
        assert np.all(x == np.float32(3.0 - (2 * k - 2 + 2.0 ** (1 - k)) / 4))


@pytest.mark.parametrize("P", [2, 3, 6])
def test_momentum_zero_threshold_is_xw_minus_gamma_v(P):
    mu = 0.75
    wl = small(P=P, steps=6, lr=0.1, grad_sigma=0.01)
    o = eo.Oracle(P, wl.numel, mode=eo.FIXED, delta_fixed=0.0, force_first_event=False, momentum=mu)
    x = W.distinct_init_params(wl).numpy().copy()
    Wm = ring_matrix(P)
    v = np.zeros_like(x)
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        v = (mu * v.astype(np.float64) + g.astype(np.float64)).astype(np.float32)
        ref = Wm @ x.astype(np.float64) - np.float64(np.float32(wl.lr)) * v.astype(np.float64)
        o.step(x, g, wl.lr)
        assert np.array_equal(o.velocity(), v)
        assert np.all(np.abs(x.astype(np.float64) - ref) <= 0.5000001 * ulp32(ref) + 1e-300)


def test_momentum_reset_clears_the_velocity_and_range_is_checked():
    wl = small(P=2, steps=2)
    o = eo.from_workload(wl, momentum=0.9)
    x = W.distinct_init_params(wl).numpy().copy()
    o.step(x, wl.grads(0).numpy(), wl.lr)
    assert np.any(o.velocity() != 0)
    o.reset()
    assert np.all(o.velocity() == 0)
    for bad in (-0.1, 1.0, float("nan")):
        with pytest.raises(ValueError):
            eo.from_workload(wl, momentum=bad)



# ---------------------------------------------------------------------------------------
# after training: averaged model (last line of Algorithms A and B)
# ---------------------------------------------------------------------------------------
# ---------------------------------------------------------------------------------------
# Quantised messages (Section 7: quantization can be applied on top of the events; the scheme is
# the reading taken here, stated in the oracle's header)
# ---------------------------------------------------------------------------------------
def _exact_quantised_message(x_row, h_row, bits):
    """The reading restated with exact rational arithmetic: (E, new x_hat) of one tensor."""
    from fractions import Fraction
    L = (1 << (bits - 1)) - 1
    d = (x_row - h_row).astype(np.float32)                 # the fp32 differences the method ranks
    dmax = max((abs(Fraction(float(v))) for v in d), default=Fraction(0))
    E = 0
    if dmax > 0:
        E = -400
        while L * Fraction(2) ** E < dmax:
            E += 1
    out = np.empty_like(h_row)
    for e in range(len(d)):
        r = Fraction(float(d[e])) / Fraction(2) ** E
        lo = r.numerator // r.denominator                  # floor
        frac = r - lo
        q = lo + (1 if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1) else 0)   # ties to even
        assert abs(q) <= L
        exact = Fraction(float(h_row[e])) + q * Fraction(2) ** E
        out[e] = np.float32(float(exact))                  # to fp64 (correctly rounded), then to fp32
    return E, out


@pytest.mark.parametrize("bits", [2, 4, 8, 16])
def test_quantised_messages_against_exact_rational_arithmetic(bits):
    wl = small(P=4, numel=(1, 9, 64, 257), steps=6, lr=0.1, grad_sigma=0.02)
    o = eo.from_workload(wl, mode=eo.FIXED, delta_fixed=0.0, quant_bits=bits)      # every tensor sends every step
    x = W.distinct_init_params(wl).numpy().copy()
    off = np.concatenate([[0], np.cumsum(wl.numel)])
    L = (1 << (bits - 1)) - 1
    bytes_before = 0
    for k in range(wl.steps):
        h_before = o.xhat().copy()
        x_before = x.copy()
        o.step(x, wl.grads(k).numpy(), wl.lr)
        h_after, qe, qd = o.xhat(), o.quant_exponents(), o.quantised()
        payload = 0
        for i in range(wl.P):
            for t in range(wl.T):
                a, b = off[t], off[t + 1]
                if k == 0:
                    # the first message of a tensor goes out in full
                    assert qd[i, t] == 0 and np.array_equal(h_after[i, a:b], x_before[i, a:b])
                    payload += 4 * wl.numel[t]
                    continue
                assert qd[i, t] == 1
                E, want = _exact_quantised_message(x_before[i, a:b], h_before[i, a:b], bits)
                assert qe[i, t] == E
                assert np.array_equal(h_after[i, a:b], want)
                # round trip: what the receivers hold is within half a step of x (plus the two
                # roundings to fp32, of the difference and of the sum)
                err = np.abs(x_before[i, a:b].astype(np.float64) - h_after[i, a:b])
                slack = ulp32(x_before[i, a:b] - h_before[i, a:b]) / 2 + ulp32(h_after[i, a:b]) / 2
                assert np.all(err <= 2.0 ** E / 2 + slack)
                # E is the smallest exponent whose grid reaches the largest change
                dmax = float(np.abs((x_before[i, a:b] - h_before[i, a:b]).astype(np.float32)).max())
                assert L * 2.0 ** E >= dmax and (dmax == 0 or L * 2.0 ** (E - 1) < dmax)
                payload += 4 + (wl.numel[t] * bits + 7) // 8
        deg = 2
        assert o.stats()["bytes"] - bytes_before == deg * payload
        bytes_before = o.stats()["bytes"]


def test_quantised_changes_on_the_grid_are_reproduced_exactly():
    """Changes that are integer multiples of 2^e with the largest equal to L 2^e: E = e, every code
    is the multiple itself, and the receivers end up with x exactly."""
    bits, e = 6, -7
    L = (1 << (bits - 1)) - 1
    n = 50
    wl = W.synthetic(3, [n], steps=2, lr=0.0, grad_sigma=0.0)
    o = eo.from_workload(wl, mode=eo.FIXED, delta_fixed=0.0, quant_bits=bits)
    rng = np.random.default_rng(5)
    x = (rng.integers(-1000, 1000, size=(3, n)) * 2.0 ** -4).astype(np.float32)
    g = np.zeros_like(x)
    o.step(x, g, 0.0)                                   # first messages, in full: x_hat == x
    sent = o.xhat().copy()
    # lr = 0 and identical mailboxes: the average moves x; put it back on a chosen grid
    mult = rng.integers(-L, L + 1, size=(3, n))
    mult[:, 0] = L                                      # the largest change sits on the end of the grid
    x[:] = (sent.astype(np.float64) + mult * 2.0 ** e).astype(np.float32)
    assert np.array_equal((x - sent).astype(np.float32), (mult * 2.0 ** e).astype(np.float32))   # representable
    x_sent = x.copy()
    o.step(x, g, 0.0)
    assert np.all(o.quantised() == 1) and np.all(o.quant_exponents() == e)
    assert np.array_equal(o.xhat(), x_sent)


def test_thirty_two_bits_and_the_first_message_are_full_precision():
    wl = small(P=5, steps=8, lr=0.1, grad_sigma=0.01)
    a, b = eo.from_workload(wl), eo.from_workload(wl, quant_bits=32)
    xa = W.distinct_init_params(wl).numpy().copy()
    xb = xa.copy()
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        a.step(xa, g, wl.lr)
        b.step(xb, g, wl.lr)
        assert np.array_equal(xa, xb) and np.array_equal(a.xhat(), b.xhat())
    assert a.stats() == b.stats() and a.stats()["events"] > wl.P * wl.T
    assert b.quantised() is None
    with pytest.raises(ValueError):
        eo.from_workload(wl, quant_bits=1)
    with pytest.raises(ValueError):
        eo.from_workload(wl, quant_bits=17)


@pytest.mark.parametrize("bits", [3, 8])
def test_quantised_topk_messages_against_brute_force_and_exact_arithmetic(bits):
    """Both compressions together: the K_t entries of largest |x - x_hat| (brute-force lexsort, ties
    to the lower index), their values sent as codes of the change on the grid of the largest change
    (exact rational arithmetic), x_hat untouched elsewhere, 4 + 4 K + ceil(K b / 8) bytes."""
    from fractions import Fraction
    wl = small(P=3, numel=(1, 40, 257), steps=5, lr=0.1, grad_sigma=0.02, topk=(10, 100))
    o = eo.from_workload(wl, mode=eo.FIXED, delta_fixed=0.0, quant_bits=bits)
    x = W.distinct_init_params(wl).numpy().copy()
    off = np.concatenate([[0], np.cumsum(wl.numel)])
    L = (1 << (bits - 1)) - 1
    bytes_before = 0
    for k in range(wl.steps):
        h_before, x_before = o.xhat().copy(), x.copy()
        o.step(x, wl.grads(k).numpy(), wl.lr)
        h_after = o.xhat()
        payload = 0
        for i in range(wl.P):
            for t in range(wl.T):
                a, b = off[t], off[t + 1]
                n = wl.numel[t]
                if k == 0:
                    assert np.array_equal(h_after[i, a:b], x_before[i, a:b])
                    payload += 4 * n
                    continue
                K = o.topk_count(t)
                d = (x_before[i, a:b] - h_before[i, a:b]).astype(np.float32)
                keys = np.abs(d).view(np.uint32)
                order = np.lexsort((np.arange(n), -keys.astype(np.int64)))      # key descending, index ascending
                chosen = np.sort(order[:K])
                idx, val = o.outbox(i, t)
                assert np.array_equal(idx, chosen)
                dmax = max(abs(Fraction(float(v))) for v in d)
                E = 0
                if dmax > 0:
                    E = -400
                    while L * Fraction(2) ** E < dmax:
                        E += 1
                assert o.quant_exponents()[i, t] == E and o.quantised()[i, t] == 1
                want = h_before[i, a:b].copy()
                for e in chosen:
                    r = Fraction(float(d[e])) / Fraction(2) ** E
                    lo = r.numerator // r.denominator
                    frac = r - lo
                    q = lo + (1 if frac > Fraction(1, 2) or (frac == Fraction(1, 2) and lo % 2 == 1) else 0)
                    want[e] = np.float32(float(Fraction(float(h_before[i, a + e])) + q * Fraction(2) ** E))
                assert np.array_equal(h_after[i, a:b], want)
                assert np.array_equal(val, want[chosen])            # the message's values: what arrives
                payload += 4 + 4 * K + (K * bits + 7) // 8
        assert o.stats()["bytes"] - bytes_before == 2 * payload
        bytes_before = o.stats()["bytes"]


def test_quantised_topk_with_every_entry_selected_is_the_quantised_dense_message():
    wl = small(P=4, numel=(9, 64, 300), steps=8, lr=0.1, grad_sigma=0.02)
    dense = eo.from_workload(wl, quant_bits=6)
    wl_all = small(P=4, numel=(9, 64, 300), steps=8, lr=0.1, grad_sigma=0.02, topk=(1, 1))
    sparse = eo.from_workload(wl_all, quant_bits=6)
    xa = W.distinct_init_params(wl).numpy().copy()
    xb = xa.copy()
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        dense.step(xa, g, wl.lr)
        sparse.step(xb, g, wl.lr)
        assert np.array_equal(xa, xb) and np.array_equal(dense.xhat(), sparse.xhat())
        assert np.array_equal(dense.flags(), sparse.flags())
        assert np.array_equal(dense.quant_exponents(), sparse.quant_exponents())
    assert dense.stats()["events"] == sparse.stats()["events"] > wl.P * wl.T


def test_quantised_run_keeps_the_error_bound_and_saves_bytes():
    """With the adaptive threshold the trigger still bounds what the neighbours are missing:
    after every step ||x_before - x_hat|| of a tensor that did not fire is below the threshold it
    was tested against (Section 5), quantised or not -- the un-sent remainder is part of the tested
    norm -- and the run sends fewer bytes than the same run in full precision."""
    wl = small(P=4, numel=(40, 300, 1000), steps=30, lr=0.1, grad_sigma=0.02)
    full, q8 = eo.from_workload(wl), eo.from_workload(wl, quant_bits=8)
    xf = W.distinct_init_params(wl).numpy().copy()
    xq = xf.copy()
    for k in range(wl.steps):
        g = wl.grads(k).numpy()
        full.step(xf, g, wl.lr)
        before = xq.copy()
        q8.step(xq, g, wl.lr)
        fl, nr, th = q8.flags(), q8.norms(), q8.thresholds_used()
        assert np.all(nr[fl == 0] < th[fl == 0])
        assert np.all(np.isfinite(before)) and np.all(np.isfinite(q8.xhat()))
    assert 0 < q8.stats()["bytes"] < full.stats()["bytes"]
    assert np.any(q8.quantised() == 1) or q8.stats()["events"] > wl.P * wl.T


def test_average_model_and_consensus_distance():
    wl = small(P=5)
    o = eo.from_workload(wl)
    x = W.distinct_init_params(wl).numpy()
    x64 = x.astype(np.float64)
    mean = x64.mean(axis=0)
    assert np.all(np.abs(o.average_model(x) - mean) <= ulp32(mean))
    assert o.consensus_distance(x) == pytest.approx(((x64 - mean) ** 2).sum(), rel=1e-12)


# ---------------------------------------------------------------------------------------
# the input generator (shared by both sides): tensor form == pure-Python definition
# ---------------------------------------------------------------------------------------
def test_generator_matches_python_definition():
    base = W.stream_base(W.MASTER_SEED, W.STREAM_GRAD, 3, 1)
    t = W.ih8_integers(base, 5, 50, "cpu").tolist()
    assert t == [W.ih8_integers_py(base, e) for e in range(5, 55)]
    z = W.ih8_integers(base, 0, 200000, "cpu").double()
    assert abs(z.mean().item()) < 4 * W.IH8_STD / math.sqrt(200000)
    assert z.std().item() == pytest.approx(W.IH8_STD, rel=0.01)


def test_workload_sizes():
    sizes = {1: (4, 6, 52650), 2: (8, 59, 269722), 3: (16, 62, 11173962),
             4: (8, 62, 11173962), 5: (64, 161, 25557032)}
    for idx, (P, T, N) in sizes.items():
        for wl in W.config(idx):
            assert (wl.P, wl.T, wl.N) == (P, T, N)
