"""CUDA library (through the C ABI) against the CPU oracle, element by element."""
import os

import numpy as np
import pytest
import torch

from paper_2103_07454_b200 import binding as B
from paper_2103_07454_b200 import workload as W

pytestmark = pytest.mark.gpu

from parity_harness import lockstep  # noqa: E402

RAGGED = [1, 3, 4, 5, 31, 32, 33, 1023, 1024, 1025, 4095, 4096, 4097, 10000, (1 << 20) + 1]
INF = float("inf")


@pytest.mark.parametrize("P", [1, 2, 3, 4, 5, 6, 7, 11, 64, 130])
@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_REGISTER, B.FUSED_AUTO])
def test_ragged_dense(P, carry, kernel):
    """Under the automatic choice the cases without the 2^20 + 1 element tensor and with at most
    16 replicas run as one launch per iteration; the others take the pipelined kernel."""
    numel = RAGGED if P <= 4 else RAGGED[:-1]
    wl = W.synthetic(P, numel, steps=12, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=carry, fused_kernel=kernel)
    assert rep.params_bit_exact and not rep.near_threshold
    assert 0 < rep.events < P * wl.T * wl.steps


@pytest.mark.parametrize("own,con", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_REGISTER])
def test_variants_own_term_and_change_of_norm(own, con, carry, kernel):
    wl = W.synthetic(5, RAGGED[:-1], steps=16, lr=0.1, grad_sigma=0.01, history_len=2)
    rep = lockstep(wl, init="distinct", carry=carry, fused_kernel=kernel,
                   oracle_kw=dict(own_last_sent=own, change_of_norm=con))
    assert rep.params_bit_exact and not rep.near_threshold
    assert 0 < rep.events < 5 * wl.T * wl.steps


@pytest.mark.parametrize("P,hops", [(1, 2), (2, 2), (3, 2), (4, 2), (5, 2), (6, 2), (7, 3), (8, 3), (9, 4),
                                    (13, 4), (16, 2), (16, 3), (16, 8), (64, 2)])
@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_REGISTER])
def test_more_neighbours_per_side(P, hops, carry, kernel):
    """Rings of at least 2 hops + 1 replicas with up to 4 hops take the staged kernel under the
    default kernel choice and the plain one under the other; the rest always take the plain one."""
    wl = W.synthetic(P, RAGGED[:-1], steps=10, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=carry, oracle_kw=dict(hops=hops), fused_kernel=kernel)
    assert rep.params_bit_exact and not rep.near_threshold


def test_more_neighbours_with_topk_and_variants():
    wl = W.synthetic(6, RAGGED[:-1], steps=12, lr=0.1, grad_sigma=0.01, topk=(5, 100))
    rep = lockstep(wl, init="distinct", carry=True, outbox_samples=32,
                   oracle_kw=dict(hops=2, own_last_sent=True, change_of_norm=True))
    assert rep.params_bit_exact


@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_AUTO])
def test_geometric_threshold_cap(carry, kernel):
    wl = W.synthetic(4, RAGGED[:-1], steps=20, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=carry, oracle_kw=dict(threshold_cap=(1e-3, 0.7)),
                   fused_kernel=kernel)
    free = lockstep(wl, init="distinct", carry=carry, fused_kernel=kernel)
    assert rep.params_bit_exact and not rep.near_threshold
    assert rep.events > free.events          # a shrinking bound makes tensors communicate more


def _random_links(P, T, p_up, seed):
    rng = np.random.default_rng(seed)

    def fn(k):
        if k % 7 == 6:
            return None                      # NULL mask: everything outstanding arrives
        return (rng.random((P, T)) < p_up).astype(np.uint8)
    return fn


@pytest.mark.parametrize("P,hops", [(1, 1), (2, 1), (3, 1), (5, 1), (16, 1), (5, 2), (9, 3), (4, 2), (12, 4)])
@pytest.mark.parametrize("p_up", [0.0, 0.5, 1.0])
@pytest.mark.parametrize("carry", [False, True])
def test_intermittent_delivery_dense(P, hops, p_up, carry):
    """With the carried norm the averaging kernel also leaves the next change norms, taken
    against what every replica has SENT (not what its neighbours hold)."""
    wl = W.synthetic(P, RAGGED[:-1], steps=16, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", oracle_kw=dict(hops=hops), carry=carry,
                   deliver_fn=_random_links(P, wl.T, p_up, seed=P * 10 + hops))
    assert rep.params_bit_exact and not rep.near_threshold
    assert rep.launches == (wl.steps * 2 + 1 if carry else wl.steps * 3)


@pytest.mark.parametrize("con", [False, True])
def test_intermittent_delivery_topk(con):
    wl = W.synthetic(6, RAGGED[:-1], steps=16, lr=0.1, grad_sigma=0.01, topk=(5, 100))
    rep = lockstep(wl, init="distinct", outbox_samples=32, carry=True,
                   oracle_kw=dict(change_of_norm=con), deliver_fn=_random_links(6, wl.T, 0.4, seed=3))
    assert rep.params_bit_exact


def _random_case(seed):
    """One seeded draw over the options of a context; combinations the library documents as
    unavailable (delivery masks with the own-term variant) are not drawn."""
    rng = np.random.default_rng(1000 + seed)
    P = int(rng.integers(1, 12))
    sizes = [int(v) for v in rng.choice(RAGGED[:-1], size=int(rng.integers(1, 6)), replace=False)]
    topk = [None, (1, 100), (7, 100), (1, 2)][int(rng.integers(0, 4))]
    hops = int(rng.integers(1, 5))
    deliver = bool(rng.integers(0, 3) == 0)
    okw = dict(hops=hops, history_len=int(rng.integers(1, 5)), horizon=float(rng.choice([0.5, 1.0, 2.0])),
               own_last_sent=bool(rng.integers(0, 2)) and not deliver,
               change_of_norm=bool(rng.integers(0, 2)))
    if rng.integers(0, 4) == 0:
        okw["threshold_cap"] = (1e-3, 0.8)
    if rng.integers(0, 5) == 0:
        okw.update(mode=1, delta_fixed=float(rng.choice([0.0, 0.01])), force_first_event=bool(rng.integers(0, 2)))
    if rng.integers(0, 3) == 0:
        okw["momentum"] = float(rng.choice([0.0, 0.5, 0.9]))
    if rng.integers(0, 2) == 0:
        okw["quant_bits"] = int(rng.choice([3, 8, 12]))
    return dict(P=P, sizes=sizes, topk=topk, okw=okw, carry=bool(rng.integers(0, 2)),
                kernel=[B.FUSED_PIPELINED, B.FUSED_REGISTER][int(rng.integers(0, 2))],
                deliver=_random_links(P, len(sizes), float(rng.choice([0.3, 0.8])), seed) if deliver else None)


@pytest.mark.parametrize("seed", range(48))
def test_random_option_combinations(seed):
    case = _random_case(seed)
    wl = W.synthetic(case["P"], case["sizes"], steps=14, lr=0.1, grad_sigma=0.01, topk=case["topk"],
                     seed=77 + seed)
    rep = lockstep(wl, init="distinct", carry=case["carry"], fused_kernel=case["kernel"],
                   oracle_kw=case["okw"], deliver_fn=case["deliver"], outbox_samples=16)
    assert rep.params_bit_exact, case


@pytest.mark.parametrize("seed", range(16))
def test_random_momentum_and_kernel_choice_combinations(seed):
    """Seeded draws over what momentum and the automatic kernel choice combine with: ring size,
    tensor sizes, dense / Top-K, history, horizon, threshold bound, fixed thresholds, carried norm."""
    rng = np.random.default_rng(5000 + seed)
    P = int(rng.integers(1, 20))
    sizes = [int(v) for v in rng.choice(RAGGED[:-1], size=int(rng.integers(1, 7)), replace=False)]
    topk = [None, None, (1, 100), (1, 3)][int(rng.integers(0, 4))]
    okw = dict(history_len=int(rng.integers(1, 5)), horizon=float(rng.choice([0.5, 1.0, 2.0])))
    if rng.integers(0, 2):
        okw["momentum"] = float(rng.choice([0.0, 0.5, 0.9, 0.99]))
    if rng.integers(0, 4) == 0:
        okw["threshold_cap"] = (1e-3, 0.8)
    if rng.integers(0, 5) == 0:
        okw.update(mode=1, delta_fixed=float(rng.choice([0.0, 0.01])), force_first_event=bool(rng.integers(0, 2)))
    kernel = [B.FUSED_PIPELINED, B.FUSED_AUTO][int(rng.integers(0, 2))]
    wl = W.synthetic(P, sizes, steps=14, lr=0.1, grad_sigma=0.01, topk=topk, seed=177 + seed)
    rep = lockstep(wl, init="distinct", carry=bool(rng.integers(0, 2)), fused_kernel=kernel, oracle_kw=okw,
                   outbox_samples=16)
    assert rep.params_bit_exact, (P, sizes, topk, okw, kernel)


def test_delivery_masks_enabled_mid_run_and_refusals():
    from oracle import eg_oracle as eo
    wl = W.synthetic(4, [5, 1000, 4097], steps=12, lr=0.1, grad_sigma=0.01)
    o, eg = eo.from_workload(wl), B.from_workload(wl)
    xh = W.distinct_init_params(wl).numpy().copy()
    xd = eg.to_layout(torch.from_numpy(xh))
    rng = np.random.default_rng(1)
    with pytest.raises(B.EventGradError):          # a mask before the second copy exists
        eg.step_masked(xd, xd, 0.1, torch.ones(4 * wl.T, dtype=torch.uint8, device="cuda"))
    for k in range(wl.steps):
        g = wl.grads(k)
        if k == 4:
            eg.enable_delivery_masks()
            o.enable_delivery_masks()
        mask = (rng.random((4, wl.T)) < 0.5).astype(np.uint8) if k >= 4 else None
        o.step(xh, g.numpy(), wl.lr, deliver=mask)
        if mask is None:
            eg.step(xd, eg.to_layout(g), wl.lr)
        else:
            eg.step_masked(xd, eg.to_layout(g), wl.lr, torch.from_numpy(mask).cuda())
        assert np.array_equal(eg.last_decisions()[0], o.flags())
    assert np.array_equal(eg.from_layout(xd).cpu().numpy(), xh)
    assert np.array_equal(eg.from_layout(eg.received()).numpy(), o.received())
    eg.close()


def test_checkpoint_with_messages_in_flight_and_velocities():
    """A checkpoint carries the delivery state (received copies, what is still in flight, the
    arrival count) and the velocities: a context restored from it continues bit for bit."""
    wl = W.synthetic(5, [5, 1000, 4097], steps=12, lr=0.1, grad_sigma=0.01, history_len=2)
    rng = np.random.default_rng(11)
    masks = [torch.from_numpy((rng.random((5, wl.T)) < 0.4).astype(np.uint8)).cuda() for _ in range(wl.steps)]
    g = None

    def run(eg, x, k0, k1):
        for k in range(k0, k1):
            eg.step_masked(x, eg.to_layout(wl.grads(k, "cuda")), wl.lr, masks[k])

    a = B.from_workload(wl)
    a.enable_delivery_masks()
    xa = a.to_layout(W.distinct_init_params(wl, "cuda"))
    run(a, xa, 0, 6)
    assert a.delivery_status()[0].any()            # something is in flight at the checkpoint
    blob, x_mid = a.export_state(), xa.clone()
    run(a, xa, 6, 12)
    b = B.from_workload(wl)
    with pytest.raises(B.EventGradError):
        b.import_state(blob)                       # not a context with delivery masks
    b.enable_delivery_masks()
    b.import_state(blob)
    xb = x_mid.clone()
    run(b, xb, 6, 12)
    assert torch.equal(xa, xb) and a.stats() == b.stats()
    assert torch.equal(a.received(), b.received()) and torch.equal(a.mailboxes(), b.mailboxes())
    pa, pb = a.delivery_status(), b.delivery_status()
    assert np.array_equal(pa[0], pb[0]) and pa[1] == pb[1]
    a.close(); b.close()

    # momentum: the velocities travel with the state
    a, b = B.from_workload(wl), B.from_workload(wl)
    a.set_momentum(0.9)
    xa = a.to_layout(W.distinct_init_params(wl, "cuda"))
    for k in range(6):
        a.step(xa, a.to_layout(wl.grads(k, "cuda")), wl.lr)
    blob, xb = a.export_state(), xa.clone()
    with pytest.raises(B.EventGradError):
        b.import_state(blob)                       # no velocity buffer there
    b.set_momentum(0.5)
    with pytest.raises(B.EventGradError):
        b.import_state(blob)                       # another coefficient
    b.set_momentum(0.9)
    b.import_state(blob)
    for k in range(6, 12):
        gk = a.to_layout(wl.grads(k, "cuda"))
        a.step(xa, gk, wl.lr)
        b.step(xb, gk, wl.lr)
    assert torch.equal(xa, xb) and torch.equal(a.velocity(), b.velocity()) and a.stats() == b.stats()
    a.close(); b.close()


def test_checkpoint_is_refused_by_a_differently_configured_context():
    wl = W.synthetic(6, [5, 1000, 4097], steps=4, lr=0.1, grad_sigma=0.01, history_len=2)
    src = B.from_workload(wl)
    src.set_threshold_cap(1e-3, 0.9)
    x = src.to_layout(W.distinct_init_params(wl, "cuda"))
    for k in range(3):
        src.step(x, src.to_layout(wl.grads(k, "cuda")), wl.lr)
    blob = src.export_state()
    same = B.from_workload(wl)
    same.set_threshold_cap(1e-3, 0.9)
    same.import_state(blob)
    others = [B.from_workload(wl, hops=2), B.from_workload(wl, horizon=2.0), B.from_workload(wl, delta_init=0.5),
              B.from_workload(wl, mode=B.THRESH_FIXED, delta_fixed=0.1), B.from_workload(wl, force_first_event=False),
              B.from_workload(wl), B.from_workload(wl)]
    others[-1].set_threshold_cap(1e-3, 0.8)
    for other in others:
        with pytest.raises(B.EventGradError):
            other.import_state(blob)
        other.close()
    # the bound continues from the restored iteration
    y = x.clone()
    g = src.to_layout(wl.grads(3, "cuda"))
    src.step(x, g, wl.lr)
    same.step(y, g, wl.lr)
    assert torch.equal(x, y)
    for a, b in zip(src.last_decisions(), same.last_decisions()):
        assert np.array_equal(a, b)
    src.close(); same.close()


def test_variant_with_topk():
    wl = W.synthetic(4, RAGGED[:-1], steps=14, lr=0.1, grad_sigma=0.01, topk=(5, 100))
    rep = lockstep(wl, init="distinct", carry=True, outbox_samples=64,
                   oracle_kw=dict(own_last_sent=True, change_of_norm=True))
    assert rep.params_bit_exact


def test_variant_only_before_the_first_step():
    wl = W.synthetic(2, [8, 100])
    eg = B.from_workload(wl)
    eg.set_variant(True, True)
    x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
    eg.step(x, eg.to_layout(wl.grads(0, "cuda")), 0.1)
    with pytest.raises(B.EventGradError):
        eg.set_variant(False, False)
    eg.reset()
    eg.set_variant(False, False)
    eg.close()


def test_resynchronise_through_the_checkpoint_interface():
    """The harness's recovery path (used after a reported near-threshold disagreement): the
    CUDA context takes over the oracle's whole state and the comparison goes on."""
    import numpy as np
    from oracle import eg_oracle as eo
    from parity_harness import resynchronise
    wl = W.synthetic(3, [5, 1000, 4097], steps=10, lr=0.1, grad_sigma=0.01, history_len=3)
    o, eg = eo.from_workload(wl), B.from_workload(wl)
    xh = W.distinct_init_params(wl).numpy().copy()
    xd = eg.to_layout(torch.from_numpy(xh))
    for k in range(4):                      # only the oracle advances
        o.step(xh, wl.grads(k).numpy(), wl.lr)
    resynchronise(eg, o, xd, xh)
    for k in range(4, 10):
        g = wl.grads(k)
        o.step(xh, g.numpy(), wl.lr)
        eg.step(xd, eg.to_layout(g), wl.lr)
        f, _, _ = eg.last_decisions()
        assert np.array_equal(f, o.flags())
    assert eg.stats() == o.stats()
    assert np.array_equal(eg.from_layout(xd).cpu().numpy(), xh)


@pytest.mark.parametrize("hist,horizon", [(1, 1.0), (4, 1.0), (2, 0.5)])
@pytest.mark.parametrize("kernel,carry", [(B.FUSED_PIPELINED, False), (B.FUSED_AUTO, False), (B.FUSED_AUTO, True)])
def test_history_and_horizon(hist, horizon, kernel, carry):
    wl = W.synthetic(5, RAGGED[:-1], steps=25, lr=0.1, grad_sigma=0.01, history_len=hist,
                     horizon=horizon)
    rep = lockstep(wl, init="distinct", fused_kernel=kernel, carry=carry)
    assert rep.params_bit_exact and not rep.near_threshold


@pytest.mark.parametrize("delta,force", [(0.0, False), (INF, False), (INF, True), (0.02, True)])
@pytest.mark.parametrize("kernel,carry", [(B.FUSED_PIPELINED, False), (B.FUSED_AUTO, False), (B.FUSED_AUTO, True)])
def test_fixed_threshold_modes(delta, force, kernel, carry):
    wl = W.synthetic(4, RAGGED[:-1], steps=6, lr=0.1, grad_sigma=0.01)
    kw = dict(mode=1, delta_fixed=delta, force_first_event=force)
    rep = lockstep(wl, init="distinct", oracle_kw=kw, fused_kernel=kernel, carry=carry)
    assert rep.params_bit_exact
    if delta == 0.0:
        assert rep.events == 4 * wl.T * wl.steps
    if delta == INF:
        assert rep.events == (4 * wl.T if force else 0)


@pytest.mark.parametrize("frac", [(1, 100), (10, 100), (1, 1)])
@pytest.mark.parametrize("P", [1, 3, 8])
def test_ragged_topk(P, frac):
    wl = W.synthetic(P, RAGGED, steps=14, lr=0.1, grad_sigma=0.01, topk=frac)

    def ties(k, g):  # engineered ties: many equal |delta|, and exact zeros
        g[:, 3000:9000] = torch.round(g[:, 3000:9000] * 256) / 256
        g[:, 12000:12500] = 0.0
        return g

    rep = lockstep(wl, init="distinct", outbox_samples=10 ** 6, grad_hook=ties)
    assert rep.params_bit_exact and rep.sparse_checked > 10


@pytest.mark.parametrize("separate", [False, True])
def test_topk_degenerate_all_keys_equal(separate, monkeypatch):
    """Threshold 0 with zero gradients and identical replicas: every |x - x_hat| is exactly 0
    from the third step on, so all keys tie, every element is a candidate and the message is
    the first K_t indices."""
    if separate:
        monkeypatch.setenv("EG_TOPK_SEPARATE_LAUNCHES", "1")
    wl = W.synthetic(3, [1, 5, 33, 4095, 4096, 4097, 20000], steps=6, lr=0.1, grad_sigma=0.01, topk=(7, 100))

    def zero_after_first(k, g):
        return g if k == 0 else torch.zeros_like(g)

    rep = lockstep(wl, oracle_kw=dict(mode=1, delta_fixed=0.0), outbox_samples=10 ** 6,
                   grad_hook=zero_after_first)
    assert rep.params_bit_exact and rep.events == 3 * wl.T * wl.steps and rep.sparse_checked >= 3 * wl.T * 4


def test_topk_with_separate_launches(monkeypatch):
    """The single-phase Top-K launches (fallback where a cooperative launch is unavailable)."""
    monkeypatch.setenv("EG_TOPK_SEPARATE_LAUNCHES", "1")
    wl = W.synthetic(3, RAGGED, steps=10, lr=0.1, grad_sigma=0.01, topk=(10, 100))
    rep = lockstep(wl, init="distinct", outbox_samples=64)
    assert rep.params_bit_exact and rep.sparse_checked > 5
    assert rep.launches == 10 * 18


@pytest.mark.parametrize("separate", [False, True])
@pytest.mark.parametrize("margin", ["-8", "0", "5"])
def test_topk_guess_and_exact_repeat(separate, margin, monkeypatch):
    """Tensors large enough to be sampled (2^20 + 1 and 300,000 elements at 1 % and 7 %).  A negative
    margin makes every guessed bin too high, so every such message takes the exact repeat; margin 0
    fails about every other time; the default margin practically never.  The messages are the
    oracle's in all three cases."""
    monkeypatch.setenv("EG_TOPK_GUESS_MARGIN", margin)
    if separate:
        monkeypatch.setenv("EG_TOPK_SEPARATE_LAUNCHES", "1")
    for frac in ((1, 100), (7, 100)):
        wl = W.synthetic(3, [5, 300000, 4097, (1 << 20) + 1, 70000], steps=8, lr=0.1, grad_sigma=0.01, topk=frac)
        rep = lockstep(wl, init="distinct", outbox_samples=10 ** 6, carry=True)
        assert rep.params_bit_exact and rep.sparse_checked > 10
        if margin == "-8":
            assert rep.topk_repeats >= 6          # the two sampled tensors of three replicas, several iterations
        if margin == "5":
            assert rep.topk_repeats <= 1


@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_REGISTER])
def test_topk_carry_norm(kernel):
    wl = W.synthetic(4, RAGGED, steps=14, lr=0.1, grad_sigma=0.01, topk=(5, 100))
    rep = lockstep(wl, init="distinct", carry=True, outbox_samples=64, fused_kernel=kernel)
    assert rep.params_bit_exact and rep.sparse_checked > 10


@pytest.mark.parametrize("P", [1, 2, 3, 5, 16])
@pytest.mark.parametrize("carry", [False, True])
def test_momentum_ragged_dense(P, carry):
    numel = RAGGED if P <= 3 else RAGGED[:-1]
    wl = W.synthetic(P, numel, steps=12, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=carry, oracle_kw=dict(momentum=0.9))
    assert rep.params_bit_exact and not rep.near_threshold
    assert 0 < rep.events < P * wl.T * wl.steps


@pytest.mark.parametrize("carry", [False, True])
def test_momentum_with_topk_and_history(carry):
    wl = W.synthetic(4, RAGGED, steps=14, lr=0.1, grad_sigma=0.01, topk=(5, 100), history_len=3)
    rep = lockstep(wl, init="distinct", carry=carry, outbox_samples=32, oracle_kw=dict(momentum=0.5))
    assert rep.params_bit_exact and rep.sparse_checked > 10


def test_momentum_zero_reset_roundtrip_and_refusals():
    wl = W.synthetic(3, RAGGED[:-1], steps=6, lr=0.1, grad_sigma=0.01)
    dev = torch.device("cuda")
    plain, mom = B.from_workload(wl), B.from_workload(wl)
    mom.set_momentum(0.0)
    xa = plain.to_layout(W.distinct_init_params(wl, dev))
    xb = xa.clone()
    for k in range(wl.steps):
        g = plain.to_layout(wl.grads(k, dev))
        plain.step(xa, g, wl.lr)
        mom.step(xb, g, wl.lr)
    assert torch.equal(xa, xb) and plain.stats() == mom.stats()      # mu = 0: the plain update, bit for bit
    v = mom.velocity()
    assert torch.equal(mom.from_layout(v), wl.grads(wl.steps - 1))
    # read / write round trip; reset clears; turning it off leaves the plain path
    w = torch.randn_like(v)
    mom.write_velocity(w)
    assert torch.equal(mom.velocity(), w)
    mom.reset()
    assert not mom.velocity().any()
    mom.set_momentum(None)
    plain.reset()
    xa = plain.to_layout(W.distinct_init_params(wl, dev))
    xb = xa.clone()
    g = plain.to_layout(wl.grads(0, dev))
    plain.step(xa, g, wl.lr)
    mom.step(xb, g, wl.lr)
    assert torch.equal(xa, xb) and not mom.velocity().any()
    with pytest.raises(B.EventGradError):
        plain.velocity()                      # never enabled: no buffer
    for bad in (-0.5, 1.0, float("nan")):
        with pytest.raises(B.EventGradError):
            mom.set_momentum(bad)
    for e in (plain, mom):
        e.close()


@pytest.mark.parametrize("what", ["hops2", "hops3_small_ring", "own_last_sent", "change_of_norm", "delivery",
                                  "delivery_hops", "register", "topk_hops", "everything"])
@pytest.mark.parametrize("carry", [False, True])
def test_momentum_with_every_other_option(what, carry):
    """Heavy-ball momentum next to more neighbours, the other readings, intermittent delivery, the
    register kernel and Top-K: velocities, parameters, mailboxes and counters are the oracle's."""
    okw, kw, topk, P = dict(momentum=0.9), {}, None, 7
    if what == "hops2":
        okw.update(hops=2)
    elif what == "hops3_small_ring":
        okw.update(hops=3); P = 4
    elif what == "own_last_sent":
        okw.update(own_last_sent=True)
    elif what == "change_of_norm":
        okw.update(change_of_norm=True)
    elif what == "delivery":
        kw.update(deliver_fn=_random_links(P, len(RAGGED) - 1, 0.5, seed=5))
    elif what == "delivery_hops":
        okw.update(hops=2); kw.update(deliver_fn=_random_links(P, len(RAGGED) - 1, 0.5, seed=6))
    elif what == "register":
        kw.update(fused_kernel=B.FUSED_REGISTER)
    elif what == "topk_hops":
        okw.update(hops=2); topk = (5, 100)
    else:
        okw.update(hops=2, change_of_norm=True, history_len=3, threshold_cap=(1e-3, 0.8)); topk = (5, 100)
        kw.update(deliver_fn=_random_links(P, len(RAGGED) - 1, 0.6, seed=7))
    wl = W.synthetic(P, RAGGED[:-1], steps=12, lr=0.1, grad_sigma=0.01, topk=topk)
    rep = lockstep(wl, init="distinct", carry=carry, oracle_kw=okw, outbox_samples=16, **kw)
    assert rep.params_bit_exact and not rep.near_threshold


def test_momentum_resnet18_shapes_p16():
    """Many tiles, tensors of 10 ... 2.4 M elements, carried norm; the oracle follows a sample."""
    (wl,) = W.config(3)
    rep = lockstep(wl, steps=12, tensors=_sample_tensors(wl), carry=True, check_every=3,
                   oracle_kw=dict(momentum=0.9))
    assert rep.params_bit_exact


def test_quantised_resnet18_shapes_p16():
    """The 16-replica ResNet-18 ring with 8-bit messages: many tiles per tensor, the walking form of
    the averaging kernel, carried norm; the oracle follows a sample of the tensors."""
    (wl,) = W.config(3)
    rep = lockstep(wl, steps=12, tensors=_sample_tensors(wl), carry=True, check_every=3,
                   oracle_kw=dict(quant_bits=8))
    assert rep.params_bit_exact and rep.quantised_checked > 50


def test_quantised_topk_resnet18_shapes_p8():
    """The 8-replica ResNet-18 ring with Top-K 1 % messages whose values go out as 4-bit codes."""
    wl = W.config(4)[0]
    rep = lockstep(wl, steps=40, tensors=_sample_tensors(wl), carry=True, check_every=5,
                   oracle_kw=dict(quant_bits=4), outbox_samples=16)
    assert rep.params_bit_exact and rep.quantised_checked > 50 and rep.sparse_checked > 10


@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_AUTO])
def test_config1_mlp(carry, kernel):
    (wl,) = W.config(1)
    rep = lockstep(wl, carry=carry, fused_kernel=kernel)
    assert rep.params_bit_exact and not rep.near_threshold
    if kernel == B.FUSED_AUTO:      # one launch per iteration (plus the norm pass when nothing is carried)
        assert rep.launches == (wl.steps + 1 if carry else 2 * wl.steps)


@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("kernel", [B.FUSED_PIPELINED, B.FUSED_AUTO])
def test_config2_resnet20(carry, kernel):
    (wl,) = W.config(2)
    rep = lockstep(wl, carry=carry, fused_kernel=kernel)
    assert rep.params_bit_exact and not rep.near_threshold
    if kernel == B.FUSED_AUTO:
        assert rep.launches == (wl.steps + 1 if carry else 2 * wl.steps)


def _report(name, rep):
    """What a configured run did, on the test log (shown with -s or on failure)."""
    print(f"{name}: steps {rep.steps}, events {rep.events}, sparse messages checked {rep.sparse_checked}, "
          f"Top-K messages selected again exactly {rep.topk_repeats}, "
          f"largest norm error {rep.max_norm_rel:.2e} of its tolerance, parameters bit-exact {rep.params_bit_exact}, "
          f"decisions within 1e-6 of the threshold that differed {rep.near_threshold}; seconds spent on "
          + ", ".join(f"{k} {v:.1f}" for k, v in rep.seconds.items()))


@pytest.mark.parametrize("carry", [False, True])
def test_config3_resnet18_p16(carry):
    """Configuration 3 as configured: 100 iterations, all 62 tensors, both norm variants."""
    (wl,) = W.config(3)
    rep = lockstep(wl, carry=carry, check_every=5)
    _report(f"{wl.name} carry={carry}", rep)
    assert rep.steps == wl.steps == 100
    assert rep.params_bit_exact and not rep.near_threshold
    assert rep.launches == (wl.steps * 2 + 1 if carry else wl.steps * 3)


def _sample_tensors(wl, n_small=6, n_mid=3, n_big=2):
    order = np.argsort(wl.numel)
    mid = len(order) // 2
    pick = list(order[:n_small]) + list(order[mid:mid + n_mid]) + list(order[-n_big:])
    return sorted(set(int(t) for t in pick))


def _size_classes_and_boosted(wl):
    """Tensors the oracle follows at configuration 5: the first tensor of every distinct size
    (all 22 size classes of ResNet-50, the 2048 x 1000 classifier among them) and every tensor
    whose gradients are scaled by ten (t mod 10 == 0): 35 of 161 tensors, 43 % of the elements."""
    first = {}
    for t, n in enumerate(wl.numel):
        first.setdefault(n, t)
    return sorted(set(first.values()) | set(range(0, wl.T, 10)))


@pytest.mark.parametrize("which", [0, 1])
def test_config4_resnet18_topk(which):
    """Configuration 4 as configured: 100 iterations at K = 1 % and K = 10 %, the oracle follows
    all 62 tensors, so the message and byte counters are compared as well."""
    wl = W.config(4)[which]
    rep = lockstep(wl, check_every=5, outbox_samples=12)
    _report(wl.name, rep)
    assert rep.steps == wl.steps == 100
    assert rep.params_bit_exact and not rep.near_threshold and rep.sparse_checked > 10


@pytest.mark.parametrize("which", [0, 1])
def test_config5_resnet50_p64(which):
    """Configuration 5 as configured: 50 iterations, dense (carried norm) and K = 1 % (two-pass);
    the library runs all 161 tensors of the 64 replicas, the oracle a 35-tensor sample."""
    wl = W.config(5)[which]
    tensors = _size_classes_and_boosted(wl)
    assert len(tensors) == 35 and wl.numel.index(2048 * 1000) in tensors
    rep = lockstep(wl, tensors=tensors, check_every=5, outbox_samples=12, carry=(which == 0))
    _report(wl.name, rep)
    assert rep.steps == wl.steps == 50
    assert rep.params_bit_exact and not rep.near_threshold
    if which == 1:
        assert rep.sparse_checked > 10


def test_checkpoint_roundtrip_and_reset():
    wl = W.synthetic(3, [5, 1000, 4097], steps=8, lr=0.1, grad_sigma=0.01, history_len=3)
    eg = B.from_workload(wl)
    x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
    g = [eg.to_layout(wl.grads(k, "cuda")) for k in range(wl.steps)]
    for k in range(4):
        eg.step(x, g[k], wl.lr)
    blob, x_mid = eg.export_state(), x.clone()
    for k in range(4, 8):
        eg.step(x, g[k], wl.lr)
    ref_x, ref_stats, ref_dec = x.clone(), eg.stats(), eg.last_decisions()
    eg.reset()
    assert eg.stats() == {"messages": 0, "bytes": 0, "events": 0}
    assert float(eg.mailboxes().abs().max()) == 0.0
    eg.import_state(blob)
    x.copy_(x_mid)
    for k in range(4, 8):
        eg.step(x, g[k], wl.lr)
    assert torch.equal(x, ref_x) and eg.stats() == ref_stats
    for a, b in zip(eg.last_decisions(), ref_dec):
        assert np.array_equal(a, b)
    with pytest.raises(B.EventGradError):
        eg.import_state(blob[:100])
    eg.close()


@pytest.mark.parametrize("numel", [[7, 3000], RAGGED[:-1], [5000]])
@pytest.mark.parametrize("hist,mu", [(1, None), (3, None), (1, 0.9)])
def test_host_buffer_entry_point(numel, hist, mu):
    """eg_step_host (host buffers; tensors pipelined in groups through the device when the
    context allows it) gives the same iteration as eg_step on device buffers, with and without
    momentum (the velocities stay on the device)."""
    wl = W.synthetic(3, numel, steps=6, lr=0.1, grad_sigma=0.01, history_len=hist)
    a, b = B.from_workload(wl), B.from_workload(wl)
    if mu is not None:
        a.set_momentum(mu)
        b.set_momentum(mu)
    x0 = a.to_layout(W.distinct_init_params(wl, "cuda"))
    xa, xb = x0.clone(), x0.cpu().pin_memory()
    for k in range(wl.steps):
        g = a.to_layout(wl.grads(k, "cuda"))
        a.step(xa, g, wl.lr)
        b.step_host(xb, g.cpu().pin_memory(), wl.lr)
        for u, v in zip(a.last_decisions(), b.last_decisions()):
            assert np.array_equal(u, v)
    assert torch.equal(xa.cpu(), xb) and a.stats() == b.stats()
    assert torch.equal(a.mailboxes(), b.mailboxes())
    if mu is not None:
        assert torch.equal(a.velocity(), b.velocity()) and a.velocity().any()
    b.step(xa, g, wl.lr)        # a plain step afterwards covers all tensors again
    a.step(xa.clone(), g, wl.lr)
    assert a.stats() == b.stats()


def test_run_twice_is_deterministic():
    wl = W.synthetic(6, RAGGED, steps=6, lr=0.1, grad_sigma=0.01, topk=(3, 100))
    outs = []
    for _ in range(2):
        eg = B.from_workload(wl)
        x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
        for k in range(wl.steps):
            eg.step(x, eg.to_layout(wl.grads(k, "cuda")), wl.lr)
        outs.append((x.clone(), eg.last_decisions(), eg.stats(), eg.mailboxes()))
        eg.close()
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][3], outs[1][3])
    assert outs[0][2] == outs[1][2]
    assert all(np.array_equal(a, b) for a, b in zip(outs[0][1], outs[1][1]))


def test_steps_replayed_from_a_cuda_graph_match_direct_calls():
    """eg_step only enqueues work and takes no decision on the host, so a captured step can be
    replayed: the trigger state lives on the device and advances with every replay."""
    wl = W.synthetic(4, [5, 1000, 4097, 70000], steps=8, lr=0.1, grad_sigma=0.01)
    g = None
    outs = []
    for use_graph in (False, True):
        eg = B.from_workload(wl)
        eg.set_carry_norm(True)
        x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
        grad = eg.to_layout(wl.grads(0, "cuda"))
        eg.step(x, grad, wl.lr)                       # first step (computes the norms itself)
        if use_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                eg.step(x, grad, wl.lr)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):                 # recorded, not executed
                eg.step(x, grad, wl.lr)
            for _ in range(6):
                g.replay()
        else:
            for _ in range(7):
                eg.step(x, grad, wl.lr)
        torch.cuda.synchronize()
        outs.append((x.clone(), eg.stats(), eg.last_decisions()))
        eg.close()
    assert torch.equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    assert all(np.array_equal(a, b) for a, b in zip(outs[0][2], outs[1][2]))


@pytest.mark.parametrize("what", ["pipelined_carry_cap", "small_cap", "topk_cap", "two_pass", "walking_cap",
                                  "quantised_cap"])
def test_graph_replay_of_every_launch_form_matches_direct_calls_and_the_oracle(what):
    """Replays of one captured eg_step against direct calls and the oracle, for the launch forms a
    step can take: decision + pipelined kernel started as dependent launches (carried norm), the
    single-launch kernel, norm + decision + pipelined kernel, the cooperative Top-K launch, and the
    pipelined kernel walking more tiles than it has CTAs (their order comes from a counter that
    every replay has to find at zero); with a geometric bound on the thresholds, whose sequence
    advances on the device."""
    from oracle import eg_oracle as eo
    topk = (10, 100) if what == "topk_cap" else None
    if what == "walking_cap":       # 6 replicas, 680 tiles of 1024 elements for 444 CTAs
        wl = W.synthetic(6, [5, 4097, 690000], steps=9, lr=0.1, grad_sigma=0.01)
    else:
        wl = W.synthetic(4, [5, 1000, 4097, 70000], steps=9, lr=0.1, grad_sigma=0.01, topk=topk)
    kernel = B.FUSED_AUTO if what == "small_cap" else B.FUSED_PIPELINED
    cap = None if what == "two_pass" else (4e-3, 0.6)
    carry = what != "two_pass"
    outs = []
    for use_graph in (False, True):
        eg = B.from_workload(wl)
        eg.set_carry_norm(carry)
        eg.set_fused_kernel(kernel)
        if cap:
            eg.set_threshold_cap(*cap)
        if what == "quantised_cap":
            eg.set_quantisation(6)
        x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
        grad = eg.to_layout(wl.grads(0, "cuda"))
        eg.step(x, grad, wl.lr)
        if use_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                eg.step(x, grad, wl.lr)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                eg.step(x, grad, wl.lr)
            for _ in range(7):
                g.replay()
        else:
            for _ in range(8):
                eg.step(x, grad, wl.lr)
        torch.cuda.synchronize()
        outs.append((x.clone(), eg.stats(), eg.last_decisions(), eg.mailboxes()))
        eg.close()
    assert torch.equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    assert torch.equal(outs[0][3], outs[1][3])
    assert all(np.array_equal(a, b) for a, b in zip(outs[0][2], outs[1][2]))
    # and the oracle, fed the same gradient nine times
    okw = dict(threshold_cap=cap) if cap else {}
    if what == "quantised_cap":
        okw["quant_bits"] = 6
    o = eo.from_workload(wl, **okw)
    xh = W.distinct_init_params(wl).numpy().copy()
    gh = wl.grads(0).numpy()
    for _ in range(9):
        o.step(xh, gh, wl.lr)
    eg = B.from_workload(wl)
    assert np.array_equal(eg.from_layout(outs[1][0]).cpu().numpy(), xh)
    assert np.array_equal(eg.from_layout(outs[1][3]).numpy().view(np.uint32), o.xhat().view(np.uint32))
    assert outs[1][1] == o.stats()
    assert np.array_equal(outs[1][2][0], o.flags())
    if cap:
        assert 0 < outs[1][1]["events"] < 9 * wl.P * wl.T
    eg.close()


# ---------------------------------------------------------------------------------------
# quantised messages (Section 7: quantization on top of the events; the reading is in the header)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("carry", [False, True])
@pytest.mark.parametrize("bits", [2, 5, 8, 16])
def test_quantised_messages_ragged(bits, carry):
    """Every element of x_hat after a quantised message, the scale exponents, which messages were
    quantised and the byte counter equal the oracle's; ragged sizes over several tiles."""
    wl = W.synthetic(5, RAGGED, steps=10, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=carry, oracle_kw=dict(quant_bits=bits))
    assert rep.params_bit_exact and rep.quantised_checked > 20
    # every tensor sends every step: nothing but quantised messages after the first
    rep = lockstep(wl, init="distinct", carry=carry, steps=5,
                   oracle_kw=dict(quant_bits=bits, mode=1, delta_fixed=0.0))
    assert rep.params_bit_exact and rep.quantised_checked == 4 * wl.P * wl.T


def test_quantised_messages_large_tensor_and_many_replicas():
    wl = W.synthetic(7, [3, (1 << 20) + 1, 4096, 70001], steps=6, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=True, oracle_kw=dict(quant_bits=8))
    assert rep.params_bit_exact and rep.quantised_checked > 10
    wl = W.synthetic(64, [5, 1000, 4097], steps=6, lr=0.1, grad_sigma=0.01)
    rep = lockstep(wl, init="distinct", carry=True, oracle_kw=dict(quant_bits=4))
    assert rep.params_bit_exact and rep.quantised_checked > 100


@pytest.mark.parametrize("what", ["momentum", "hops", "own_last_sent", "change_of_norm", "register", "history_cap",
                                  "delivery"])
def test_quantised_messages_with_every_other_option(what):
    wl = W.synthetic(6, [5, 1000, 4097, 30000], steps=12, lr=0.1, grad_sigma=0.01, history_len=3)
    okw = dict(quant_bits=6)
    kw = dict(init="distinct", carry=what not in ("delivery",))
    if what == "momentum":
        okw["momentum"] = 0.9
    elif what == "hops":
        okw["hops"] = 2
    elif what == "own_last_sent":
        okw["own_last_sent"] = True
    elif what == "change_of_norm":
        okw["change_of_norm"] = True
    elif what == "register":
        kw["fused_kernel"] = B.FUSED_REGISTER
    elif what == "history_cap":
        okw["threshold_cap"] = (4e-3, 0.8)
    elif what == "delivery":
        rng = np.random.default_rng(3)
        kw["deliver_fn"] = lambda k: (rng.random((wl.P, wl.T)) < 0.6).astype(np.uint8)
    rep = lockstep(wl, oracle_kw=okw, **kw)
    assert rep.params_bit_exact and rep.quantised_checked > 10


def test_quantised_messages_small_problem_and_zero_change():
    """A problem small enough for the single-launch kernel takes the other path when messages are
    quantised; a tensor whose change is zero sends codes that are all zero (E = 0)."""
    wl = W.synthetic(4, [7, 300, 2000], steps=6, lr=0.0, grad_sigma=0.0)

    def no_gradient(k, g):
        return torch.zeros_like(g)

    # identical replicas, no gradient, every tensor sends every step: x never moves, the change is zero
    rep = lockstep(wl, oracle_kw=dict(quant_bits=8, mode=1, delta_fixed=0.0), grad_hook=no_gradient,
                   fused_kernel=B.FUSED_AUTO)
    assert rep.params_bit_exact and rep.quantised_checked == 5 * wl.P * wl.T


def test_quantised_message_with_a_change_that_is_not_finite_goes_out_in_full():
    from oracle import eg_oracle as eo
    wl = W.synthetic(3, [10, 5000], steps=3, lr=0.1, grad_sigma=0.01)
    eg = B.from_workload(wl, mode=B.THRESH_FIXED, delta_fixed=0.0)
    eg.set_quantisation(8)
    o = eo.from_workload(wl, mode=eo.FIXED, delta_fixed=0.0, quant_bits=8)
    x = W.distinct_init_params(wl)
    xh = x.numpy().copy()
    xd = eg.to_layout(x.cuda())
    for k in range(3):
        g = wl.grads(k)
        if k == 1:                                  # an infinity in tensor 1 of replica 2
            xh[2, 10 + 4321] = np.inf
            xd[2, eg.tensor_offset[1] + 4321] = float("inf")
        eg.step(xd, eg.to_layout(g.cuda()), wl.lr)
        o.step(xh, g.numpy(), wl.lr)
        q, _ = eg.last_quantised()
        if k == 1:
            assert q[2, 1] == 2 and o.quantised()[2, 1] == 0
            assert np.array_equal((q == 1), (o.quantised() == 1))
        assert eg.stats() == o.stats()
        got = eg.from_layout(eg.mailboxes()).numpy()
        assert np.array_equal(got.view(np.uint32), o.xhat().view(np.uint32))
    eg.close()


@pytest.mark.parametrize("separate", [False, True])
@pytest.mark.parametrize("bits", [3, 8])
def test_quantised_topk_messages(bits, separate, monkeypatch):
    """Both compressions: index sets and the values that arrive (outbox), every element of x_hat,
    exponents and the byte counter against the oracle; cooperative and single-phase launches."""
    if separate:
        monkeypatch.setenv("EG_TOPK_SEPARATE_LAUNCHES", "1")
    wl = W.synthetic(5, RAGGED, steps=10, lr=0.1, grad_sigma=0.01, topk=(5, 100))
    rep = lockstep(wl, init="distinct", carry=True, outbox_samples=64, oracle_kw=dict(quant_bits=bits))
    assert rep.params_bit_exact and rep.sparse_checked > 10 and rep.quantised_checked > 20
    rep = lockstep(wl, init="distinct", steps=5, outbox_samples=10 ** 6,
                   oracle_kw=dict(quant_bits=bits, mode=1, delta_fixed=0.0))
    assert rep.params_bit_exact and rep.quantised_checked == 4 * wl.P * wl.T


def test_quantised_topk_with_delivery_masks_and_momentum():
    wl = W.synthetic(6, RAGGED[:-1], steps=14, lr=0.1, grad_sigma=0.01, topk=(7, 100), history_len=2)
    rep = lockstep(wl, init="distinct", outbox_samples=32, carry=True,
                   oracle_kw=dict(quant_bits=6, momentum=0.9), deliver_fn=_random_links(6, wl.T, 0.5, seed=9))
    assert rep.params_bit_exact and rep.quantised_checked > 10


def test_quantised_messages_through_host_buffers():
    """eg_step_host with quantised messages (whole-step form: the messages need every tensor's
    decision before the averaging kernel) against eg_step on device buffers."""
    wl = W.synthetic(4, [5, 1000, 4097, 30000], steps=6, lr=0.1, grad_sigma=0.01)
    a, b = B.from_workload(wl), B.from_workload(wl)
    a.set_quantisation(8)
    b.set_quantisation(8)
    x = a.to_layout(W.distinct_init_params(wl, "cuda"))
    xh = x.cpu().pin_memory()
    for k in range(wl.steps):
        g = a.to_layout(wl.grads(k, "cuda"))
        a.step(x, g, wl.lr)
        b.step_host(xh, g.cpu().pin_memory(), wl.lr)
    torch.cuda.synchronize()
    assert torch.equal(x.cpu(), xh) and a.stats() == b.stats()
    assert torch.equal(a.mailboxes(), b.mailboxes())
    a.close()
    b.close()


def test_quantisation_refusals_and_checkpoint():
    wl = W.synthetic(3, [7, 3000], steps=3, lr=0.1, grad_sigma=0.01)
    eg = B.from_workload(wl)
    for bad in (1, 17, -3, 33):
        with pytest.raises(B.EventGradError):
            eg.set_quantisation(bad)
    with pytest.raises(B.EventGradError):
        eg.last_quantised()                         # never switched on
    eg.set_quantisation(8)
    eg.set_quantisation(32)                         # off again
    eg.set_quantisation(8)
    x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
    eg.step(x, eg.to_layout(wl.grads(0, "cuda")), wl.lr)
    with pytest.raises(B.EventGradError, match="not allowed"):
        eg.set_quantisation(4)                      # only before the first step
    blob = eg.export_state()
    other = B.from_workload(wl)                     # full precision: another set of rules
    with pytest.raises(B.EventGradError):
        other.import_state(blob)
    other.set_quantisation(8)
    other.import_state(blob)
    y = x.clone()
    g = eg.to_layout(wl.grads(1, "cuda"))
    eg.step(x, g, wl.lr)
    other.step(y, g, wl.lr)
    assert torch.equal(x, y) and eg.stats() == other.stats()
    assert torch.equal(eg.mailboxes(), other.mailboxes())
    for c in (eg, other):
        c.close()


def test_one_stream_at_a_time():
    """A context moves to another stream only once the stream of its previous step has run dry."""
    wl = W.synthetic(3, [7, 3000], steps=3, lr=0.1, grad_sigma=0.01)
    eg, ref = B.from_workload(wl), B.from_workload(wl)
    x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
    y = x.clone()
    g = eg.to_layout(wl.grads(0, "cuda"))
    a, b = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    eg.step(x, g, wl.lr, stream=a)
    with torch.cuda.stream(a):
        torch.cuda._sleep(400_000_000)             # keeps stream a busy for a fraction of a second
    with pytest.raises(B.EventGradError, match="not allowed"):
        eg.step(x, g, wl.lr, stream=b)
    eg.step(x, g, wl.lr, stream=a)                 # the same stream is always fine
    a.synchronize()
    eg.step(x, g, wl.lr, stream=b)
    b.synchronize()
    for _ in range(3):
        ref.step(y, g, wl.lr)
    torch.cuda.synchronize()
    assert torch.equal(x, y) and eg.stats() == ref.stats()
    eg.close(); ref.close()


def test_average_model_and_consensus():
    from oracle import eg_oracle as eo
    wl = W.synthetic(5, [3, 1000, 4097])
    eg = B.from_workload(wl)
    xp = W.distinct_init_params(wl, "cuda")
    x = eg.to_layout(xp)
    avg, cons = eg.average_model(x, consensus=True)
    o = eo.from_workload(wl)
    xn = xp.cpu().numpy()
    assert np.array_equal(eg.from_layout(avg.unsqueeze(0))[0].cpu().numpy(), o.average_model(xn))
    assert cons == pytest.approx(o.consensus_distance(xn), rel=1e-12)


def test_generator_is_device_independent():
    base = W.stream_base(W.MASTER_SEED, W.STREAM_GRAD, 7, 2)
    a = W.ih8_integers(base, 0, 1 << 16, "cpu")
    b = W.ih8_integers(base, 0, 1 << 16, "cuda").cpu()
    assert torch.equal(a, b)
    (wl,) = W.config(1)
    assert torch.equal(wl.grads(3, "cpu"), wl.grads(3, "cuda").cpu())
    assert torch.equal(wl.init_params("cpu"), wl.init_params("cuda").cpu())


def test_bounded_wait_gives_up_and_the_context_survives():
    """Failure detection without a fault: a wait that nothing satisfies runs out after about a
    millisecond, the kernel returns, the error surfaces as a status, and after eg_reset the
    context works as before."""
    wl = W.synthetic(3, [7, 3000], steps=3, lr=0.1, grad_sigma=0.01)
    eg, ref = B.from_workload(wl), B.from_workload(wl)
    assert eg.selftest_wait_timeout() == 0
    with pytest.raises(B.EventGradError, match="timeout"):
        eg.stats()
    eg.reset()
    x = eg.to_layout(W.distinct_init_params(wl, "cuda"))
    y = x.clone()
    for k in range(wl.steps):
        g = eg.to_layout(wl.grads(k, "cuda"))
        eg.step(x, g, wl.lr)
        ref.step(y, g, wl.lr)
    assert torch.equal(x, y) and eg.stats() == ref.stats()


def test_every_allocation_failure_is_reported_and_leaks_nothing():
    """Host-made failure: the n-th device allocation of eg_create fails (test hook, the device
    is not touched).  Every n must give EG_ERR_OOM and a NULL handle, release what was allocated
    before it, and leave the library usable."""
    import ctypes
    lib = B.load_library()
    wl = W.synthetic(4, [5, 1000, 70000], steps=2, topk=(5, 100))
    thr = B.ThresholdParams(0, 1.0, 2, 0.0, 0.0, 1)
    tk = B.TopkParams(1, 5, 100)
    numel = (ctypes.c_int64 * wl.T)(*wl.numel)
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    free0, _ = torch.cuda.mem_get_info()
    n = 1
    while True:
        lib.eg_debug_fail_allocation(n)
        h = ctypes.c_void_p()
        st = lib.eg_create(ctypes.byref(h), 0, wl.P, numel, wl.T, ctypes.byref(thr), ctypes.byref(tk))
        if st == 0:
            break
        assert st == 2 and not h.value, f"allocation {n}: status {st}"
        assert lib.eg_strerror(st) == b"out of memory"
        n += 1
        assert n < 200
    lib.eg_debug_fail_allocation(0)
    assert n > 20                       # a Top-K context makes dozens of allocations
    lib.eg_destroy(h)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 >= free0 - (4 << 20), "memory of the failed creations was not released"
    # the hook is off again: the library works as before
    rep = lockstep(wl, init="distinct", outbox_samples=4)
    assert rep.params_bit_exact
    # later allocations fail the same way: the velocity buffer and the second copy of the mailboxes
    eg = B.from_workload(W.synthetic(3, [100, 5000], steps=2))
    lib.eg_debug_fail_allocation(1)
    with pytest.raises(B.EventGradError):
        eg.set_momentum(0.9)
    lib.eg_debug_fail_allocation(1)
    with pytest.raises(B.EventGradError):
        eg.enable_delivery_masks()
    lib.eg_debug_fail_allocation(0)
    eg.set_momentum(0.9)
    eg.close()


def test_named_ranges_do_not_change_results(monkeypatch):
    """EG_NVTX wraps the kernel groups in named ranges (no-ops without a profiler attached)."""
    monkeypatch.setenv("EG_NVTX", "1")
    wl = W.synthetic(4, RAGGED, steps=6, lr=0.1, grad_sigma=0.01, topk=(5, 100))
    rep = lockstep(wl, init="distinct", carry=True, outbox_samples=8)
    assert rep.params_bit_exact


def test_invalid_arguments_are_reported():
    wl = W.synthetic(2, [8])
    eg = B.from_workload(wl)
    x = eg.empty_params()
    lib = B.load_library()
    assert lib.eg_step(eg._h, None, x.data_ptr(), 0.1, None) == 1
    assert lib.eg_step(eg._h, x.data_ptr() + 4, x.data_ptr(), 0.1, None) == 1   # misaligned
    with pytest.raises(B.EventGradError):
        B.EventGrad(2000, [8])                                                  # P over the limit
