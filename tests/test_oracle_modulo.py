"""Pins for the oracle's modulo-layer schedule (K sub-iterations of the FC stack per iteration): the paper's worked
example, the K = 1 and lr = 0 special cases, and a re-composition out of the (separately pinned) synchronous
forward()/backward() on the sub-batches."""
import os

import numpy as np
import pytest

import sb_inputs as si
from oracle import splitbrain_oracle as so
from test_oracle_model import batch, make, maxrel, small_net

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def wl_of(b, R, K, classes=6):
    return si.Workload("modulo", small_net(classes), 8, 8, 3, b, R, K)


def test_sub_iteration_rows_match_the_papers_worked_example():
    rows = [[int(v) for v in l.split()] for l in open(os.path.join(GOLDEN, "modulo_schedule_example.txt")) if not l.startswith("#")]
    m = so.from_workload(wl_of(2, 2, 2))          # K = 2 workers, local batch 2: size = B/K = 1
    for k, pos, worker, local in rows:
        g = m.modulo_rows(k)[pos]
        assert g // m.b == worker and g % m.b == local
    # in general: every row is visited exactly once per iteration, b/K rows of every replica per sub-iteration
    m = so.from_workload(wl_of(6, 4, 3))
    seen = np.concatenate([m.modulo_rows(k) for k in range(3)])
    assert sorted(seen.tolist()) == list(range(24))
    for k in range(3):
        r = m.modulo_rows(k)
        assert len(r) == 4 * 2 and all(np.sum(r // 6 == rep) == 2 for rep in range(4))
        assert np.array_equal(r // 6, np.repeat(np.arange(4), 2))      # position p belongs to replica p // (b/K)


@pytest.mark.parametrize("real", ["double", "float"])
def test_K1_is_the_synchronous_step(real):
    wl = wl_of(4, 2, 1)
    xs, ys = batch(wl)
    a, b_ = make(wl, real), make(wl, real)
    for _ in range(2):
        la = a.step(xs, ys, 0.05, 0.9)
        lb = b_.step_modulo(xs, ys, 0.05, 0.9)
        assert la == lb
    for pa, pb in zip(a.full_params(), b_.full_params()):
        if pa is not None:
            assert np.array_equal(pa["w"], pb["w"]) and np.array_equal(pa["b"], pb["b"])
    for pa, pb in zip(a.full_mom(), b_.full_mom()):
        if pa is not None:
            assert np.array_equal(pa["w"], pb["w"]) and np.array_equal(pa["b"], pb["b"])


def test_zero_learning_rate_gradients_add_up_to_the_synchronous_ones():
    """With lr = 0 no FC weight moves between the sub-iterations, so the K sub-iteration FC gradients (each already
    divided by K through the 1/B normalisation) sum to the synchronous FC gradient, and the conv gradients and the
    loss are the synchronous ones."""
    wl = wl_of(4, 2, 2)
    xs, ys = batch(wl)
    a, m = make(wl), make(wl)
    la = a.forward(xs, ys); a.backward()
    lm = m.step_modulo(xs, ys, 0.0, 0.0)
    assert abs(la - lm) <= 1e-13 * abs(la)
    ga = a.full_grads()
    for li, (kind, _) in enumerate(wl.layers):
        if kind == si.CONV3X3_RELU:
            assert maxrel(m.grads[li]["w"], ga[li]["w"]) <= 1e-12 and maxrel(m.grads[li]["b"], ga[li]["b"]) <= 1e-12
        elif kind in (si.FC_RELU, si.FC):
            w = sum(np.concatenate([s["w"] for s in gk[li]], 0) for gk in m.mod_fc_grads)
            b_ = sum(np.concatenate([s["b"] for s in gk[li]], 0) for gk in m.mod_fc_grads)
            assert maxrel(w, ga[li]["w"]) <= 1e-12 and maxrel(b_, ga[li]["b"]) <= 1e-12
    # the compensation: one sub-iteration's FC gradient is (mean over its sub-batch) / K
    sub = si.Workload("sub", wl.layers, wl.H, wl.W, wl.C, wl.b // wl.K, wl.R, wl.K)
    s = make(sub)
    rows = m.modulo_rows(0)
    xa, ya = np.concatenate(xs, 0), np.concatenate(ys, 0)
    s.forward(si.split_replicas(xa[rows], wl.R), si.split_replicas(ya[rows], wl.R)); s.backward()   # loss = mean over the sub-batch
    li = max(i for i, (k, _) in enumerate(wl.layers) if k == si.FC)
    w0 = np.concatenate([sh["w"] for sh in m.mod_fc_grads[0][li]], 0)
    assert maxrel(w0, s.full_grads()[li]["w"] / wl.K) <= 1e-12


@pytest.mark.parametrize("R,K,b", [(2, 2, 4), (3, 2, 2), (1, 4, 4)])
def test_recomposition_from_synchronous_passes_on_the_sub_batches(R, K, b):
    """Sub-iteration k is a synchronous forward/backward on the rows S_k with the loss normalised by the full batch
    B, followed by an update of the FC parameters only; the conv gradient of the iteration is the sum over k.
    forward()/backward() are pinned on their own (finite differences, float64 autograd), so this pins step_modulo."""
    wl = wl_of(b, R, K)
    xs, ys = batch(wl)
    xa, ya = np.concatenate(xs, 0), np.concatenate(ys, 0)
    lr, mu = 0.05, 0.9
    m = make(wl)
    ref = make(wl)                                    # holds the reference parameters / momentum
    sub = si.Workload("sub", wl.layers, wl.H, wl.W, wl.C, b // K, R, K)
    for step in range(2):
        conv_g = None
        row_losses = np.zeros(wl.B)
        for k in range(K):
            rows = m.modulo_rows(k)
            s = so.from_workload(sub, real="double", loss_B=wl.B)
            s.params, s.mom, s.bounds = ref.params, ref.mom, ref.bounds      # shared storage: updates land in `ref`
            s.forward(si.split_replicas(xa[rows], R), si.split_replicas(ya[rows], R))
            s.backward()
            row_losses[rows] = s.row_loss
            cg = {li: {"w": s.grads[li]["w"].copy(), "b": s.grads[li]["b"].copy()} for li, (kd, _) in enumerate(wl.layers) if kd == si.CONV3X3_RELU}
            conv_g = cg if conv_g is None else {li: {key: conv_g[li][key] + cg[li][key] for key in ("w", "b")} for li in cg}
            for li, (kd, _) in enumerate(wl.layers):                          # FC update only
                if kd in (si.FC_RELU, si.FC):
                    for j in range(K):
                        for key in ("w", "b"):
                            s.P.sgd(ref.params[li][j][key], ref.mom[li][j][key], s.grads[li][j][key], lr, mu)
        for li, g in conv_g.items():                                           # conv update once
            for key in ("w", "b"):
                ref.P.sgd(ref.params[li][key], ref.mom[li][key], g[key], lr, mu)
        loss = m.step_modulo(xs, ys, lr, mu)
        assert abs(loss - row_losses.mean()) <= 1e-12 * abs(loss)
        for pa, pb in zip(m.full_params(), ref.full_params()):
            if pa is not None:
                assert maxrel(pa["w"], pb["w"]) <= 1e-12 and maxrel(pa["b"], pb["b"]) <= 1e-12, step
        for pa, pb in zip(m.full_mom(), ref.full_mom()):
            if pa is not None:
                assert maxrel(pa["w"], pb["w"]) <= 1e-11 and maxrel(pa["b"], pb["b"]) <= 1e-11, step


def test_modulo_schedule_differs_from_the_synchronous_step_for_K_above_one():
    """The paper's schedule is a different algorithm: with K = 2 the FC weights of the second sub-iteration have
    already moved, so the result is not the synchronous step's."""
    wl = wl_of(4, 2, 2)
    xs, ys = batch(wl)
    a, m = make(wl), make(wl)
    a.step(xs, ys, 0.05, 0.9); m.step_modulo(xs, ys, 0.05, 0.9)
    li = max(i for i, (k, _) in enumerate(wl.layers) if k == si.FC)
    assert maxrel(m.full_params()[li]["w"], a.full_params()[li]["w"]) > 1e-6
