"""Pins for the oracle's partitioned training step: the paper's equivalence claim (R/K invariance),
its worked modulo-layer example and Table 1, finite differences in double, and an independent
float64 autograd computation of the unpartitioned network with library routines."""
import os

import numpy as np
import pytest
import torch

import sb_inputs as si
from oracle import splitbrain_oracle as so

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_net(classes=6):
    # conv-conv-pool-conv-pool-fc-fc-fc: has conv->conv, pool->conv, conv->pool->fc transitions
    return [(si.CONV3X3_RELU, 4), (si.CONV3X3_RELU, 5), (si.MAXPOOL2, 0), (si.CONV3X3_RELU, 6), (si.MAXPOOL2, 0),
            (si.FC_RELU, 12), (si.FC_RELU, 9), (si.FC, classes), (si.SOFTMAX_XENT, classes)]


def make(wl, real="double", bf16=False, bias_std=0.3):
    m = so.from_workload(wl, real=real, bf16=bf16)
    m.load_params(si.make_params(wl, bias_std=bias_std))
    return m


def batch(wl):
    x, y = si.make_batch(wl)
    return si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)


def maxrel(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64))) / (np.max(np.abs(b)) + 1e-300))


# ---- the paper's own statements ------------------------------------------------------------------
def test_modulo_layer_worked_example_owner_map():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "modulo_layer_example.txt")) if not l.startswith("#")]
    for B, K, ex, owner in [[int(v) for v in r] for r in rows]:
        size = B // K
        # oracle's gather: row g comes from replica g // b with b = B/K rows per worker
        wl = si.Workload("t", [(si.CONV3X3_RELU, 2), (si.FC, 3), (si.SOFTMAX_XENT, 3)], 2, 2, 1, size, K, K)
        m = make(wl)
        xs = [np.full((size, 2, 2, 1), float(r + 1)) for r in range(K)]
        for li in (0,):
            m.params[li]["w"][:] = 0; m.params[li]["w"][:, 1, 1, 0] = 1; m.params[li]["b"][:] = 0
        m.forward(xs, [np.zeros(size, np.int32)] * K)
        assert np.all(m.fc_in[1][ex] == owner + 1)        # example ex carries its owner's data


def test_table1_parameter_counts():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_vgg_variant_params.txt")) if not l.startswith("#")]
    table = {r[0]: r[1:] for r in rows}
    wl = si.Workload("paper_vgg", si.paper_vgg_variant_layers(), 32, 32, 3, 1, 1, 1)
    m = so.from_workload(wl); m.load_params(si.make_params(wl))
    trainable = [p for p in m.full_params() if p is not None]
    names = ["Conv%d" % i for i in range(7)] + ["FC%d" % i for i in range(3)]
    for name, p in zip(names, trainable):
        assert p["w"].size == int(table[name][2]), name
    conv = sum(p["w"].size + p["b"].size for p in trainable[:7])
    fc = sum(p["w"].size + p["b"].size for p in trainable[7:])
    # the printed shares are reproduced by the bias-inclusive counts
    assert round(100.0 * conv / (conv + fc), 2) == float(table["share_conv_percent"][0])
    assert round(100.0 * fc / (conv + fc), 2) == float(table["share_fc_percent"][0])


@pytest.mark.parametrize("out,K", [(4096, 4), (10, 4), (10, 8), (1000, 4), (64, 2), (7, 7)])
def test_shard_sizes_are_one_over_K(out, K):
    cb = so.shard_bounds(out, K)
    assert cb[0] == 0 and cb[-1] == out and len(cb) == K + 1
    sizes = np.diff(cb)
    assert sizes.sum() == out and sizes.min() >= out // K and sizes.max() <= -(-out // K)
    assert cb == si.shard_bounds(out, K)


# ---- partition invariance (the paper: same output error as the complete local model) ---------------
@pytest.mark.parametrize("R,K", [(1, 2), (2, 1), (2, 2), (4, 3), (8, 4), (4, 8)])
def test_RK_invariance_double(R, K):
    base = si.Workload("inv", small_net(), 8, 8, 3, 8, 1, 1)
    ref = make(base)
    wl = base.with_partition(R, K)
    m = make(wl)
    xs, ys = batch(base)
    xr, yr = batch(wl)
    for step in range(2):                                   # two steps so momentum matters
        l0 = ref.step(xs, ys, 0.05, 0.9)
        l1 = m.step(xr, yr, 0.05, 0.9)
        assert l1 == pytest.approx(l0, rel=1e-13)
        # forward activations are bit-identical: no forward sum is re-ordered by the partitioning
        # (first step only: afterwards the weights themselves differ by summation-order noise)
        if step == 0:
            assert np.array_equal(m.logits, ref.logits)
            assert np.array_equal(np.concatenate([m.conv_out[r][4] for r in range(R)]), ref.conv_out[0][4])
        for a, b_ in zip(m.full_grads(), ref.full_grads()):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-12 and maxrel(a["b"], b_["b"]) < 1e-12
        for a, b_ in zip(m.full_params(), ref.full_params()):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-13 and maxrel(a["b"], b_["b"]) < 1e-13
        for a, b_ in zip(m.full_mom(), ref.full_mom()):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-12


def test_RK_invariance_float_cfg0():
    base = si.config(0).with_partition(1, 1)
    ref = make(base, real="float", bias_std=0.0)
    xs, ys = batch(base)
    ref.step(xs, ys, 0.01, 0.9)
    for R, K in [(2, 2), (4, 2), (8, 5)]:
        wl = base.with_partition(R, K)
        m = make(wl, real="float", bias_std=0.0)
        xr, yr = batch(wl)
        m.step(xr, yr, 0.01, 0.9)
        assert np.array_equal(m.logits, ref.logits)
        assert abs(float(m.loss) - float(ref.loss)) < 1e-6
        for a, b_ in zip(m.full_grads(), ref.full_grads()):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-5 and maxrel(a["b"], b_["b"]) < 1e-5
        for a, b_ in zip(m.full_params(), ref.full_params()):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-6


# ---- independent second opinion: float64 autograd with library routines ---------------------------
def torch_reference(wl, params, x, y, lr, mu, steps):
    """Unpartitioned network with torch.nn.functional in float64; returns per-step losses, first-step
    grads, final weights."""
    tp = []
    for p in params:
        if p is None:
            tp.append(None)
        else:
            w = torch.tensor(p["w"], dtype=torch.float64)
            if w.dim() == 4:
                w = w.permute(0, 3, 1, 2).contiguous()       # [Cout,3,3,Cin] -> [Cout,Cin,3,3]
            tp.append({"w": w.requires_grad_(True), "b": torch.tensor(p["b"], dtype=torch.float64).requires_grad_(True)})
    leaves = [t for p in tp if p is not None for t in (p["w"], p["b"])]
    opt = torch.optim.SGD(leaves, lr=lr, momentum=mu)
    xt = torch.tensor(x, dtype=torch.float64).permute(0, 3, 1, 2)
    yt = torch.tensor(y).long()
    losses, grads1 = [], None
    for s in range(steps):
        a = xt
        flat = False
        for (kind, _), p in zip(wl.layers, tp):
            if kind == si.CONV3X3_RELU:
                a = torch.relu(torch.nn.functional.conv2d(a, p["w"], p["b"], padding=1))
            elif kind == si.MAXPOOL2:
                a = torch.nn.functional.max_pool2d(a, 2)
            elif kind in (si.FC_RELU, si.FC):
                if not flat:
                    a = a.permute(0, 2, 3, 1).reshape(a.shape[0], -1)      # (h, w, c) flatten order
                    flat = True
                a = torch.nn.functional.linear(a, p["w"], p["b"])
                if kind == si.FC_RELU:
                    a = torch.relu(a)
            else:
                loss = torch.nn.functional.cross_entropy(a, yt)
        opt.zero_grad()
        loss.backward()
        if s == 0:
            grads1 = [None if p is None else
                      {"w": (p["w"].grad.permute(0, 2, 3, 1) if p["w"].dim() == 4 else p["w"].grad).numpy().copy(),
                       "b": p["b"].grad.numpy().copy()} for p in tp]
        opt.step()
        losses.append(loss.item())
    final = [None if p is None else
             {"w": (p["w"].detach().permute(0, 2, 3, 1) if p["w"].dim() == 4 else p["w"].detach()).numpy(),
              "b": p["b"].detach().numpy()} for p in tp]
    return losses, grads1, final


def test_partitioned_step_matches_float64_autograd():
    wl = si.Workload("ag", small_net(), 8, 8, 3, 3, 2, 3)
    params = si.make_params(wl, bias_std=0.3)
    x, y = si.make_batch(wl)
    losses, g1, final = torch_reference(wl, params, x, y, 0.05, 0.9, steps=3)
    m = so.from_workload(wl, real="double"); m.load_params(params)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    for s in range(3):
        l = m.forward(xr, yr); m.backward()
        assert l == pytest.approx(losses[s], rel=1e-12)
        if s == 0:
            for a, b_ in zip(m.full_grads(), g1):
                if a is not None:
                    assert maxrel(a["w"], b_["w"]) < 1e-11 and maxrel(a["b"], b_["b"]) < 1e-11
        m.sgd_step(0.05, 0.9)
    for a, b_ in zip(m.full_params(), final):
        if a is not None:
            assert maxrel(a["w"], b_["w"]) < 1e-12 and maxrel(a["b"], b_["b"]) < 1e-12


# ---- finite differences -----------------------------------------------------------------------------
def test_finite_difference_gradients_double():
    wl = si.Workload("fd", small_net(classes=5), 8, 8, 2, 2, 2, 2)
    params = si.make_params(wl, bias_std=0.3)
    x, y = si.make_batch(wl)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    m = so.from_workload(wl, real="double"); m.load_params(params)
    m.forward(xr, yr); m.backward()
    g = m.full_grads()
    rng = np.random.default_rng(3)
    h = 1e-6
    checked = 0
    for li, p in enumerate(params):
        if p is None:
            continue
        for key in ("w", "b"):
            flat = p[key].reshape(-1)
            for idx in rng.choice(flat.size, size=min(6, flat.size), replace=False):
                vals = []
                for sgn in (+1, -1):
                    pp = [None if q is None else {"w": q["w"].astype(np.float64).copy(), "b": q["b"].astype(np.float64).copy()} for q in params]
                    pp[li][key].reshape(-1)[idx] += sgn * h
                    mm = so.from_workload(wl, real="double"); mm.load_params(pp)
                    vals.append(float(mm.forward(xr, yr)))
                fd = (vals[0] - vals[1]) / (2 * h)
                an = float(g[li][key].reshape(-1)[idx])
                # skip coordinates sitting on a ReLU/max kink (the two one-sided slopes differ)
                if abs(fd - an) > 1e-6 * max(1.0, abs(an)):
                    mm0 = float(m.loss)
                    one_sided = (vals[0] - mm0) / h
                    other = (mm0 - vals[1]) / h
                    assert abs(one_sided - other) > 1e-4 * max(1.0, abs(an)), (li, key, idx, fd, an)
                    continue
                checked += 1
    assert checked > 60


def test_zero_last_layer_gives_log_C():
    wl = si.config(0)
    params = si.make_params(wl)
    params[5]["w"][:] = 0
    m = so.from_workload(wl, real="float"); m.load_params(params)
    xr, yr = batch(wl)
    assert float(m.forward(xr, yr)) == pytest.approx(np.log(10.0), rel=1e-6)


def test_he_init_variance_and_fc_sweep_inputs():
    wl = si.config(1).with_batch(1)
    for s, p in zip(si.layer_shapes(wl), si.make_params(wl)):
        if p is None or p["w"].size < 20000:
            continue
        fan_in = 9 * s["Cin"] if s["kind"] == si.CONV3X3_RELU else s["in"]
        assert float(p["w"].var()) == pytest.approx(2.0 / fan_in, rel=0.05)
        assert not p["b"].any()
    assert si.param_count(wl) == (14710464, 4224, 18915328, 8202)


def test_bf16_mode_stays_close_to_fp32_mode():
    """The mixed-precision contract only rounds operands.  Forward tensors stay within the 1e-2
    max-normalised band of the fp32 oracle; in the backward pass a rounded activation can flip a
    ReLU mask or a pooling argmax, which moves single gradient elements by their full size (a fraction f
    of flipped routes costs about sqrt(2f) in the Frobenius norm: 0.3 % flips -> 8 %), so gradients
    only get a loose Frobenius bound here."""
    wl = si.config(0)
    xr, yr = batch(wl)
    a = make(wl, real="float", bias_std=0.0); b_ = make(wl, real="float", bf16=True, bias_std=0.0)
    la, lb = a.step(xr, yr, 0.01, 0.9), b_.step(xr, yr, 0.01, 0.9)
    assert abs(float(la) - float(lb)) < 5e-3
    assert maxrel(b_.logits, a.logits) < 1e-2
    for r in range(wl.R):
        for li in range(4):
            assert maxrel(b_.conv_out[r][li], a.conv_out[r][li]) < 1e-2
    for ga, gb in zip(a.full_grads(), b_.full_grads()):
        if ga is not None:
            assert np.linalg.norm(gb["w"] - ga["w"]) / np.linalg.norm(ga["w"]) < 0.2


def test_sampled_rows_of_a_large_batch_are_independent():
    """A sub-batch run with loss_B = size of the full batch reproduces the full batch's activations and
    activation gradients for those rows (pins the sampled-image parity tests used at full sizes)."""
    full = si.Workload("full", small_net(), 8, 8, 3, 6, 1, 2)
    params = si.make_params(full, bias_std=0.3)
    x, y = si.make_batch(full)
    mf = so.from_workload(full, real="double"); mf.load_params(params)
    mf.forward([x], [y]); mf.backward()
    pick = [1, 4]
    sub = si.Workload("sub", small_net(), 8, 8, 3, len(pick), 1, 2)
    ms = so.from_workload(sub, real="double", loss_B=full.B); ms.load_params(params)
    ms.forward([x[pick]], [y[pick]]); ms.backward()
    assert np.array_equal(ms.logits, mf.logits[pick])
    np.testing.assert_allclose(ms.row_loss, mf.row_loss[pick], rtol=1e-14)
    for li in range(5):
        assert np.array_equal(ms.conv_out[0][li], mf.conv_out[0][li][pick])
        np.testing.assert_allclose(ms.d_conv[0][li], mf.d_conv[0][li][pick], rtol=1e-13, atol=1e-18)
