"""Pins for the oracle's dropout layer [Listing 1, case DROPOUT | RELU]: the generator against its published
known-answer vectors, the mask's statistics and its independence of the partitioning, and the layer's forward /
backward arithmetic against float64 autograd and finite differences."""
import os

import numpy as np
import pytest
import torch

import sb_inputs as si
from oracle import splitbrain_oracle as so

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
P25 = 16384      # drop probability 0.25 in units of 1/65536
SEED = 0x5EED0123456789


def net(classes=6, units=P25):
    return [(si.CONV3X3_RELU, 4), (si.MAXPOOL2, 0), (si.CONV3X3_RELU, 6), (si.MAXPOOL2, 0),
            (si.FC_RELU, 24), (si.DROPOUT, units), (si.FC_RELU, 18), (si.DROPOUT, units // 2), (si.FC, classes),
            (si.SOFTMAX_XENT, classes)]


def make(wl, real="double", bf16=False, step=0):
    m = so.from_workload(wl, real=real, bf16=bf16)
    m.load_params(si.make_params(wl, bias_std=0.3))
    m.set_dropout(SEED, step)
    return m


def batch(wl):
    x, y = si.make_batch(wl)
    return si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)


def maxrel(a, b):
    return float(np.max(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64))) / (np.max(np.abs(b)) + 1e-300))


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_known_answers.txt")) if not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = so.philox4x32_10(v[0], v[1], v[2], v[3], v[4], v[5])
        assert [int(o) for o in out] == v[6:]
    # vectorised evaluation equals element-wise evaluation
    c0 = np.arange(5, dtype=np.uint64)
    many = so.philox4x32_10(c0, 7, 8, 9, 10, 11)[0]
    assert [int(so.philox4x32_10(int(c), 7, 8, 9, 10, 11)[0]) for c in c0] == [int(t) for t in many]


def test_keep_mask_is_a_function_of_seed_step_layer_and_logical_element():
    full = so.dropout_keep(SEED, 3, 5, np.arange(64), 37, P25)
    assert full.shape == (64, 37) and full.dtype == bool
    assert np.array_equal(so.dropout_keep(SEED, 3, 5, np.arange(64), 37, P25), full)
    # rows are addressed by their global index: any subset gives the same bits
    assert np.array_equal(so.dropout_keep(SEED, 3, 5, [9, 40, 63], 37, P25), full[[9, 40, 63]])
    # element index e = row*width + column: the flat stream does not depend on how it is cut into rows
    assert np.array_equal(so.dropout_keep(SEED, 3, 5, np.arange(37), 64, P25).reshape(-1), full.reshape(-1))
    for other in (so.dropout_keep(SEED + 1, 3, 5, np.arange(64), 37, P25), so.dropout_keep(SEED + (1 << 32), 3, 5, np.arange(64), 37, P25),
                  so.dropout_keep(SEED, 4, 5, np.arange(64), 37, P25), so.dropout_keep(SEED, 3, 6, np.arange(64), 37, P25)):
        assert 0.25 < np.mean(other != full) < 0.5          # two independent p = 0.25 masks differ in 37.5 % of the bits
    # a larger drop probability only removes elements (one threshold on one uniform word)
    more = so.dropout_keep(SEED, 3, 5, np.arange(64), 37, 2 * P25)
    assert not np.any(more & ~full)
    # element indices beyond 2^32 use the second counter word
    far = so.dropout_keep(SEED, 3, 5, [2 ** 31, 2 ** 31 + 1], 8, P25)
    x0 = so.philox4x32_10((2 ** 31 * 8 + 3) & 0xFFFFFFFF, (2 ** 31 * 8 + 3) >> 32, 5, 3, SEED & 0xFFFFFFFF, SEED >> 32)[0]
    assert bool(far[0, 3]) == (int(x0) >= P25 << 16)


@pytest.mark.parametrize("units", [1024, P25, 32768, 60000])
def test_keep_probability_and_unbiased_scaling(units):
    n_rows, width = 512, 512
    keep = so.dropout_keep(SEED, 0, 1, np.arange(n_rows), width, units)
    p = units / 65536.0
    n = keep.size
    assert abs(keep.mean() - (1 - p)) < 5 * np.sqrt(p * (1 - p) / n)
    scale = so.dropout_scale(units)
    assert scale == np.float32(65536.0) / np.float32(65536 - units) and scale.dtype == np.float32
    assert abs(float(scale) * (1 - p) - 1) < 1e-6
    # expectation preserved: mean of keep * scale is 1 within the same sampling bound
    assert abs(keep.mean() * float(scale) - 1) < 5 * np.sqrt(p / ((1 - p) * n)) + 1e-6
    # rows and columns are kept evenly (no stripe pattern)
    assert abs(keep.mean(0) - (1 - p)).max() < 6 * np.sqrt(p * (1 - p) / n_rows)
    assert abs(keep.mean(1) - (1 - p)).max() < 6 * np.sqrt(p * (1 - p) / width)


def torch_reference(wl, params, x, y, keeps, lr, mu, steps):
    """Unpartitioned network in float64 autograd; keeps[s][li] = the keep mask of dropout layer li in step s."""
    tp = []
    for p in params:
        if p is None:
            tp.append(None)
            continue
        w = torch.tensor(p["w"], dtype=torch.float64)
        if w.dim() == 4:
            w = w.permute(0, 3, 1, 2).contiguous()
        tp.append({"w": w.requires_grad_(True), "b": torch.tensor(p["b"], dtype=torch.float64).requires_grad_(True)})
    leaves = [t for p in tp if p is not None for t in (p["w"], p["b"])]
    opt = torch.optim.SGD(leaves, lr=lr, momentum=mu)
    xt = torch.tensor(x, dtype=torch.float64).permute(0, 3, 1, 2)
    yt = torch.tensor(y).long()
    losses, grads = [], []
    for s in range(steps):
        a, flat = xt, False
        for li, ((kind, out), p) in enumerate(zip(wl.layers, tp)):
            if kind == si.CONV3X3_RELU:
                a = torch.relu(torch.nn.functional.conv2d(a, p["w"], p["b"], padding=1))
            elif kind == si.MAXPOOL2:
                a = torch.nn.functional.max_pool2d(a, 2)
            elif kind in (si.FC_RELU, si.FC):
                if not flat:
                    a, flat = a.permute(0, 2, 3, 1).reshape(a.shape[0], -1), True
                a = torch.nn.functional.linear(a, p["w"], p["b"])
                if kind == si.FC_RELU:
                    a = torch.relu(a)
            elif kind == si.DROPOUT:
                a = a * torch.tensor(keeps[s][li], dtype=torch.float64) / (1.0 - out / 65536.0)
            else:
                loss = torch.nn.functional.cross_entropy(a, yt)
        opt.zero_grad()
        loss.backward()
        grads.append([None if p is None else
                      {"w": (p["w"].grad.permute(0, 2, 3, 1) if p["w"].dim() == 4 else p["w"].grad).numpy().copy(),
                       "b": p["b"].grad.numpy().copy()} for p in tp])
        opt.step()
        losses.append(loss.item())
    final = [None if p is None else
             {"w": (p["w"].detach().permute(0, 2, 3, 1) if p["w"].dim() == 4 else p["w"].detach()).numpy(),
              "b": p["b"].detach().numpy()} for p in tp]
    return losses, grads, final


def test_dropout_step_matches_float64_autograd():
    wl = si.Workload("drop_ag", net(), 8, 8, 3, 3, 2, 3)
    params = si.make_params(wl, bias_std=0.3)
    x, y = si.make_batch(wl)
    widths = {5: 24, 7: 18}
    keeps = [{li: so.dropout_keep(SEED, 11 + s, li, np.arange(wl.B), w, wl.layers[li][1]) for li, w in widths.items()} for s in range(3)]
    losses, grads, final = torch_reference(wl, params, x, y, keeps, 0.05, 0.9, steps=3)
    m = so.from_workload(wl, real="double"); m.load_params(params); m.set_dropout(SEED, 11)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    for s in range(3):
        l = m.forward(xr, yr); m.backward()
        assert m.dropout_step == 12 + s
        for li in widths:
            assert np.array_equal(m.drop_keep[li], keeps[s][li])
        # (float32 scale factor against the exact 1/(1-p) of the reference: 6e-8 relative)
        assert l == pytest.approx(losses[s], rel=1e-6)
        for a, b_ in zip(m.full_grads(), grads[s]):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-6 and maxrel(a["b"], b_["b"]) < 1e-6
        m.sgd_step(0.05, 0.9)
    for a, b_ in zip(m.full_params(), final):
        if a is not None:
            assert maxrel(a["w"], b_["w"]) < 1e-6 and maxrel(a["b"], b_["b"]) < 1e-6
    # dropped elements are exactly zero, kept ones exactly the input times the scale
    below, outp = m.fc_out[4], m.fc_out[5]
    assert np.all(outp[~m.drop_keep[5]] == 0)
    assert np.array_equal(outp[m.drop_keep[5]], (below * np.float64(so.dropout_scale(P25)))[m.drop_keep[5]])


@pytest.mark.parametrize("R,K", [(1, 2), (2, 1), (3, 3), (6, 4)])
def test_dropout_is_partition_invariant(R, K):
    base = si.Workload("drop_inv", net(), 8, 8, 3, 6, 1, 1)
    ref = make(base, step=5)
    wl = base.with_partition(R, K)
    m = make(wl, step=5)
    xs, ys = batch(base)
    xr, yr = batch(wl)
    for step in range(2):
        l0 = ref.step(xs, ys, 0.05, 0.9)
        l1 = m.step(xr, yr, 0.05, 0.9)
        assert l1 == pytest.approx(l0, rel=1e-13)
        for li in (5, 7):
            assert np.array_equal(m.drop_keep[li], ref.drop_keep[li])
        if step == 0:
            assert np.array_equal(m.logits, ref.logits)
        for a, b_ in zip(m.full_grads(), ref.full_grads()):
            if a is not None:
                assert maxrel(a["w"], b_["w"]) < 1e-12 and maxrel(a["b"], b_["b"]) < 1e-12
    assert not np.array_equal(ref.drop_keep[5][:, :18], ref.drop_keep[7])      # layers draw different bits


def test_dropout_finite_differences_with_the_mask_held_fixed():
    wl = si.Workload("drop_fd", net(classes=5), 8, 8, 2, 2, 2, 2)
    params = si.make_params(wl, bias_std=0.3)
    xr, yr = batch(wl)
    m = so.from_workload(wl, real="double"); m.load_params(params); m.set_dropout(SEED, 2)
    m.forward(xr, yr); m.backward()
    g = m.full_grads()
    rng = np.random.default_rng(4)
    h, checked = 1e-6, 0
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
                    mm = so.from_workload(wl, real="double"); mm.load_params(pp); mm.set_dropout(SEED, 2)
                    vals.append(float(mm.forward(xr, yr)))
                fd = (vals[0] - vals[1]) / (2 * h)
                an = float(g[li][key].reshape(-1)[idx])
                if abs(fd - an) > 1e-6 * max(1.0, abs(an)):
                    one_sided = (vals[0] - float(m.loss)) / h
                    other = (float(m.loss) - vals[1]) / h
                    assert abs(one_sided - other) > 1e-4 * max(1.0, abs(an)), (li, key, idx, fd, an)     # a ReLU / max kink
                    continue
                checked += 1
    assert checked > 50


def test_tiny_drop_probability_reduces_to_the_plain_network():
    # p = 1/65536: with this seed no element of the two small layers is dropped, and the scale is 1 + 1.5e-5
    layers = net(units=2)
    wl = si.Workload("drop_tiny", layers, 8, 8, 3, 4, 1, 2)
    plain = si.Workload("plain", [l for l in layers if l[0] != si.DROPOUT], 8, 8, 3, 4, 1, 2)
    params = si.make_params(wl, bias_std=0.3)
    m = so.from_workload(wl, real="double"); m.load_params(params); m.set_dropout(SEED, 0)
    q = so.from_workload(plain, real="double"); q.load_params([p for p, l in zip(params, layers) if l[0] != si.DROPOUT])
    xr, yr = batch(wl)
    l1 = m.forward(xr, yr); m.backward()
    l0 = q.forward(xr, yr); q.backward()
    assert m.drop_keep[5].all() and m.drop_keep[7].all()
    assert l1 == pytest.approx(l0, rel=1e-3)
    g1 = [g for g in m.full_grads() if g is not None]
    g0 = [g for g in q.full_grads() if g is not None]
    for a, b_ in zip(g1, g0):
        assert maxrel(a["w"], b_["w"]) < 1e-3


def test_bf16_mode_rounds_the_stored_dropout_tensors():
    wl = si.Workload("drop_bf16", net(), 8, 8, 3, 4, 2, 2)
    m = make(wl, real="float", bf16=True, step=1)
    xr, yr = batch(wl)
    m.forward(xr, yr); m.backward()
    for li in (5, 7):
        assert np.array_equal(so.round_bf16(m.fc_out[li]), m.fc_out[li])
        assert np.array_equal(so.round_bf16(m.d_pre[li]), m.d_pre[li])
        exact = np.where(m.drop_keep[li], m.fc_out[li - 1] * so.dropout_scale(wl.layers[li][1]), np.float32(0))
        assert np.array_equal(m.fc_out[li], so.round_bf16(exact)) and not np.array_equal(m.fc_out[li], exact)


def test_modulo_schedule_draws_the_same_masks_for_the_same_examples():
    """The sub-iteration schedule sends every example through the FC stack exactly once per iteration: with the learning
    rate at zero its FC gradients add up to the synchronous step's, its input gradients are the same, and so are the conv
    gradients -- provided each example meets the same dropout mask in both schedules."""
    wl = si.Workload("drop_mod", net(), 8, 8, 3, 4, 2, 2)
    xr, yr = batch(wl)
    a = make(wl, step=9); b_ = make(wl, step=9)
    la = a.forward(xr, yr); a.backward()
    lb = b_.step_modulo(xr, yr, 0.0, 0.9)
    assert lb == pytest.approx(la, rel=1e-13)
    assert a.dropout_step == b_.dropout_step == 10
    ga = a.full_grads()
    for li in range(len(wl.layers)):
        if ga[li] is None:
            continue
        if li < a.first_fc:
            assert maxrel(b_.grads[li]["w"], ga[li]["w"]) < 1e-12
        else:
            tot = sum(np.concatenate([s_["w"] for s_ in gk[li]], 0) for gk in b_.mod_fc_grads)
            assert maxrel(tot, ga[li]["w"]) < 1e-12
    # K = 1: one sub-iteration, the same iteration as step()
    wl1 = wl.with_partition(4, 1)
    x1, y1 = batch(wl1)
    c = make(wl1, step=3); d = make(wl1, step=3)
    assert c.step(x1, y1, 0.05, 0.9) == d.step_modulo(x1, y1, 0.05, 0.9)
    for p_, q_ in zip(c.full_params(), d.full_params()):
        if p_ is not None:
            assert np.array_equal(p_["w"], q_["w"])
