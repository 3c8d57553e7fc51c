"""Pins of the oracle's bf16 mode: WHERE it rounds.

The mixed-precision contract: a tensor is rounded to bfloat16 (nearest, ties to even) exactly where it is stored as
an operand of a later contraction -- input images, every stored activation (conv + ReLU outputs, pooled maps, FC + ReLU
outputs), every stored activation gradient (the loss gradient dZ included) and the weight copy a contraction reads.
Nothing else is rounded: accumulators, bias add, ReLU, logits, loss, weight and bias gradients, master weights, momentum.

Three independent checks, none of which uses the oracle's own rounding helper (torch's bfloat16 cast is the yardstick):

 1. representability: tensors at a rounding point hold only bfloat16 values, tensors that must stay in float do not;
 2. replay: the unpartitioned network written out here, primitive by primitive, with the roundings placed by this
    file according to the sentence above, gives bit-identical tensors; the partitioned oracle agrees with it;
 3. sensitivity: switching off any single rounding call of the oracle (one at a time) makes check 2 fail, so no
    rounding point is outside the reach of the replay, and adding one where none belongs fails check 1 or 2.
"""
import numpy as np
import pytest
import torch

import sb_inputs as si
from oracle import splitbrain_oracle as so


def to_bf16(a):
    """bfloat16 rounding by torch (independent of the oracle's integer implementation)."""
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(torch.bfloat16).to(torch.float32).numpy()


def is_bf16(a):
    return np.array_equal(to_bf16(a), np.asarray(a, np.float32))


def frac_not_bf16(a):
    """Fraction of the non-zero values that are not bfloat16 numbers (zeros, e.g. of dead ReLU units, are exact in both)."""
    a = np.asarray(a, np.float32).ravel()
    a = a[a != 0]
    return float(np.mean(to_bf16(a) != a))


def three_conv_net():
    return [(si.CONV3X3_RELU, 8), (si.CONV3X3_RELU, 16), (si.MAXPOOL2, 0), (si.CONV3X3_RELU, 8), (si.MAXPOOL2, 0),
            (si.FC_RELU, 24), (si.FC_RELU, 12), (si.FC, 5), (si.SOFTMAX_XENT, 5)]


WORKLOADS = {
    "cfg0": lambda R, K: si.config(0).with_partition(R, K),
    "three_conv": lambda R, K: si.Workload("three_conv", three_conv_net(), 8, 12, 3, 6 // R, R, K),
}


def run_oracle(wl, bf16=True, steps=1):
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    m = so.from_workload(wl, real="float", bf16=bf16)
    m.load_params(params)
    for _ in range(steps):
        m.forward(si.split_replicas(x, wl.R), si.split_replicas(y, wl.R))
        m.backward()
        m.sgd_step(0.05, 0.9)
    return m, params, x, y


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_rounded_tensors_are_bf16_and_unrounded_ones_are_not(name):
    wl = WORKLOADS[name](2, 2)
    m, _, _, _ = run_oracle(wl)
    first_fc = m.first_fc
    for r in range(wl.R):
        assert is_bf16(m.x_in[r])
        for li in range(first_fc):
            assert is_bf16(m.conv_out[r][li]), ("stored activation", li)
            assert is_bf16(m.d_conv[r][li]), ("stored activation gradient", li)
    for li in range(first_fc, len(wl.layers) - 1):
        kind = wl.layers[li][0]
        assert is_bf16(m.d_pre[li]), ("stored FC activation gradient", li)
        if kind == si.FC_RELU:
            assert is_bf16(m.fc_out[li]), ("stored FC activation", li)
    # what must stay in float: most values of these tensors are not bfloat16 numbers
    assert frac_not_bf16(m.logits) > 0.8
    assert frac_not_bf16(m.row_loss) > 0.8
    assert frac_not_bf16(m.dZ) > 0.8                       # the loss gradient before it is stored
    for li in range(first_fc, len(wl.layers) - 1):
        assert frac_not_bf16(m.d_fc_in[li]) > 0.8          # shard sum of input gradients, before mask and store
    for g, p, v in zip(m.full_grads(), m.full_params(), m.full_mom()):
        if g is not None:
            # (a gradient is a sum of a few products of bf16 numbers, so some of its values happen to be short; a
            # rounded tensor would have none that are not)
            for t in (g["w"], g["b"], p["w"], v["w"]):
                assert frac_not_bf16(t) > 0.5


def replay_unpartitioned(wl, params, x, y):
    """The network with R = K = 1, one primitive call per line of the method, roundings placed here."""
    P = so.Prims("float")
    q = to_bf16
    nl = len(wl.layers)
    act = [None] * nl           # stored output of every layer
    idx = [None] * nl
    a = q(x)                    # input images
    x_in = a
    feat_shape = None
    for li, (kind, out) in enumerate(wl.layers):
        if kind == si.CONV3X3_RELU:
            a = q(P.conv_fwd(a, q(params[li]["w"]), params[li]["b"], relu=True))      # weight copy rounded, bias not
        elif kind == si.MAXPOOL2:
            a, idx[li] = P.pool_fwd(a)                                                # maxima of bf16 values are bf16
        elif kind in (si.FC_RELU, si.FC):
            if a.ndim == 4:
                feat_shape = a.shape
                a = a.reshape(a.shape[0], -1)
            a = P.fc_fwd(a, q(params[li]["w"]), params[li]["b"], relu=(kind == si.FC_RELU))
            if kind == si.FC_RELU:
                a = q(a)                                                              # logits stay in float
        else:
            row_loss, dZ = P.softmax_xent(a, y, 1.0 / wl.B)
            break
        act[li] = a
    grads = [None] * nl
    d_store = [None] * nl       # the stored gradient w.r.t. each layer's (pre-activation) output
    d = q(dZ)
    for li in range(nl - 2, -1, -1):
        kind = wl.layers[li][0]
        below = act[li - 1] if li > 0 else x_in
        if kind in (si.FC_RELU, si.FC):
            d_store[li] = d
            xin = below.reshape(below.shape[0], -1)
            dW, db, dX = P.fc_bwd(xin, q(params[li]["w"]), d)
            grads[li] = {"w": dW, "b": db}
            if li > 0 and wl.layers[li - 1][0] == si.FC_RELU:
                d = q(dX * (act[li - 1] > 0))
            else:
                d = dX.reshape(feat_shape)                                             # into the conv side: stored by the layer below
        elif kind == si.MAXPOOL2:
            d = q(d)
            d_store[li] = d
            d = P.pool_bwd(d, idx[li])
        else:
            d = q(d * (act[li] > 0))
            d_store[li] = d
            dw, db = P.conv_wgrad(below, d)
            grads[li] = {"w": dw, "b": db}
            if li > 0:
                d = P.conv_dgrad(d, q(params[li]["w"]))
    return dict(x_in=x_in, act=act, idx=idx, row_loss=row_loss, dZ=dZ, grads=grads, d_store=d_store)


def compare_with_replay(m, rp, wl, exact_grads):
    """Oracle model m (any partition of wl's batch) against the replay; returns a list of mismatches."""
    bad = []
    b = wl.b
    first_fc = m.first_fc

    def same(a, ref, what):
        if not np.array_equal(np.asarray(a).reshape(np.asarray(ref).shape), ref):
            bad.append(what)

    for r in range(wl.R):
        rows = slice(r * b, (r + 1) * b)
        same(m.x_in[r], rp["x_in"][rows], ("x_in", r))
        for li in range(first_fc):
            same(m.conv_out[r][li], rp["act"][li][rows], ("act", li, r))
            if exact_grads:
                same(m.d_conv[r][li], rp["d_store"][li][rows], ("dact", li, r))
            else:
                # (the shard sum adds in another order before the gradient is stored: one bf16 unit at most)
                ref = rp["d_store"][li][rows]
                if np.max(np.abs(m.d_conv[r][li] - ref)) > 2.0 ** -7 * np.max(np.abs(ref)):
                    bad.append(("dact", li, r))
            if wl.layers[li][0] == si.MAXPOOL2:
                same(m.pool_idx[r][li], rp["idx"][li][rows], ("idx", li, r))
    for li in range(first_fc, len(wl.layers) - 1):
        same(m.fc_out[li], rp["act"][li], ("fc act", li))
        if li == len(wl.layers) - 2 or exact_grads:
            same(m.d_pre[li], rp["d_store"][li], ("fc dact", li))
    same(m.row_loss, rp["row_loss"], ("row loss",))
    same(m.dZ, rp["dZ"], ("dZ",))
    for li, g in enumerate(m.full_grads()):
        if g is None:
            continue
        for k in ("w", "b"):
            if exact_grads:
                same(g[k], rp["grads"][li][k], ("grad", li, k))
            else:
                err = np.max(np.abs(g[k] - rp["grads"][li][k])) / np.max(np.abs(rp["grads"][li][k]))
                if err > 1e-5:
                    bad.append(("grad", li, k, float(err)))
    return bad


def forward_backward(wl, params, x, y):
    m = so.from_workload(wl, real="float", bf16=True)
    m.load_params(params)
    m.forward(si.split_replicas(x, wl.R), si.split_replicas(y, wl.R))
    m.backward()
    return m


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_bf16_mode_equals_the_replay_with_explicit_roundings(name):
    wl1 = WORKLOADS[name](1, 1)
    params = si.make_params(wl1, bias_std=0.2)
    x, y = si.make_batch(wl1)
    rp = replay_unpartitioned(wl1, params, x, y)
    # unpartitioned oracle: bit for bit, gradients included
    assert compare_with_replay(forward_backward(wl1, params, x, y), rp, wl1, exact_grads=True) == []
    # partitioned oracle: the forward pass reorders no sum, so it is still bit-identical; the shard sum and the
    # replica sum reorder float additions in the backward pass (1e-5)
    wl2 = WORKLOADS[name](2, 2)
    bad = compare_with_replay(forward_backward(wl2, params, x, y), rp, wl2, exact_grads=False)
    assert bad == []


@pytest.mark.parametrize("name", list(WORKLOADS))
def test_every_single_rounding_call_is_seen_by_the_replay(name, monkeypatch):
    """Switch off one rounding call of the oracle at a time: the comparison with the replay must then fail.  (With all
    of them on it passes: the test above.)  So the replay pins every place where the oracle rounds."""
    wl = WORKLOADS[name](1, 1)
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    rp = replay_unpartitioned(wl, params, x, y)
    real_q = so.OracleModel._q
    counter = {"n": 0, "skip": -1}

    def q_with_one_hole(self, a):
        k = counter["n"]
        counter["n"] += 1
        return a if k == counter["skip"] else real_q(self, a)

    monkeypatch.setattr(so.OracleModel, "_q", q_with_one_hole)
    forward_backward(wl, params, x, y)
    n_calls = counter["n"]
    assert n_calls >= 2 * sum(1 for k, _ in wl.layers if k in (si.CONV3X3_RELU, si.FC_RELU, si.FC))
    unseen = []
    for k in range(n_calls):
        counter["n"], counter["skip"] = 0, k
        m = forward_backward(wl, params, x, y)
        if compare_with_replay(m, rp, wl, exact_grads=True) == []:
            unseen.append(k)
    # A rounding applied to values that are bf16 numbers already changes nothing, so it cannot be seen: that is the
    # gradient store of a conv layer that sits directly below a pooling layer (the pooling layer's backward pass only
    # routes the gradient values it has just stored, and the ReLU mask multiplies them by 0 or 1).
    idempotent = sum(1 for li, (kind, _) in enumerate(wl.layers[:-1]) if kind == si.CONV3X3_RELU and wl.layers[li + 1][0] == si.MAXPOOL2)
    assert len(unseen) <= idempotent, unseen
