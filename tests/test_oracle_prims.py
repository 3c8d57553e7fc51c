"""Pins for the oracle's layer primitives: brute-force single-element evaluators written from the
definitions, closed forms, adjoint identities and library routines (float64 torch) as a second
opinion.  None of these re-use the oracle's own code."""
import math

import numpy as np
import pytest
import torch

from oracle import splitbrain_oracle as so

P64 = so.Prims("double")
P32 = so.Prims("float")
rng = np.random.default_rng(7)


def _rand(*shape):
    return rng.standard_normal(shape)


# ---- independent single-element evaluators (definitions typed out again, scalar Python) --------
def conv_elem(x, w, bias, n, h, ww, k):
    N, H, W, C = x.shape
    acc = float(bias[k])
    for r in range(3):
        for s in range(3):
            hh, wc = h + r - 1, ww + s - 1
            if 0 <= hh < H and 0 <= wc < W:
                for c in range(C):
                    acc += float(x[n, hh, wc, c]) * float(w[k, r, s, c])
    return acc


def dgrad_elem(dy, w, n, h, ww, c):
    N, H, W, K = dy.shape
    acc = 0.0
    for r in range(3):
        for s in range(3):
            hh, wc = h - r + 1, ww - s + 1
            if 0 <= hh < H and 0 <= wc < W:
                for k in range(K):
                    acc += float(dy[n, hh, wc, k]) * float(w[k, r, s, c])
    return acc


def wgrad_elem(x, dy, k, r, s, c):
    N, H, W, _ = x.shape
    acc = 0.0
    for n in range(N):
        for h in range(H):
            for ww in range(W):
                hh, wc = h + r - 1, ww + s - 1
                if 0 <= hh < H and 0 <= wc < W:
                    acc += float(dy[n, h, ww, k]) * float(x[n, hh, wc, c])
    return acc


def test_conv_fwd_brute_force_elements():
    x, w, b = _rand(2, 6, 5, 3), _rand(4, 3, 3, 3), _rand(4)
    y = P64.conv_fwd(x, w, b, relu=False)
    for _ in range(60):
        n, h, ww, k = rng.integers(2), rng.integers(6), rng.integers(5), rng.integers(4)
        assert y[n, h, ww, k] == pytest.approx(conv_elem(x, w, b, n, h, ww, k), rel=1e-12, abs=1e-12)
    # all four corners and an edge explicitly (padding)
    for (h, ww) in [(0, 0), (0, 4), (5, 0), (5, 4), (0, 2), (3, 0)]:
        assert y[1, h, ww, 2] == pytest.approx(conv_elem(x, w, b, 1, h, ww, 2), rel=1e-12, abs=1e-12)


def test_conv_fwd_ones_counts_padding():
    """All-ones 3x3 kernel on an all-ones single-channel image counts the in-bounds taps:
    9 inside, 6 on an edge, 4 in a corner."""
    x = np.ones((1, 5, 7, 1))
    y = P64.conv_fwd(x, np.ones((1, 3, 3, 1)), np.zeros(1), relu=False)[0, :, :, 0]
    assert y[2, 3] == 9 and y[0, 3] == 6 and y[2, 0] == 6 and y[4, 6] == 4 and y[0, 0] == 4
    assert y.sum() == 9 * 3 * 5 + 6 * (2 * 5 + 2 * 3) + 4 * 4


def test_conv_fwd_centre_tap_is_identity_and_shift_direction():
    x = _rand(1, 4, 4, 2)
    w = np.zeros((2, 3, 3, 2))
    w[0, 1, 1, 0] = 1.0
    w[1, 1, 1, 1] = 1.0
    y = P64.conv_fwd(x, w, np.zeros(2), relu=True)
    assert np.array_equal(y, np.maximum(x, 0))
    # tap (r=0,s=2) reads x[h-1, w+1]: cross-correlation, no kernel flip
    w = np.zeros((1, 3, 3, 2))
    w[0, 0, 2, 1] = 1.0
    y = P64.conv_fwd(x, w, np.zeros(1), relu=False)
    assert y[0, 2, 1, 0] == x[0, 1, 2, 1]
    assert y[0, 0, 1, 0] == 0.0 and y[0, 2, 3, 0] == 0.0


def test_conv_matches_torch_float64():
    x, w, b = _rand(3, 8, 6, 5), _rand(7, 3, 3, 5), _rand(7)
    y = P64.conv_fwd(x, w, b, relu=False)
    xt = torch.tensor(x).permute(0, 3, 1, 2).requires_grad_(True)
    wt = torch.tensor(w).permute(0, 3, 1, 2).requires_grad_(True)
    bt = torch.tensor(b, requires_grad=True)
    yt = torch.nn.functional.conv2d(xt, wt, bt, padding=1)
    np.testing.assert_allclose(y, yt.detach().permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    dy = _rand(3, 8, 6, 7)
    yt.backward(torch.tensor(dy).permute(0, 3, 1, 2))
    dx = P64.conv_dgrad(dy, w)
    dw, db = P64.conv_wgrad(x, dy)
    np.testing.assert_allclose(dx, xt.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(dw, wt.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-11, atol=1e-11)
    np.testing.assert_allclose(db, bt.grad.numpy(), rtol=1e-11, atol=1e-11)


def test_conv_dgrad_wgrad_brute_force_elements():
    x, w, dy = _rand(2, 5, 4, 3), _rand(4, 3, 3, 3), _rand(2, 5, 4, 4)
    dx = P64.conv_dgrad(dy, w)
    dw, db = P64.conv_wgrad(x, dy)
    for _ in range(40):
        n, h, ww, c = rng.integers(2), rng.integers(5), rng.integers(4), rng.integers(3)
        assert dx[n, h, ww, c] == pytest.approx(dgrad_elem(dy, w, n, h, ww, c), rel=1e-12, abs=1e-12)
    for k in range(4):
        for r in range(3):
            for s in range(3):
                c = int(rng.integers(3))
                assert dw[k, r, s, c] == pytest.approx(wgrad_elem(x, dy, k, r, s, c), rel=1e-12, abs=1e-12)
    np.testing.assert_allclose(db, dy.sum((0, 1, 2)), rtol=1e-12)


def test_conv_adjoint_identities():
    """<conv(x), dy> = <x, dgrad(dy)> = <w, wgrad(x, dy)> for the bias-free, ReLU-free map."""
    x, w, dy = _rand(2, 7, 6, 4), _rand(5, 3, 3, 4), _rand(2, 7, 6, 5)
    y = P64.conv_fwd(x, w, np.zeros(5), relu=False)
    lhs = float((y * dy).sum())
    assert float((x * P64.conv_dgrad(dy, w)).sum()) == pytest.approx(lhs, rel=1e-12)
    assert float((w * P64.conv_wgrad(x, dy)[0]).sum()) == pytest.approx(lhs, rel=1e-12)


def test_float_build_agrees_with_double_build():
    x, w, b, dy = _rand(2, 6, 6, 8), _rand(6, 3, 3, 8) * 0.2, _rand(6), _rand(2, 6, 6, 6)
    for f in ("conv_fwd", ):
        np.testing.assert_allclose(P32.conv_fwd(x, w, b), P64.conv_fwd(x, w, b), rtol=2e-5, atol=2e-5)
    np.testing.assert_allclose(P32.conv_dgrad(dy, w), P64.conv_dgrad(dy, w), rtol=2e-5, atol=2e-5)
    np.testing.assert_allclose(P32.conv_wgrad(x, dy)[0], P64.conv_wgrad(x, dy)[0], rtol=2e-5, atol=5e-5)


# ---- max-pool --------------------------------------------------------------------------------
def test_maxpool_brute_force_argmax_and_routing():
    x = _rand(2, 6, 4, 3)
    p, idx = P64.pool_fwd(x)
    for n in range(2):
        for h in range(3):
            for w in range(2):
                for c in range(3):
                    win = [x[n, 2 * h + (q >> 1), 2 * w + (q & 1), c] for q in range(4)]
                    assert p[n, h, w, c] == max(win)
                    assert idx[n, h, w, c] == win.index(max(win))
    dp = _rand(2, 3, 2, 3)
    dx = P64.pool_bwd(dp, idx)
    assert dx.sum() == pytest.approx(dp.sum(), rel=1e-12)
    nz = (dx.reshape(2, 3, 2, 2, 2, 3).transpose(0, 1, 3, 5, 2, 4).reshape(2, 3, 2, 3, 4) != 0).sum(-1)
    assert np.all(nz == 1)
    pt = torch.tensor(x).permute(0, 3, 1, 2).requires_grad_(True)
    yt = torch.nn.functional.max_pool2d(pt, 2)
    yt.backward(torch.tensor(dp).permute(0, 3, 1, 2))
    np.testing.assert_array_equal(p, yt.detach().permute(0, 2, 3, 1).numpy())
    np.testing.assert_array_equal(dx, pt.grad.permute(0, 2, 3, 1).numpy())


def test_maxpool_tie_goes_to_first_in_scan_order():
    x = np.zeros((1, 2, 2, 3))
    x[0, 0, 1, 1] = x[0, 1, 0, 1] = 5.0      # tie between positions 1 and 2
    x[0, 1, 1, 2] = x[0, 1, 0, 2] = 2.0      # tie between positions 2 and 3
    p, idx = P64.pool_fwd(x)
    assert list(idx[0, 0, 0]) == [0, 1, 2] and list(p[0, 0, 0]) == [0.0, 5.0, 2.0]


# ---- FC shard --------------------------------------------------------------------------------
def test_fc_matches_matmul_float64():
    X, Wt, b, dY = _rand(5, 11), _rand(7, 11), _rand(7), _rand(5, 7)
    Y = P64.fc_fwd(X, Wt, b, relu=False)
    np.testing.assert_allclose(Y, (torch.tensor(X) @ torch.tensor(Wt).T + torch.tensor(b)).numpy(), rtol=1e-12, atol=1e-12)
    assert np.array_equal(P64.fc_fwd(X, Wt, b, relu=True), np.maximum(Y, 0))
    dW, db, dX = P64.fc_bwd(X, Wt, dY)
    np.testing.assert_allclose(dW, (torch.tensor(dY).T @ torch.tensor(X)).numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dX, (torch.tensor(dY) @ torch.tensor(Wt)).numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(db, dY.sum(0), rtol=1e-12)
    # orientation: weight row o produces output column o
    Wt2 = np.zeros((7, 11)); Wt2[3, 4] = 2.0
    assert P64.fc_fwd(X, Wt2, np.zeros(7), relu=False)[2, 3] == 2.0 * X[2, 4]


# ---- loss ------------------------------------------------------------------------------------
@pytest.mark.parametrize("C", [10, 1000])
def test_softmax_xent_zero_logits_closed_form(C):
    B = 4
    labels = np.array([0, C - 1, 3, 3], np.int32)
    row, dZ = P64.softmax_xent(np.zeros((B, C)), labels, 1.0 / B)
    np.testing.assert_allclose(row, math.log(C), rtol=1e-14)
    exp = np.full((B, C), 1.0 / C) ; exp[np.arange(B), labels] -= 1.0
    np.testing.assert_allclose(dZ, exp / B, rtol=1e-13, atol=1e-16)


def test_softmax_xent_matches_torch_and_is_shift_invariant():
    Z = _rand(6, 10) * 3
    labels = rng.integers(0, 10, 6).astype(np.int32)
    row, dZ = P64.softmax_xent(Z, labels, 1.0 / 6)
    zt = torch.tensor(Z, requires_grad=True)
    lt = torch.nn.functional.cross_entropy(zt, torch.tensor(labels).long(), reduction="mean")
    lt.backward()
    assert row.mean() == pytest.approx(lt.item(), rel=1e-13)
    np.testing.assert_allclose(dZ, zt.grad.numpy(), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(dZ.sum(1), 0, atol=1e-15)
    row2, dZ2 = P64.softmax_xent(Z + 1000.0, labels, 1.0 / 6)     # no overflow, same answer
    np.testing.assert_allclose(row2, row, rtol=1e-9)
    np.testing.assert_allclose(dZ2, dZ, atol=1e-12)


def test_label_indexing_exact():
    """The row loss picks column labels[g] exactly: a one-hot-like logit row gives ~0 only there."""
    C = 10
    for y in range(C):
        Z = np.full((1, C), -50.0); Z[0, y] = 50.0
        for lab in range(C):
            row, _ = P64.softmax_xent(Z, np.array([lab], np.int32), 1.0)
            assert (row[0] < 1e-9) == (lab == y)
            if lab != y:
                assert row[0] == pytest.approx(100.0, rel=1e-12)


# ---- SGD -------------------------------------------------------------------------------------
def test_sgd_momentum_closed_form():
    """Constant gradient g: v_t = g (1-mu^t)/(1-mu), w_t = w_0 - lr * sum_{s<=t} v_s."""
    lr, mu, T = 0.01, 0.9, 7
    g = _rand(9)
    w0 = _rand(9)
    w, v = w0.copy(), np.zeros(9)
    for _ in range(T):
        P64.sgd(w, v, g, lr, mu)
    vt = g * (1 - mu ** T) / (1 - mu)
    ssum = sum((1 - mu ** s) / (1 - mu) for s in range(1, T + 1))
    np.testing.assert_allclose(v, vt, rtol=1e-13)
    np.testing.assert_allclose(w, w0 - lr * g * ssum, rtol=1e-12, atol=1e-14)
    w, v = w0.copy(), np.ones(9)
    P64.sgd(w, v, g, lr, 0.0)                      # mu = 0: plain gradient step, old v ignored
    np.testing.assert_allclose(w, w0 - lr * g, rtol=1e-14)


# ---- bf16 rounding helper ----------------------------------------------------------------------
def test_round_bf16_matches_torch_and_ties_to_even():
    a = (_rand(4000) * np.exp(_rand(4000) * 8)).astype(np.float32)
    ref = torch.tensor(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(so.round_bf16(a), ref)
    # 1 + 2^-8 is exactly halfway between 1 and 1+2^-7: ties to even -> 1 ; 1+3*2^-8 -> 1+2^-6
    assert so.round_bf16(np.array([1 + 2.0 ** -8], np.float32))[0] == 1.0
    assert so.round_bf16(np.array([1 + 3 * 2.0 ** -8], np.float32))[0] == np.float32(1 + 2.0 ** -6)
