"""GPU parity of the dropout layer [Listing 1, case DROPOUT | RELU]: the CUDA library through the C ABI against the CPU
oracle.  The keep mask is an integer decision (one 32-bit generator word against a threshold) and must agree bit for
bit; the float arithmetic around it is one multiplication per element and must agree exactly as well; whole iterations
hold the contract's element-wise tolerance in float mode."""
import numpy as np
import pytest

import sb_inputs as si
from sb_testutil import Checks, device_batch, gpu_model, maxrel, oracle_model

pytestmark = pytest.mark.gpu

SEED = 0x1234ABCD9876EF01
P25, P50 = 16384, 32768


def sb():
    from paper_2112_15317_b200 import binding
    return binding


def tc_net(classes=16):
    # FC widths that take the tensor-core kernels; two dropout layers with different probabilities
    return [(si.CONV3X3_RELU, 64), (si.MAXPOOL2, 0), (si.CONV3X3_RELU, 64), (si.MAXPOOL2, 0),
            (si.FC_RELU, 256), (si.DROPOUT, P25), (si.FC_RELU, 128), (si.DROPOUT, P50), (si.FC, classes), (si.SOFTMAX_XENT, classes)]


def ragged_net(classes=7):
    # widths that K = 3 does not divide; CUDA-core FC kernels; one FC layer kept whole below a dropout layer
    return [(si.CONV3X3_RELU, 24), (si.MAXPOOL2, 0), (si.FC_RELU, 70), (si.DROPOUT, 20000), (si.FC_RELU_WHOLE, 33), (si.DROPOUT, 3000),
            (si.FC, classes), (si.SOFTMAX_XENT, classes)]


WORKLOADS = {
    "tensor_core": lambda: si.Workload("drop_tc", tc_net(), 8, 8, 3, 4, 2, 2),
    "ragged": lambda: si.Workload("drop_ragged", ragged_net(), 12, 8, 4, 3, 2, 3),
}


def fc_act(gm, what, li):
    return gm.read(what, li, 0, squeeze=False)[:, :, 0, 0]


def drop_layers(wl):
    return [li for li, (k, _) in enumerate(wl.layers) if k == si.DROPOUT]


@pytest.mark.parametrize("name", ["tensor_core", "ragged"])
def test_float_mode_whole_iterations(name):
    b = sb()
    wl = WORKLOADS[name]()
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    om = oracle_model(wl, params, False); om.set_dropout(SEED, 41)
    gm = gpu_model(wl, params, b.SB_FP32); gm.dropout_seed(SEED, 41)
    xs, ys = device_batch(wl, x, y, False)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    c = Checks()
    for step in range(3):
        lo = float(om.forward(xr, yr)); om.backward()
        gm.forward(xs, ys); gm.backward()
        c.le((step, "loss"), abs(gm.loss() - lo) / abs(lo), 1e-4)
        for li in range(om.first_fc, len(wl.layers) - 1):
            act = fc_act(gm, b.SB_T_ACT, li)
            c.le((step, li, "act"), maxrel(act, om.fc_out[li]), 1e-4)
            dact = fc_act(gm, b.SB_T_DACT, li)
            if wl.layers[li][0] == si.DROPOUT:
                # the mask itself: bit for bit
                assert np.array_equal(act != 0, om.fc_out[li] != 0), (step, li)
                assert np.array_equal(act != 0, om.drop_keep[li] & (om.fc_out[li - 1] > 0)), (step, li)
                c.le((step, li, "dact"), maxrel(dact, om.d_pre[li] * (om.fc_out[li] != 0)), 1e-4)
            else:
                c.le((step, li, "dact"), maxrel(dact, om.d_pre[li]), 1e-4)
        gw, gb = gm.gather_params(b.SB_T_GRAD_W, b.SB_T_GRAD_B), None
        for li, g in enumerate(om.full_grads()):
            if g is not None:
                c.le((step, li, "dW"), maxrel(gw[li]["w"], g["w"]), 1e-4)
                c.le((step, li, "db"), maxrel(gw[li]["b"], g["b"]), 1e-4)
        om.sgd_step(0.02, 0.9); gm.sgd_step(0.02, 0.9)
    pw = gm.gather_params(b.SB_T_WEIGHT, b.SB_T_BIAS)
    for li, p in enumerate(om.full_params()):
        if p is not None:
            c.le((li, "w after 3 steps"), maxrel(pw[li]["w"], p["w"]), 1e-4)
    c.finish()
    # three iterations drew three different masks
    assert om.dropout_step == 44


@pytest.mark.parametrize("name", ["tensor_core", "ragged"])
def test_bf16_mode_layer_is_exact_on_the_stored_tensors(name):
    from oracle import splitbrain_oracle as so
    b = sb()
    wl = WORKLOADS[name]()
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    gm = gpu_model(wl, params, b.SB_BF16); gm.dropout_seed(SEED, 7)
    xs, ys = device_batch(wl, x, y, True)
    gm.forward(xs, ys); gm.backward()
    om = oracle_model(wl, params, True); om.set_dropout(SEED, 7)
    lo = float(om.forward(si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)))
    assert abs(gm.loss() - lo) / abs(lo) < 1e-2
    for li in drop_layers(wl):
        units = wl.layers[li][1]
        below = fc_act(gm, b.SB_T_ACT, li - 1)
        keep = so.dropout_keep(SEED, 7, li, np.arange(wl.B), below.shape[1], units)
        want = so.round_bf16(np.where(keep, below * so.dropout_scale(units), np.float32(0)))
        assert np.array_equal(fc_act(gm, b.SB_T_ACT, li), want), li
        assert abs(np.mean(~keep) - units / 65536.0) < 0.05
        # backward: the stored gradient w.r.t. the output is zero where the output is zero, and goes down times 1/(1 - p)
        dact = fc_act(gm, b.SB_T_DACT, li)
        assert np.all(dact[want == 0] == 0)
        assert np.array_equal(fc_act(gm, b.SB_T_DACT, li - 1), so.round_bf16(dact * so.dropout_scale(units))), li


def test_masks_do_not_depend_on_the_partitioning():
    b = sb()
    base = WORKLOADS["tensor_core"]().with_partition(1, 1)
    params = si.make_params(base, bias_std=0.2)
    x, y = si.make_batch(base)
    ref = None
    for R, K in [(1, 1), (2, 2), (4, 1), (2, 4), (8, 8)]:
        wl = base.with_partition(R, K)
        gm = gpu_model(wl, params, b.SB_BF16); gm.dropout_seed(SEED, 3)
        xs, ys = device_batch(wl, x, y, True)
        gm.forward(xs, ys)
        acts = [fc_act(gm, b.SB_T_ACT, li) for li in range(4, len(wl.layers) - 1)]
        if ref is None:
            ref = acts
        else:
            for a, r in zip(acts, ref):
                assert np.array_equal(a, r), (R, K)


def test_graph_replays_advance_the_iteration_and_match_the_oracle():
    b = sb()
    import torch
    wl = WORKLOADS["tensor_core"]()
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    om = oracle_model(wl, params, False); om.set_dropout(SEED, 0xFFFFFFFE)      # the 32-bit iteration word wraps inside the run
    gm = gpu_model(wl, params, b.SB_FP32); gm.dropout_seed(SEED, 0xFFFFFFFE)
    xs, ys = device_batch(wl, x, y, False)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    s = torch.cuda.Stream()
    losses_o, losses_g = [], []
    with torch.cuda.stream(s):
        for step in range(5):                     # direct, capture, three replays
            losses_o.append(float(om.step(xr, yr, 0.02, 0.9)))
            gm.graph_step(xs, ys, 0.02, 0.9)
            losses_g.append(gm.loss())
    s.synchronize()
    assert len(set(np.round(losses_o, 6))) == 5
    for lo, lg in zip(losses_o, losses_g):
        assert abs(lg - lo) / abs(lo) < 1e-4, (losses_o, losses_g)
    pw = gm.gather_params(b.SB_T_WEIGHT, b.SB_T_BIAS)
    for li, p in enumerate(om.full_params()):
        if p is not None:
            assert maxrel(pw[li]["w"], p["w"]) < 1e-4, li
    # same seed and iteration again: the same masks
    gm2 = gpu_model(wl, params, b.SB_FP32); gm2.dropout_seed(SEED, 0xFFFFFFFE)
    om2 = oracle_model(wl, params, False); om2.set_dropout(SEED, 0xFFFFFFFE)
    gm2.forward(xs, ys); om2.forward(xr, yr)
    assert np.array_equal(fc_act(gm2, b.SB_T_ACT, 5) != 0, om2.fc_out[5] != 0)


def test_full_size_vgg16_with_dropout_in_the_classifier():
    """The metric's network (VGG-16, CIFAR shape, batch 128, R = K = 4, bf16) with p = 0.5 dropout after both 4096-wide FC
    layers, in the launch configuration the benchmark times (sb_graph_step: multi-stream backward, update folded into the
    FC weight-gradient kernels).  Forward against the oracle; the dropout layers exactly, on the stored tensors; two
    graph iterations draw different masks."""
    from oracle import splitbrain_oracle as so
    b = sb()
    base = si.config(1)
    layers = []
    for kind, out in base.layers:
        layers.append((kind, out))
        if kind == si.FC_RELU:
            layers.append((si.DROPOUT, P50))
    wl = si.Workload("cfg1_dropout", layers, base.H, base.W, base.C, base.b, base.R, base.K)
    params = si.make_params(wl)
    x, y = si.make_batch(wl)
    gm = gpu_model(wl, params, b.SB_BF16); gm.dropout_seed(SEED, 100)
    xs, ys = device_batch(wl, x, y, True)
    gm.forward(xs, ys)
    om = oracle_model(wl, params, True); om.set_dropout(SEED, 100)
    lo = float(om.forward(si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)))
    assert abs(gm.loss() - lo) / abs(lo) < 1e-2
    drops = drop_layers(wl)
    assert len(drops) == 2
    masks = []
    for li in drops:
        below = fc_act(gm, b.SB_T_ACT, li - 1)
        keep = so.dropout_keep(SEED, 100, li, np.arange(wl.B), 4096, P50)
        want = so.round_bf16(np.where(keep, below * so.dropout_scale(P50), np.float32(0)))
        assert np.array_equal(fc_act(gm, b.SB_T_ACT, li), want), li
        assert abs(keep.mean() - 0.5) < 5 * 0.5 / np.sqrt(keep.size)
        assert maxrel(fc_act(gm, b.SB_T_ACT, li), om.fc_out[li]) < 2e-2
        masks.append(keep)
    # whole iterations through the graph path: iteration 101 (direct), 102 (captured), 103 (replayed)
    import torch
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for it in (101, 102, 103):
            gm.graph_step(xs, ys, 1e-3, 0.9)
            s.synchronize()
            li = drops[0]
            below = fc_act(gm, b.SB_T_ACT, li - 1)
            keep = so.dropout_keep(SEED, it, li, np.arange(wl.B), 4096, P50)
            assert np.array_equal(fc_act(gm, b.SB_T_ACT, li), so.round_bf16(np.where(keep, below * so.dropout_scale(P50), np.float32(0)))), it
            assert 0.4 < np.mean(keep != masks[0]) < 0.6
            # backward through the layer, on the stored gradients
            dact = fc_act(gm, b.SB_T_DACT, li)
            assert np.all(dact[fc_act(gm, b.SB_T_ACT, li) == 0] == 0)
            assert np.array_equal(fc_act(gm, b.SB_T_DACT, li - 1), so.round_bf16(dact * so.dropout_scale(P50))), it
    assert np.isfinite(gm.loss())


@pytest.mark.parametrize("name,R,K", [("tensor_core", 2, 2), ("tensor_core", 1, 4), ("ragged", 2, 3)])
def test_modulo_schedule_with_dropout(name, R, K):
    """sb_modulo_step: the K sub-iterations are one iteration, and every example meets the mask of its batch row although the
    sub-batches hold the rows in another order.  Float mode, two iterations, parameters and momentum within 1e-4; the masks
    of the last sub-iteration bit for bit."""
    b = sb()
    base = WORKLOADS[name]()
    wl = si.Workload(base.name + "_mod", base.layers, base.H, base.W, base.C, 2 * K, R, K)      # b = 2K rows per replica: sub-batches of 2R rows
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    om = oracle_model(wl, params, False); om.set_dropout(SEED, 77)
    gm = gpu_model(wl, params, b.SB_FP32, flags=b.SB_FLAG_MODULO_SCHEDULE); gm.dropout_seed(SEED, 77)
    xs, ys = device_batch(wl, x, y, False)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    from oracle import splitbrain_oracle as so
    for step in range(2):
        lo = float(om.step_modulo(xr, yr, 0.02, 0.9))
        gm.modulo_step(xs, ys, 0.02, 0.9)
        assert abs(gm.loss() - lo) / abs(lo) < 1e-4, step
        for what_w, what_b, ref_list in ((b.SB_T_WEIGHT, b.SB_T_BIAS, om.full_params()), (b.SB_T_MOM_W, b.SB_T_MOM_B, om.full_mom())):
            got = gm.gather_params(what_w, what_b)
            for li, (a, ref) in enumerate(zip(got, ref_list)):
                if ref is not None:
                    assert maxrel(a["w"].reshape(ref["w"].shape), ref["w"]) < 1e-4, (step, li)
                    assert maxrel(a["b"], ref["b"]) < 1e-4, (step, li)
        # the FC-side buffers hold the last sub-iteration in their last B/K rows, rows in sub-iteration order
        rows = om.modulo_rows(wl.K - 1)
        for li in drop_layers(wl):
            act = fc_act(gm, b.SB_T_ACT, li)[-len(rows):]
            below = fc_act(gm, b.SB_T_ACT, li - 1)[-len(rows):]
            keep = so.dropout_keep(SEED, 77 + step, li, rows, act.shape[1], wl.layers[li][1])
            assert np.array_equal(act != 0, keep & (below > 0)), (step, li)
    assert om.dropout_step == 79


def test_dropout_is_refused_where_it_is_not_supported():
    b = sb()
    bad_after_conv = [(si.CONV3X3_RELU, 8), (si.DROPOUT, P25), (si.FC, 4), (si.SOFTMAX_XENT, 4)]
    with pytest.raises(b.SBError, match="must follow an FC"):
        b.Model(bad_after_conv, 4, 4, 4, 2, 1, 1)
    bad_p = [(si.CONV3X3_RELU, 8), (si.FC_RELU, 8), (si.DROPOUT, 65536), (si.FC, 4), (si.SOFTMAX_XENT, 4)]
    with pytest.raises(b.SBError, match="drop probability"):
        b.Model(bad_p, 4, 4, 4, 2, 1, 1)
