"""GPU parity at the benchmark configurations' own sizes.

* cfg1 network at a reduced batch (same R, K, layers and tile shapes per image): every layer element-wise.
* cfg1 / cfg5 / cfg2 / cfg3 at FULL size, in the launch configuration bench.py times: every layer's kernels on forced
  inputs and one whole iteration end to end, element-wise; cfg1 and cfg5 with all 128 images distinct (the oracle
  runs the whole batch), cfg2 / cfg3 with 8 / 4 distinct images staggered over the replicas.
* cfg2 / cfg3 with all images distinct: the oracle follows a few sampled images through the forward pass (each
  image's forward computation is independent of the rest of the batch); partition invariance of the full-size run.
* cfg4: the sharded-FC sweep (25088 x 4096, batch 32/128/512, K in 1..8, R in 1,4): equality across K against
  K = 1 and sampled outputs against the oracle.
"""
import numpy as np
import pytest

import sb_inputs as si
from sb_testutil import Checks, device_batch, gpu_model, maxrel

pytestmark = pytest.mark.gpu


def sb():
    from paper_2112_15317_b200 import binding
    return binding


def test_cfg1_network_reduced_batch_every_layer():
    from test_gpu_parity_small import compare_everything, layerwise_teacher_forced
    wl = si.config(1).with_batch(4)          # B = 16, R = 4, K = 4
    layerwise_teacher_forced(wl, bf16=True, bias_std=0.05)
    compare_everything(wl, bf16=True, steps=2, bias_std=0.0)


@pytest.mark.parametrize("cfg,distinct", [(1, 128), (5, 128), (2, 8), (3, 4)])
def test_full_size_every_layer_and_whole_iteration(cfg, distinct):
    """The configuration at its FULL batch, R, K (bench.py's launch configuration).  cfg1 and cfg5: all 128 images
    distinct, the oracle runs the whole batch.  cfg2 / cfg3: 8 / 4 distinct images, staggered so that neighbouring
    replicas start with different images.  First every layer's kernels on forced inputs, element-wise (forward,
    argmax bytes, input gradient, weight and bias gradient); then one whole iteration end to end: forward tensors,
    weight / bias gradients, momentum and updated weights element-wise, activation gradients by outlier fraction."""
    from test_gpu_parity_small import Ref, end_to_end_vs_ref, layerwise_teacher_forced
    wl = si.config(cfg)
    ref = Ref(wl, True, 0.05, distinct)
    layerwise_teacher_forced(wl, bf16=True, ref=ref)
    end_to_end_vs_ref(ref)


def sampled_image_check(wl, picks):
    """Full-size GPU forward + backward on the configuration's own batch (all images distinct); the oracle follows
    the images `picks` (global batch indices) through the forward pass (the backward pass at full size:
    test_full_size_every_layer_and_whole_iteration).  Chained forward tensors: see TOL_ACT_CHAIN."""
    from test_gpu_parity_small import TOL_ACT_CHAIN
    b = sb()
    params = si.make_params(wl)
    x, y = si.make_batch(wl)
    gm = gpu_model(wl, params, b.SB_BF16)
    xs, ys = device_batch(wl, x, y, True)
    gm.forward(xs, ys)
    gm.backward()
    loss = gm.loss()
    assert np.isfinite(loss)
    sub = si.Workload(wl.name + "_picked", wl.layers, wl.H, wl.W, wl.C, len(picks), 1, wl.K)
    from oracle import splitbrain_oracle as so
    om = so.from_workload(sub, real="float", bf16=True, loss_B=wl.B)
    om.load_params(params)
    om.forward([x[picks]], [y[picks]])
    nl = len(wl.layers)
    ck = Checks()
    for li, (kind, out) in enumerate(wl.layers):
        if kind in (si.CONV3X3_RELU, si.MAXPOOL2):
            reps = sorted({g // wl.b for g in picks})
            acts = {r: gm.read(b.SB_T_ACT, li, r, squeeze=False) for r in reps}
            a = np.stack([acts[g // wl.b][g % wl.b] for g in picks])
            ck.le(("act", li), maxrel(a, om.conv_out[0][li]), TOL_ACT_CHAIN[True])
        elif kind in (si.FC_RELU, si.FC):
            a = gm.read(b.SB_T_ACT, li, 0, squeeze=False)[:, :, 0, 0][picks]
            ck.le(("fc act", li), maxrel(a, om.fc_out[li]), TOL_ACT_CHAIN[True])
    ck.le(("row loss",), maxrel(gm.read(b.SB_T_ROW_LOSS, nl - 1, 0)[picks], om.row_loss), TOL_ACT_CHAIN[True])
    ck.finish()
    return gm, (xs, ys), loss


def test_cfg2_full_size_sampled_images_and_partition_invariance():
    b = sb()
    wl = si.config(2)                         # batch 256, R = 8, K = 8
    gm, (xs, ys), loss = sampled_image_check(wl, [3, 255])
    logits = gm.read(b.SB_T_ACT, len(wl.layers) - 2, 0, squeeze=False)[:, :, 0, 0]
    grads = gm.gather_params(b.SB_T_GRAD_W, b.SB_T_GRAD_B)
    gm.close()
    # the same batch, unpartitioned (R = K = 1): loss, logits and gradients must not change
    base = wl.with_partition(1, 1)
    params = si.make_params(base)
    x, y = si.make_batch(base)
    g1 = gpu_model(base, params, b.SB_BF16)
    xs1, ys1 = device_batch(base, x, y, True)
    g1.forward(xs1, ys1); g1.backward()
    assert g1.loss() == pytest.approx(loss, rel=1e-6)
    assert np.array_equal(g1.read(b.SB_T_ACT, len(wl.layers) - 2, 0, squeeze=False)[:, :, 0, 0], logits)
    for a, ref in zip(grads, g1.gather_params(b.SB_T_GRAD_W, b.SB_T_GRAD_B)):
        if ref is not None:
            assert maxrel(a["w"], ref["w"]) <= 1e-4 and maxrel(a["b"], ref["b"]) <= 1e-4
    g1.close()


def test_cfg5_paper_vgg_variant_reduced_batch_two_steps():
    """The paper's own evaluation network (Table 1: 7 conv + 3 FC layers on 32x32 images) as one MP group of four
    workers, two whole training steps at a reduced batch (the full batch: test_full_size_every_layer_and_whole_iteration)."""
    from test_gpu_parity_small import compare_everything
    compare_everything(si.config(5).with_batch(4), bf16=True, steps=2, bias_std=0.0)


def test_cfg3_full_size_sampled_image():
    gm, _, _ = sampled_image_check(si.config(3), [21])
    gm.close()


@pytest.mark.parametrize("B", [32, 128, 512])
def test_cfg4_sharded_fc_sweep(B):
    import torch
    from oracle import splitbrain_oracle as so
    b = sb()
    d_in, d_out = 25088, 4096
    w, x, dy = si.fc_sweep_case(B)
    P = so.Prims("float")
    w_bf, x_bf, dy_bf = so.round_bf16(w), so.round_bf16(x), so.round_bf16(dy)
    layers = [(si.FC, d_out), (si.SOFTMAX_XENT, d_out)]
    xt = torch.from_numpy(x).cuda().to(torch.bfloat16)
    params = [{"w": w, "b": np.zeros(d_out, np.float32)}, None]
    results = {}
    for R in (1, 4):
        for K in (1, 2, 4, 8):
            wl = si.Workload(f"fc_sweep_B{B}_R{R}_K{K}", layers, 1, 1, d_in, B // R, R, K)
            gm = gpu_model(wl, params, b.SB_BF16, flags=b.SB_FLAG_INPUT_GRAD)
            xs = [xt[r * wl.b:(r + 1) * wl.b] for r in range(R)]          # R views of one buffer: gather by addressing
            gm.forward_layers(0, 0, xs, None)
            gm.write(b.SB_T_DACT, 0, 0, dy)
            gm.backward_layers(0, 0)
            Y = gm.read(b.SB_T_ACT, 0, 0, squeeze=False)[:, :, 0, 0]
            dX = np.concatenate([gm.read(b.SB_T_INPUT_GRAD, 0, r, squeeze=False)[:, 0, 0, :] for r in range(R)])
            dW = gm.gather_params(b.SB_T_GRAD_W, b.SB_T_GRAD_B)[0]["w"]
            results[(R, K)] = (Y, dX, dW)
            gm.close()
    Y0, dX0, dW0 = results[(1, 1)]
    for key, (Y, dX, dW) in results.items():
        assert np.array_equal(Y, Y0), key                       # forward: bit-identical for every partitioning
        assert maxrel(dX, dX0) <= 1e-2 and maxrel(dW, dW0) <= 1e-2, key
    # sampled outputs against the oracle (rows / columns it can compute one by one)
    rows = [0, B // 2, B - 1]
    cols = [0, 1023, 1024, 4095]
    Yo = P.fc_fwd(x_bf[rows], w_bf[cols], np.zeros(len(cols), np.float32), relu=False)
    assert maxrel(Y0[np.ix_(rows, cols)], Yo) <= 1e-2
    _, _, dXo = P.fc_bwd(x_bf[rows], w_bf, dy_bf[rows])
    assert maxrel(dX0[rows], so.round_bf16(dXo)) <= 1e-2
    dWo, _, _ = P.fc_bwd(x_bf, w_bf[cols], np.ascontiguousarray(dy_bf[:, cols]))
    assert maxrel(dW0[cols], dWo) <= 1e-2
