"""GPU parity of sb_modulo_step (the modulo layer's own schedule: K FC sub-iterations per iteration) against the
oracle's step_modulo, through the C ABI.  Float mode: every parameter and momentum tensor within 1e-4.  bf16 mode:
loss and parameters within 1e-2 element-wise; momentum (= sums of gradients) in the Frobenius norm, as in the
end-to-end test of the synchronous step (a ReLU mask or pool argmax that flips moves single gradient elements)."""
import numpy as np
import pytest

import sb_inputs as si
from sb_testutil import device_batch, frob, gpu_model, maxrel, oracle_model
from test_gpu_parity_small import TOL, ragged_net, tensor_core_net

pytestmark = pytest.mark.gpu

CASES = {
    # tensor-core FC layers (256, 128 wide) + the narrow logits layer; B = 8, sub-batches of 4 rows
    "tensor_core": lambda: si.Workload("modulo_tc", tensor_core_net(), 12, 20, 3, 4, 2, 2),
    # CUDA-core FC kernels, shard widths that do not divide (70, 33, 7 over K = 3); B = 12, sub-batches of 4 rows
    "ragged": lambda: si.Workload("modulo_ragged", ragged_net(), 20, 12, 4, 6, 2, 3),
    # the FC stack and partition of the VGG-16 / CIFAR configuration (512 -> 4096 -> 4096 -> 10, B = 128, R = 4,
    # K = 4: sub-batches of 32 rows) behind a one-layer conv front that also yields 512 features
    "cfg1_fc_stack": lambda: si.Workload("modulo_cfg1_fc", [(si.CONV3X3_RELU, 128), (si.MAXPOOL2, 0), (si.FC_RELU, 4096), (si.FC_RELU, 4096),
                                                           (si.FC, 10), (si.SOFTMAX_XENT, 10)], 4, 4, 3, 32, 4, 4),
    # K = 4 sub-iterations of a single replica
    "one_replica": lambda: si.Workload("modulo_r1", tensor_core_net(), 8, 8, 3, 8, 1, 4),
}


def sb():
    from paper_2112_15317_b200 import binding
    return binding


def run(wl, bf16, steps=2, lr=0.01, mu=0.9):
    b = sb()
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    om = oracle_model(wl, params, bf16)
    gm = gpu_model(wl, params, b.SB_BF16 if bf16 else b.SB_FP32, flags=b.SB_FLAG_MODULO_SCHEDULE)
    xs, ys = device_batch(wl, x, y, bf16)
    xr, yr = si.split_replicas(x, wl.R), si.split_replicas(y, wl.R)
    tol = TOL[bf16]
    for step in range(steps):
        lo = float(om.step_modulo(xr, yr, lr, mu))
        gm.modulo_step(xs, ys, lr, mu)
        lg = gm.loss()
        assert abs(lg - lo) <= tol * max(1.0, abs(lo)), (step, lg, lo)
        # the library keeps the row losses in sub-iteration order (the order the modulo layer's copy produces)
        order = np.concatenate([om.modulo_rows(k) for k in range(wl.K)])
        rl = gm.read(b.SB_T_ROW_LOSS, len(wl.layers) - 1, 0)
        if bf16 and step > 0:
            assert frob(rl, om.row_loss[order]) <= tol, (step, frob(rl, om.row_loss[order]))
        else:
            assert maxrel(rl, om.row_loss[order]) <= tol, (step, maxrel(rl, om.row_loss[order]))
        for what_w, what_b, ref_list, is_mom in ((b.SB_T_WEIGHT, b.SB_T_BIAS, om.full_params(), False),
                                                 (b.SB_T_MOM_W, b.SB_T_MOM_B, om.full_mom(), True)):
            got = gm.gather_params(what_w, what_b)
            for li, (a, ref) in enumerate(zip(got, ref_list)):
                if ref is None:
                    continue
                aw = a["w"].reshape(ref["w"].shape)
                if is_mom and bf16:
                    bound = 3 * tol if step == 0 else 0.3
                    assert frob(aw, ref["w"]) <= bound, ("mom w", step, li, frob(aw, ref["w"]))
                    assert frob(a["b"], ref["b"]) <= bound, ("mom b", step, li, frob(a["b"], ref["b"]))
                elif bf16 and step > 0:
                    # the second iteration starts from weights that already differ by flipped masks: norm-wise bound
                    assert frob(aw, ref["w"]) <= tol, ("w", step, li, frob(aw, ref["w"]))
                else:
                    assert maxrel(aw, ref["w"]) <= tol, ("w" if not is_mom else "mom w", step, li, maxrel(aw, ref["w"]))
                    if not bf16:
                        assert maxrel(a["b"], ref["b"]) <= tol, ("b", step, li)
    gm.close()


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("bf16", [False, True])
def test_modulo_step_matches_oracle(name, bf16):
    # One iteration already holds K forward / backward / update rounds of the FC stack.  A second iteration in bf16 mode starts
    # from weights that differ by flipped ReLU masks, where no element-wise bound can hold (float mode runs two).
    run(CASES[name](), bf16, steps=1 if bf16 else 2)


def test_modulo_step_with_K1_equals_the_synchronous_calls():
    b = sb()
    wl = si.Workload("modulo_k1", tensor_core_net(), 12, 20, 3, 3, 2, 1)
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    xs, ys = device_batch(wl, x, y, True)
    res = []
    for modulo in (True, False):
        gm = gpu_model(wl, params, b.SB_BF16, flags=b.SB_FLAG_MODULO_SCHEDULE)
        for _ in range(2):
            if modulo:
                gm.modulo_step(xs, ys, 0.02, 0.9)
            else:
                gm.forward(xs, ys); gm.backward(); gm.sgd_step(0.02, 0.9)
        res.append((gm.loss(), gm.gather_params(b.SB_T_WEIGHT, b.SB_T_BIAS)))
        gm.close()
    assert res[0][0] == res[1][0]
    for a, c in zip(res[0][1], res[1][1]):
        if a is not None:
            assert np.array_equal(a["w"], c["w"]) and np.array_equal(a["b"], c["b"])


def test_modulo_step_replayed_as_a_graph_equals_the_direct_calls():
    """On a side stream sb_modulo_step captures the iteration on its second call and replays it afterwards (all weight
    streams joined, the conv layers' updates applied inside their split reduces): losses and parameters must be
    bit-identical to the same steps enqueued directly on the default stream."""
    import torch
    b = sb()
    wl = si.Workload("modulo_graph", tensor_core_net(), 12, 20, 3, 4, 2, 2)
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    xs, ys = device_batch(wl, x, y, True)
    g1 = gpu_model(wl, params, b.SB_BF16, flags=b.SB_FLAG_MODULO_SCHEDULE)
    g2 = gpu_model(wl, params, b.SB_BF16, flags=b.SB_FLAG_MODULO_SCHEDULE)
    losses1 = []
    for _ in range(4):
        g1.modulo_step(xs, ys, 0.02, 0.9); losses1.append(g1.loss())
    side = torch.cuda.Stream()
    losses2 = []
    with torch.cuda.stream(side):
        for _ in range(4):
            g2.modulo_step(xs, ys, 0.02, 0.9); losses2.append(g2.loss())
        side.synchronize()
    assert losses1 == losses2
    for a, c in zip(g1.gather_params(b.SB_T_WEIGHT, b.SB_T_BIAS), g2.gather_params(b.SB_T_WEIGHT, b.SB_T_BIAS)):
        if a is not None:
            assert np.array_equal(a["w"], c["w"]) and np.array_equal(a["b"], c["b"])
    g1.close(); g2.close()


def test_modulo_step_needs_the_flag_and_a_divisible_batch():
    b = sb()
    wl = si.Workload("modulo_noflag", tensor_core_net(), 8, 8, 3, 4, 2, 2)
    params = si.make_params(wl)
    x, y = si.make_batch(wl)
    xs, ys = device_batch(wl, x, y, True)
    gm = gpu_model(wl, params, b.SB_BF16)
    with pytest.raises(b.SBError, match="SB_ERR_STATE"):
        gm.modulo_step(xs, ys, 0.01, 0.9)
    gm.close()
    bad = si.Workload("modulo_bad", tensor_core_net(), 8, 8, 3, 3, 2, 2)          # b = 3 is not a multiple of K = 2
    with pytest.raises(b.SBError, match="SB_ERR_UNSUPPORTED"):
        gpu_model(bad, si.make_params(bad), b.SB_BF16, flags=b.SB_FLAG_MODULO_SCHEDULE)
