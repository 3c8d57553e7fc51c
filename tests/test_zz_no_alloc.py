"""The allocation-free entry point sb_conv_in_wgrad_static against the model path's input-layer weight
gradient (sb_backward_layers on layer 0) and against the CPU oracle's conv weight gradient, through the C ABI,
twice in a row with different data.

The entry point is for callers that may not create device memory when they need the gradient (a hook
running beside a job whose pool owns the GPU, a host that forbids allocation after start-up): it keeps
its split partial sums in an array built into the library.  The second call checks that the contents
the first call left in that shared array do not leak into the next result.  This file is collected
last so that a run which stops at the first failure has already run every other test."""
import numpy as np
import pytest

import sb_inputs as si

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bf16", [False, True])
def test_static_scratch_wgrad_matches_model_path_twice(bf16):
    import torch
    from paper_2112_15317_b200 import binding as sb

    # a net whose first layer is a 3 -> 64 convolution; 20 images of 12x20 pixels = 75 chunks of 64 pixels
    layers = [(si.CONV3X3_RELU, 64), (si.MAXPOOL2, 0), (si.FC, 10), (si.SOFTMAX_XENT, 10)]
    wl = si.Workload("static_wgrad", layers, 12, 20, 3, 10, 2, 2)
    prec = sb.SB_BF16 if bf16 else sb.SB_FP32
    m = sb.Model.from_workload(wl, precision=prec)
    m.load_params(si.make_params(wl), si.shard_bounds)
    tdt = torch.bfloat16 if bf16 else torch.float32
    rng = np.random.default_rng(11)
    dw = torch.empty((64, 3, 3, 3), dtype=torch.float32, device="cuda")
    db = torch.empty((64,), dtype=torch.float32, device="cuda")
    tol = 1e-2 if bf16 else 1e-4
    for call in range(2):
        x = rng.standard_normal((wl.B, 12, 20, 3)).astype(np.float32) * (1.0 + call)
        dy = rng.standard_normal((wl.B, 12, 20, 64)).astype(np.float32) * (0.5 + 2 * call)
        xt = torch.from_numpy(x).cuda().to(tdt)
        xs = [xt[r * wl.b:(r + 1) * wl.b].contiguous() for r in range(wl.R)]
        # existing entry point: the model's backward of layer 0.  The forward call hands the model the
        # replica input pointers; the gradient w.r.t. layer 0's output is then written into the model.
        m.forward_layers(0, 0, xs, None)
        for r in range(wl.R):
            m.write(sb.SB_T_DACT, 0, r, dy[r * wl.b:(r + 1) * wl.b])
        m.backward_layers(0, 0)
        ref_w = m.read(sb.SB_T_GRAD_W, 0, 0, squeeze=False)
        ref_b = m.read(sb.SB_T_GRAD_B, 0, 0)
        # new entry point: the same values in the caller's own contiguous buffers
        dyt = torch.from_numpy(dy).cuda().to(tdt)
        dw.fill_(float("nan")); db.fill_(float("nan"))
        sb.conv_in_wgrad_static(xt, dyt, dw, db, prec)
        torch.cuda.synchronize()
        got_w, got_b = dw.cpu().numpy(), db.cpu().numpy()
        assert np.isfinite(got_w).all() and np.isfinite(got_b).all()
        assert np.max(np.abs(got_w - ref_w)) <= tol * np.max(np.abs(ref_w)), call
        assert np.max(np.abs(got_b - ref_b)) <= tol * np.max(np.abs(ref_b)), call
        # and the oracle's definition of the same gradient, on the values both GPU paths were given
        ow, ob = oracle_wgrad(x, dy, bf16)
        assert np.max(np.abs(got_w - ow)) <= tol * np.max(np.abs(ow)), call
        assert np.max(np.abs(got_b - ob)) <= tol * np.max(np.abs(ob)), call
    m.close()


def oracle_wgrad(x, dy, bf16):
    from oracle import splitbrain_oracle as so
    if bf16:
        x, dy = so.round_bf16(x), so.round_bf16(dy)
    return so.Prims("float").conv_wgrad(x, dy)


@pytest.mark.parametrize("cin,cout,shape", [(1, 40, (3, 7, 9)), (4, 24, (5, 6, 10)), (3, 64, (2, 13, 11))])
@pytest.mark.parametrize("bf16", [False, True])
def test_static_scratch_wgrad_matches_oracle_and_allocates_nothing(cin, cout, shape, bf16):
    """Other channel counts and pixel counts that are not multiples of the 64-pixel chunk (189, 300, 286 pixels),
    against the oracle; and the point of the entry point: a call leaves the device's free memory where it was."""
    import torch
    from paper_2112_15317_b200 import binding as sb
    B, H, W = shape
    rng = np.random.default_rng(100 * cin + cout)
    x = rng.standard_normal((B, H, W, cin)).astype(np.float32)
    dy = rng.standard_normal((B, H, W, cout)).astype(np.float32)
    tdt = torch.bfloat16 if bf16 else torch.float32
    xt, dyt = torch.from_numpy(x).cuda().to(tdt), torch.from_numpy(dy).cuda().to(tdt)
    dw = torch.full((cout, 3, 3, cin), float("nan"), dtype=torch.float32, device="cuda")
    db = torch.full((cout,), float("nan"), dtype=torch.float32, device="cuda")
    prec = sb.SB_BF16 if bf16 else sb.SB_FP32
    sb.conv_in_wgrad_static(xt, dyt, dw, db, prec)        # (a first call on a device also looks up the scratch address)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    dw.fill_(float("nan")); db.fill_(float("nan"))
    sb.conv_in_wgrad_static(xt, dyt, dw, db, prec)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    ow, ob = oracle_wgrad(x, dy, bf16)
    tol = 1e-2 if bf16 else 1e-4
    assert np.max(np.abs(dw.cpu().numpy() - ow)) <= tol * np.max(np.abs(ow))
    assert np.max(np.abs(db.cpu().numpy() - ob)) <= tol * np.max(np.abs(ob))


def test_static_scratch_rejects_sizes_beyond_its_limit():
    import torch
    from paper_2112_15317_b200 import binding as sb
    x = torch.zeros((1, 4, 4, 3), device="cuda")
    dy = torch.zeros((1, 4, 4, 256), device="cuda")
    dw = torch.zeros((256, 3, 3, 3), device="cuda")
    db = torch.zeros((256,), device="cuda")
    with pytest.raises(sb.SBError) as e:
        sb.conv_in_wgrad_static(x, dy, dw, db, sb.SB_FP32)       # 256*28 = 7168 floats > 4096
    assert e.value.status == 3 and "scratch limit" in str(e.value)
    x5 = torch.zeros((1, 4, 4, 5), device="cuda")
    with pytest.raises(sb.SBError):
        sb.conv_in_wgrad_static(x5, dy[..., :8].contiguous(), dw, db, sb.SB_FP32)   # Cin = 5 unsupported
