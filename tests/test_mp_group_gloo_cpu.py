"""MP groups as separate worker processes on CPU (torch.distributed, gloo; 2 and 4 workers, group sizes 1, 2 and 4).

Worker p is data replica p, belongs to group p // mp and holds model shard p % mp of that group (Modulo Layer / Shard
Layer paragraphs; Group MP Extension).  Every worker computes with the oracle's layer primitives on its OWN rows and
its OWN column shard only, and moves data exclusively as sb_exchange_plan says: each message of the plan becomes one
send / receive of exactly that block, each reduce entry one reduction over exactly the workers it names.  With one
group the result -- loss, every conv gradient after the replicas' reduce, every worker's FC shard gradients -- must
equal the single-process oracle's partitioned iteration (R = N, K = mp) bit for bit (same primitives, same summation
orders: shard sums and replica sums in worker order).  With several groups the forward pass, the loss terms and the
conv gradients are still bit-identical; an FC shard gradient is now the sum over the groups of per-group products and
equals the oracle's single product over all rows up to float summation order.  A wrong block anywhere in the plan
(rows of another worker or group, a neighbour's column slice, a missing message, a reduce over the wrong workers)
changes the result.

No GPU is involved: this is the host-side proof of the multi-GPU MP group's exchange schedule."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def net():
    import sb_inputs as si
    # conv-side stack, three FC layers with widths that K = 4 does not divide (10 columns -> 2, 3, 2, 3)
    return [(si.CONV3X3_RELU, 8), (si.MAXPOOL2, 0), (si.CONV3X3_RELU, 12), (si.MAXPOOL2, 0),
            (si.FC_RELU, 30), (si.FC_RELU, 22), (si.FC, 10), (si.SOFTMAX_XENT, 10)]


def exchange(group, me, mats):
    """Carry out one group of plan messages.  mats(m) -> the numpy block view that message m sends FROM (on the source)
    or receives INTO (on the destination); receives are posted first, then the sends."""
    reqs, landing = [], []
    for m in group:
        if m["dst"] == me:
            buf = torch.empty(mats(m, False).shape, dtype=torch.float32)
            reqs.append(dist.irecv(buf, src=m["src"]))
            landing.append((m, buf))
    for m in group:
        if m["src"] == me:
            reqs.append(dist.isend(torch.from_numpy(np.ascontiguousarray(mats(m, True), dtype=np.float32)), dst=m["dst"]))
    for r in reqs:
        r.wait()
    return landing


def run_worker(rank, N, mp_, port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ["OMP_NUM_THREADS"] = "2"
    dist.init_process_group("gloo", rank=rank, world_size=N)
    import sb_inputs as si
    from oracle import splitbrain_oracle as so
    from paper_2112_15317_b200 import binding as sb

    b = 3
    wl = si.Workload("mp_group", net(), 8, 8, 3, b, N, mp_)
    B = wl.B                                          # rows of the whole batch
    G = N // mp_
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    P = so.Prims("float")
    plan = sb.exchange_plan(wl.layers, wl.H, wl.W, wl.C, b, N, mp_)
    groups = {}
    for m in plan:
        groups.setdefault((m["kind"], m["layer"]), []).append(m)
    # one process group per intra-group offset (created by every worker, in the same order)
    peers = {o: dist.new_group(ranks=[g * mp_ + o for g in range(G)]) for o in range(mp_)} if G > 1 else {}
    first_fc = next(i for i, (k, _) in enumerate(wl.layers) if k in (si.FC_RELU, si.FC))
    nl = len(wl.layers)
    me, gid, off = rank, rank // mp_, rank % mp_
    g0, g1 = gid * mp_ * b, (gid + 1) * mp_ * b       # my group's rows of the whole batch
    Bg = g1 - g0
    # ---- forward: my replica's conv stack on my b images ---------------------------------------
    a = np.ascontiguousarray(x[me * b:(me + 1) * b])
    conv_in, conv_out, idx = {}, {}, {}
    for li in range(first_fc):
        conv_in[li] = a
        if wl.layers[li][0] == si.CONV3X3_RELU:
            a = P.conv_fwd(a, params[li]["w"], params[li]["b"], relu=True)
        else:
            a, idx[li] = P.pool_fwd(a)
        conv_out[li] = a
    feat_shape = a.shape
    D = int(np.prod(feat_shape[1:]))
    # every matrix below is indexed by rows of the WHOLE batch, as the plan's messages are; a worker only ever touches
    # the rows of its own group
    X = np.zeros((B, D), np.float32)
    X[me * b:(me + 1) * b] = a.reshape(b, D)
    blk = lambda M, m: M[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]]
    if mp_ > 1:
        # modulo layer: my rows are mine, the others of my group arrive as the plan says
        for m, buf in exchange(groups[(sb.SB_X_GATHER_ROWS, first_fc)], me, lambda m, send: blk(X, m)):
            assert g0 <= m["rows"][0] and m["rows"][1] <= g1
            X[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]] = buf.numpy()
    else:
        assert not any(k in (sb.SB_X_GATHER_ROWS, sb.SB_X_GATHER_COLS, sb.SB_X_REDUCE_COLS, sb.SB_X_REDUCE_ROWS) for k, _ in groups)
    X = X[g0:g1] if mp_ > 1 else X[me * b:(me + 1) * b]          # the rows this worker's FC layers see
    r0 = g0 if mp_ > 1 else me * b                                  # whole-batch index of local row 0
    rows = X.shape[0]
    labels = y.astype(np.int32)[r0:r0 + rows]
    fc_in, fc_out_mine, shard = {}, {}, {}
    for li in range(first_fc, nl - 1):
        kind, out = wl.layers[li]
        cb = si.shard_bounds(out, mp_)
        shard[li] = (cb[off], cb[off + 1])
        W_me, b_me = params[li]["w"][cb[off]:cb[off + 1]], params[li]["b"][cb[off]:cb[off + 1]]
        fc_in[li] = X
        Y_me = P.fc_fwd(X, W_me, b_me, relu=(kind == si.FC_RELU))
        fc_out_mine[li] = Y_me
        # shard layer: the full-width matrix from the group's column slices
        Yw = np.zeros((B, out), np.float32)
        Yw[r0:r0 + rows, cb[off]:cb[off + 1]] = Y_me
        if mp_ > 1:
            for m, buf in exchange(groups[(sb.SB_X_GATHER_COLS, li)], me, lambda m, send: blk(Yw, m)):
                assert m["rows"] == (g0, g1)
                Yw[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]] = buf.numpy()
        X = np.ascontiguousarray(Yw[r0:r0 + rows])
    row_loss, dZ = P.softmax_xent(X, labels, 1.0 / B)                 # the loss is the mean over the whole batch
    # ---- backward ----------------------------------------------------------------------------------
    fc_grads = {}
    dY_me = np.ascontiguousarray(dZ[:, shard[nl - 2][0]:shard[nl - 2][1]])
    for li in range(nl - 2, first_fc - 1, -1):
        out = wl.layers[li][1]
        cb = si.shard_bounds(out, mp_)
        W_me = params[li]["w"][cb[off]:cb[off + 1]]
        dW, db, dX_part = P.fc_bwd(fc_in[li], W_me, dY_me)            # full-width partial input gradient
        fc_grads[li] = [dW, db]
        full = np.zeros((B, dX_part.shape[1]), np.float32)
        full[r0:r0 + rows] = dX_part
        recv_shape = lambda m: np.empty((m["rows"][1] - m["rows"][0], m["cols"][1] - m["cols"][0]), np.float32)
        if li > first_fc:
            # shard layer backward: my column slice of every group member's partial gradient, summed in worker order
            lo, hi = shard[li - 1]
            parts = {me: dX_part[:, lo:hi]}
            if mp_ > 1:
                for m, buf in exchange(groups[(sb.SB_X_REDUCE_COLS, li - 1)], me, lambda m, send: blk(full, m) if send else recv_shape(m)):
                    assert m["cols"] == (lo, hi) and m["rows"] == (g0, g1)
                    parts[m["src"]] = buf.numpy()
            dX = np.zeros((rows, hi - lo), np.float32)
            for j in range(gid * mp_, (gid + 1) * mp_):
                dX = dX + parts[j]
            dY_me = np.ascontiguousarray(dX * (fc_out_mine[li - 1] > 0))
        else:
            # modulo layer backward: my rows of every group member's partial gradient, summed in worker order
            parts = {me: full[me * b:(me + 1) * b]}
            if mp_ > 1:
                for m, buf in exchange(groups[(sb.SB_X_REDUCE_ROWS, first_fc)], me, lambda m, send: blk(full, m) if send else recv_shape(m)):
                    assert m["rows"] == (me * b, (me + 1) * b)
                    parts[m["src"]] = buf.numpy()
            dfeat = np.zeros((b, D), np.float32)
            for j in range(gid * mp_, (gid + 1) * mp_):
                dfeat = dfeat + parts[j]
    d = dfeat.reshape((b,) + feat_shape[1:])
    conv_grads = {}
    for li in range(first_fc - 1, -1, -1):
        if wl.layers[li][0] == si.MAXPOOL2:
            d = P.pool_bwd(d, idx[li])
        else:
            d = d * (conv_out[li] > 0)
            conv_grads[li] = P.conv_wgrad(conv_in[li], d)
            if li > 0:
                d = P.conv_dgrad(d, params[li]["w"])

    def summed(t, group, n):
        mine = torch.from_numpy(np.ascontiguousarray(t, dtype=np.float32))
        got = [torch.empty_like(mine) for _ in range(n)]
        dist.all_gather(got, mine, group=group)
        acc = np.zeros_like(t)
        for j in range(n):
            acc = acc + got[j].numpy()
        return acc

    # the parameter reduces: exactly the layers, shards and workers the plan lists, summed in worker / group order
    reduced = {}
    group_reduced = set()
    for m in plan:
        li = m["layer"]
        if m["kind"] == sb.SB_X_ALLREDUCE:
            grads = conv_grads[li] if li in conv_grads else fc_grads[li]      # (pure DP: the FC layers are whole and reduced like the convs)
            for k, g in enumerate(grads):
                reduced[(li, k)] = summed(g, None, N)
        elif m["kind"] == sb.SB_X_ALLREDUCE_GROUPS and m["src"] == off:
            assert m["cols"] == shard[li]
            fc_grads[li] = [summed(g, peers[off], G) for g in fc_grads[li]]
            group_reduced.add(li)
    assert G == 1 or mp_ == 1 or group_reduced == set(fc_grads)
    q.put((rank, float(np.sum(row_loss, dtype=np.float64)), {k: v.copy() for k, v in reduced.items()},
           {li: (g[0].copy(), g[1].copy()) for li, g in fc_grads.items()}))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("N,mp_", [(2, 2), (4, 4), (4, 2), (4, 1)])
def test_mp_group_workers_driven_by_the_exchange_plan_match_the_oracle(N, mp_):
    sys.path.insert(0, ROOT)
    import __graft_entry__ as ge
    ge.build()
    import sb_inputs as si
    from oracle import splitbrain_oracle as so
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 23000 + (os.getpid() * 7 + N * 5 + mp_) % 4000
    procs = [ctx.Process(target=run_worker, args=(r, N, mp_, port, q)) for r in range(N)]
    for p in procs:
        p.start()
    res = {}
    for _ in procs:
        rank, loss_sum, conv, fc = q.get(timeout=300)
        res[rank] = (loss_sum, conv, fc)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the single-process oracle: R = N logical replicas, K = mp logical shards
    G = N // mp_
    wl = si.Workload("mp_group", net(), 8, 8, 3, 3, N, mp_)
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    om = so.from_workload(wl, real="float")
    om.load_params(params)
    loss = float(om.forward(si.split_replicas(x, N), si.split_replicas(y, N)))
    om.backward()
    # the loss: every group (every worker under pure DP) contributes the sum over its own rows
    owners = [g * mp_ for g in range(G)] if mp_ > 1 else list(range(N))
    assert sum(res[r][0] for r in owners) / wl.B == pytest.approx(loss, rel=1e-6)
    for r in range(N):
        assert res[r][0] == res[(r // mp_) * mp_][0] or mp_ == 1          # the workers of a group evaluate the same loss terms
    conv_layers = [li for li, (kind, _) in enumerate(wl.layers) if kind == si.CONV3X3_RELU]
    exact = G == 1                                                          # one group: same summation order as the oracle
    for rank in range(N):
        _, conv, fc = res[rank]
        off = rank % mp_
        for li in conv_layers:
            for k in (0, 1):
                assert np.array_equal(conv[(li, k)], om.grads[li]["w" if k == 0 else "b"]), (rank, li, k)
        assert sorted({li for li, _ in conv if li in conv_layers}) == conv_layers
        for li, (dW, db) in fc.items():
            ref_w, ref_b = om.grads[li][off]["w"], om.grads[li][off]["b"]
            if mp_ == 1:
                dW, db = conv[(li, 0)], conv[(li, 1)]                       # pure DP: reduced over all workers like the convs
            if exact:
                assert np.array_equal(dW, ref_w) and np.array_equal(db, ref_b), (rank, li)
            else:
                assert np.max(np.abs(dW - ref_w)) <= 2e-6 * np.max(np.abs(ref_w)), (rank, li)
                assert np.max(np.abs(db - ref_b)) <= 2e-6 * np.max(np.abs(ref_b)), (rank, li)
