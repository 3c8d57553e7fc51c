"""The MP group as separate worker processes on CPU (torch.distributed, gloo; world sizes 2 and 4).

Worker i is data replica i and model shard i (the paper's arrangement: Modulo Layer / Shard Layer paragraphs).  Every
worker computes with the oracle's layer primitives on its OWN rows and its OWN column shard only, and moves data
exclusively as sb_exchange_plan says: each message of the plan becomes one send / receive of exactly that block.  The
result -- loss, every conv gradient after the replicas' reduce, every worker's FC shard gradients -- must equal the
single-process oracle's partitioned iteration bit for bit (same primitives, same summation orders: shard sums and
replica sums in worker order).  A wrong block anywhere in the plan (rows of another worker, a neighbour's column
slice, a missing message) changes the result.

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


def run_worker(rank, G, port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    os.environ["OMP_NUM_THREADS"] = "2"
    dist.init_process_group("gloo", rank=rank, world_size=G)
    import sb_inputs as si
    from oracle import splitbrain_oracle as so
    from paper_2112_15317_b200 import binding as sb

    b = 3
    wl = si.Workload("mp_group", net(), 8, 8, 3, b, G, G)
    B = wl.B
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    P = so.Prims("float")
    plan = sb.exchange_plan(wl.layers, wl.H, wl.W, wl.C, b, G)
    groups = {}
    for m in plan:
        groups.setdefault((m["kind"], m["layer"]), []).append(m)
    first_fc = next(i for i, (k, _) in enumerate(wl.layers) if k in (si.FC_RELU, si.FC))
    nl = len(wl.layers)
    me = rank
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
    # modulo layer: the gathered [B, D] matrix; my rows are mine, the others arrive as the plan says
    X = np.zeros((B, D), np.float32)
    X[me * b:(me + 1) * b] = a.reshape(b, D)
    for m, buf in exchange(groups[(sb.SB_X_GATHER_ROWS, first_fc)], me, lambda m, send: X[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]]):
        X[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]] = buf.numpy()
    labels = y.astype(np.int32)                       # every worker evaluates the loss on all B rows (labels travel with the rows)
    fc_in, fc_out_mine, shard = {}, {}, {}
    for li in range(first_fc, nl - 1):
        kind, out = wl.layers[li]
        cb = si.shard_bounds(out, G)
        shard[li] = (cb[me], cb[me + 1])
        W_me, b_me = params[li]["w"][cb[me]:cb[me + 1]], params[li]["b"][cb[me]:cb[me + 1]]
        fc_in[li] = X
        Y_me = P.fc_fwd(X, W_me, b_me, relu=(kind == si.FC_RELU))
        fc_out_mine[li] = Y_me
        # shard layer: the full-width matrix from the K column slices
        Y = np.zeros((B, out), np.float32)
        Y[:, cb[me]:cb[me + 1]] = Y_me
        for m, buf in exchange(groups[(sb.SB_X_GATHER_COLS, li)], me, lambda m, send: Y[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]]):
            Y[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]] = buf.numpy()
        X = Y
    row_loss, dZ = P.softmax_xent(X, labels, 1.0 / B)
    loss = np.float32(np.sum(row_loss, dtype=np.float32) / np.float32(B))
    # ---- backward ----------------------------------------------------------------------------------
    fc_grads = {}
    dY_me = np.ascontiguousarray(dZ[:, shard[nl - 2][0]:shard[nl - 2][1]])
    for li in range(nl - 2, first_fc - 1, -1):
        out = wl.layers[li][1]
        cb = si.shard_bounds(out, G)
        W_me = params[li]["w"][cb[me]:cb[me + 1]]
        dW, db, dX_part = P.fc_bwd(fc_in[li], W_me, dY_me)            # full-width partial input gradient
        fc_grads[li] = (dW, db)
        if li > first_fc:
            # shard layer backward: my column slice of every worker's partial gradient, summed in worker order
            lo, hi = shard[li - 1]
            parts = {me: dX_part[:, lo:hi]}
            for m, buf in exchange(groups[(sb.SB_X_REDUCE_COLS, li - 1)], me, lambda m, send: dX_part[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]] if send else np.empty((m["rows"][1] - m["rows"][0], m["cols"][1] - m["cols"][0]), np.float32)):
                assert m["cols"] == (lo, hi)
                parts[m["src"]] = buf.numpy()
            dX = np.zeros((B, hi - lo), np.float32)
            for j in range(G):
                dX = dX + parts[j]
            dY_me = np.ascontiguousarray(dX * (fc_out_mine[li - 1] > 0))
        else:
            # modulo layer backward: my rows of every worker's partial gradient, summed in worker order
            parts = {me: dX_part[me * b:(me + 1) * b]}
            for m, buf in exchange(groups[(sb.SB_X_REDUCE_ROWS, first_fc)], me, lambda m, send: dX_part[m["rows"][0]:m["rows"][1], m["cols"][0]:m["cols"][1]] if send else np.empty((m["rows"][1] - m["rows"][0], m["cols"][1] - m["cols"][0]), np.float32)):
                assert m["rows"] == (me * b, (me + 1) * b)
                parts[m["src"]] = buf.numpy()
            dfeat = np.zeros((b, D), np.float32)
            for j in range(G):
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
    # the replicas' reduce: exactly the layers the plan lists, summed in worker order
    reduced = {}
    for m in plan:
        if m["kind"] == sb.SB_X_ALLREDUCE:
            li = m["layer"]
            for k, g in enumerate(conv_grads[li]):
                mine = torch.from_numpy(np.ascontiguousarray(g, dtype=np.float32))
                got = [torch.empty_like(mine) for _ in range(G)]
                dist.all_gather(got, mine)
                acc = np.zeros_like(g)
                for j in range(G):
                    acc = acc + got[j].numpy()
                reduced[(li, k)] = acc
    q.put((rank, float(loss), {k: v.copy() for k, v in reduced.items()}, {li: (g[0].copy(), g[1].copy()) for li, g in fc_grads.items()}))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("G", [2, 4])
def test_mp_group_workers_driven_by_the_exchange_plan_match_the_oracle(G):
    sys.path.insert(0, ROOT)
    import __graft_entry__ as ge
    ge.build()
    import sb_inputs as si
    from oracle import splitbrain_oracle as so
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 23000 + (os.getpid() * 7 + G) % 4000
    procs = [ctx.Process(target=run_worker, args=(r, G, port, q)) for r in range(G)]
    for p in procs:
        p.start()
    res = {}
    for _ in procs:
        rank, loss, conv, fc = q.get(timeout=300)
        res[rank] = (loss, conv, fc)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the single-process oracle: R = K = G logical partitions
    wl = si.Workload("mp_group", net(), 8, 8, 3, 3, G, G)
    params = si.make_params(wl, bias_std=0.2)
    x, y = si.make_batch(wl)
    om = so.from_workload(wl, real="float")
    om.load_params(params)
    loss = float(om.forward(si.split_replicas(x, G), si.split_replicas(y, G)))
    om.backward()
    for rank in range(G):
        wloss, conv, fc = res[rank]
        assert wloss == loss
        for (li, k), g in conv.items():
            assert np.array_equal(g, om.grads[li]["w" if k == 0 else "b"]), (rank, li, k)
        assert sorted({li for li, _ in conv}) == [li for li, (kind, _) in enumerate(wl.layers) if kind == si.CONV3X3_RELU]
        for li, (dW, db) in fc.items():
            assert np.array_equal(dW, om.grads[li][rank]["w"]) and np.array_equal(db, om.grads[li][rank]["b"]), (rank, li)
