"""Host-side partitioning table (sb_partition) and MP-group exchange schedule (sb_exchange_plan), through the C ABI,
without a GPU.  Pins: the node sequence of the paper's transformed-CNN figure (tests/golden), the Table 1 network's
layer widths, shard sizes that add up, the paper's "local 1/K, remote (K-1)/K" split of every gathered matrix, and
the rule that conv-side layers refuse a partitioned input."""
import os

import pytest

import sb_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def binding():
    import __graft_entry__ as ge
    ge.build()
    from paper_2112_15317_b200 import binding as b
    return b


def tokens(b, nodes, layers, K):
    out = []
    for nd in nodes:
        if nd["node"] == b.SB_NODE_MODULO:
            out.append("M")
        elif nd["node"] == b.SB_NODE_SHARD:
            out.append("S")
        else:
            kind = layers[nd["layer"]][0]
            if kind in (si.CONV3X3_RELU, si.MAXPOOL2):
                if not out or out[-1] != "C*":
                    out.append("C*")
            elif kind == si.SOFTMAX_XENT:
                out.append("L")
            else:
                out.append("F/K" if nd["shards"] == K and K > 1 else "F")
    return " ".join(out)


def golden_sequence():
    for line in open(os.path.join(ROOT, "tests", "golden", "partition_transformed_cnn.txt")):
        if line.strip() and not line.startswith("#"):
            return line.strip()


@pytest.mark.parametrize("K", [2, 4, 8])
def test_table1_network_transforms_as_in_the_papers_figure(K):
    b = binding()
    wl = si.config(5)                       # Table 1: 7 conv + 3 FC layers on 32x32x3 images
    nodes = b.partition(wl.layers, 32, 32, 3, K)
    assert tokens(b, nodes, wl.layers, K) == golden_sequence()
    # widths: FC0 takes 256*4*4 = 4096 features (Table 1), every FC is split to 1/K size
    fc = [nd for nd in nodes if nd["node"] == b.SB_NODE_LAYER and wl.layers[nd["layer"]][0] in (si.FC_RELU, si.FC)]
    assert [nd["dimF"] for nd in fc] == [1024, 1024, 10]
    assert [nd["dim"] for nd in fc] == [1024 // K, 1024 // K, -(-10 // K)]
    modulo = [nd for nd in nodes if nd["node"] == b.SB_NODE_MODULO]
    assert len(modulo) == 1 and modulo[0]["dimF"] == 4096 and wl.layers[modulo[0]["layer"]][0] == si.FC_RELU
    # every input layer appears exactly once, in order
    assert [nd["layer"] for nd in nodes if nd["node"] == b.SB_NODE_LAYER] == list(range(len(wl.layers)))


def test_cfg0_and_unpartitioned_network():
    b = binding()
    wl = si.config(0)
    assert tokens(b, b.partition(wl.layers, 32, 32, 3, 2), wl.layers, 2) == "C* M F/K S F/K S L"
    # K = 1: nothing is inserted, nothing is split
    nodes = b.partition(wl.layers, 32, 32, 3, 1)
    assert all(nd["node"] == b.SB_NODE_LAYER and nd["shards"] == 1 and nd["dim"] == nd["dimF"] for nd in nodes)


def test_layers_kept_whole_follow_the_listing():
    """A layer marked whole (the CCR test's outcome) is not split: no modulo layer in front of it while the input is
    whole; a shard layer in front of it when the layer below was split; the modulo layer goes in front of the FIRST
    split layer only."""
    b = binding()
    conv = [(si.CONV3X3_RELU, 8), (si.MAXPOOL2, 0)]
    net = conv + [(si.FC_RELU_WHOLE, 32), (si.FC_RELU, 64), (si.FC_RELU_WHOLE, 48), (si.FC, 10), (si.SOFTMAX_XENT, 10)]
    nodes = b.partition(net, 8, 8, 3, 4)
    assert tokens(b, nodes, net, 4) == "C* F M F/K S F F/K S L"
    # all-whole FC stack: plain data parallelism, nothing inserted
    net2 = conv + [(si.FC_RELU_WHOLE, 32), (si.FC_WHOLE, 10), (si.SOFTMAX_XENT, 10)]
    assert tokens(b, b.partition(net2, 8, 8, 3, 4), net2, 4) == "C* F F L"


def test_dropout_follows_the_partitioned_width_without_communication_nodes():
    """Listing 1, case DROPOUT | RELU: a one-to-one functional layer takes the width the layer below left (1/K of it
    behind a split layer), passes dim and dimF on unchanged, and gets neither a modulo nor a shard node in front of it;
    the shard node goes in front of the next layer that needs the full width."""
    b = binding()
    conv = [(si.CONV3X3_RELU, 8), (si.MAXPOOL2, 0)]
    net = conv + [(si.FC_RELU, 32), (si.DROPOUT, 16384), (si.FC_RELU_WHOLE, 24), (si.DROPOUT, 100), (si.FC, 10), (si.SOFTMAX_XENT, 10)]
    nodes = b.partition(net, 8, 8, 3, 4)
    seq = [(nd["node"], nd["layer"], nd["shards"], nd["dim"], nd["dimF"]) for nd in nodes]
    L, M, S = b.SB_NODE_LAYER, b.SB_NODE_MODULO, b.SB_NODE_SHARD
    assert seq == [(L, 0, 1, 512, 512), (L, 1, 1, 128, 128),
                   (M, 2, 4, 128, 128), (L, 2, 4, 8, 32), (L, 3, 4, 8, 32),          # dropout on the 1/K slice
                   (S, 4, 4, 32, 32), (L, 4, 1, 24, 24), (L, 5, 1, 24, 24),          # whole layer, dropout on the whole width
                   (L, 6, 4, 3, 10), (S, 7, 4, 10, 10), (L, 7, 1, 10, 10)]
    # the exchange schedule gathers the dropout layer's column slices (layer 3), not the FC layer's below it
    msgs = b.exchange_plan(net, 8, 8, 3, 2, 4)
    gathers = {m["layer"] for m in msgs if m["kind"] == b.SB_X_GATHER_COLS}
    assert gathers == {3, 6}
    with pytest.raises(b.SBError, match="must follow an FC"):
        b.partition(conv + [(si.DROPOUT, 100), (si.FC, 4), (si.SOFTMAX_XENT, 4)], 8, 8, 3, 2)
    with pytest.raises(b.SBError, match="drop probability"):
        b.partition(conv + [(si.FC_RELU, 8), (si.DROPOUT, 0), (si.FC, 4), (si.SOFTMAX_XENT, 4)], 8, 8, 3, 2)


def test_conv_side_layers_refuse_a_partitioned_input_and_bad_lists_are_rejected():
    b = binding()
    with pytest.raises(b.SBError):
        b.partition([(si.FC_RELU, 16), (si.CONV3X3_RELU, 8), (si.FC, 4), (si.SOFTMAX_XENT, 4)], 4, 4, 3, 2)
    with pytest.raises(b.SBError, match="exceeds the FC width"):
        b.partition([(si.FC_RELU, 16), (si.FC, 3), (si.SOFTMAX_XENT, 3)], 4, 4, 3, 4)
    with pytest.raises(b.SBError, match="unknown kind"):
        b.partition([(99, 16)], 4, 4, 3, 2)


@pytest.mark.parametrize("G,b_", [(2, 4), (4, 32), (8, 3)])
def test_exchange_plan_blocks_tile_every_matrix(G, b_):
    """Every gathered matrix is covered exactly once by the owner's block plus the G - 1 blocks that arrive: each
    worker holds 1/K of it locally and receives (K-1)/K from the others (Shard Layer paragraph); the backward blocks
    mirror the forward ones (what was gathered from a worker is what goes back to it)."""
    bnd = binding()
    wl = si.config(5)
    msgs = bnd.exchange_plan(wl.layers, 32, 32, 3, b_, G)
    B = G * b_
    groups = {}
    for m in msgs:
        groups.setdefault((m["kind"], m["layer"], m["backward"]), []).append(m)
    order = [k for k in dict.fromkeys((m["kind"], m["layer"], m["backward"]) for m in msgs)]
    fc = [li for li, (k, _) in enumerate(wl.layers) if k in (si.FC_RELU, si.FC)]
    conv = [li for li, (k, _) in enumerate(wl.layers) if k == si.CONV3X3_RELU]
    # execution order: modulo gather, a column gather after every FC layer; then the mirror image, then (interleaved with
    # it, in backward layer order) the conv-stack parameter reduces
    assert order[:4] == [(bnd.SB_X_GATHER_ROWS, fc[0], 0)] + [(bnd.SB_X_GATHER_COLS, li, 0) for li in fc]
    assert order[4:7] == [(bnd.SB_X_REDUCE_COLS, fc[1], 1), (bnd.SB_X_REDUCE_COLS, fc[0], 1), (bnd.SB_X_REDUCE_ROWS, fc[0], 1)]
    assert order[7:] == [(bnd.SB_X_ALLREDUCE, li, 1) for li in reversed(conv)]
    for (kind, li, bw), ms in groups.items():
        if kind == bnd.SB_X_ALLREDUCE:
            continue
        assert len(ms) == G * (G - 1)
        width = ms[0]["width"]
        for dst in range(G):
            got = [m for m in ms if m["dst"] == dst]
            assert sorted(m["src"] for m in got) == [s for s in range(G) if s != dst]
            if kind == bnd.SB_X_GATHER_ROWS:
                cover = sorted([m["rows"] for m in got] + [(dst * b_, (dst + 1) * b_)])
                assert cover == [(s * b_, (s + 1) * b_) for s in range(G)] and all(m["cols"] == (0, width) for m in got)
                assert all(m["rows"] == (m["src"] * b_, (m["src"] + 1) * b_) for m in got)          # the owner of row g is g // b
            elif kind == bnd.SB_X_GATHER_COLS:
                cb = si.shard_bounds(width, G)
                assert all(m["cols"] == (cb[m["src"]], cb[m["src"] + 1]) and m["rows"] == (0, B) for m in got)
                remote = sum(m["cols"][1] - m["cols"][0] for m in got)
                assert remote + cb[dst + 1] - cb[dst] == width                                       # local 1/K + remote (K-1)/K
            elif kind == bnd.SB_X_REDUCE_COLS:
                cb = si.shard_bounds(width, G)
                assert all(m["cols"] == (cb[dst], cb[dst + 1]) and m["rows"] == (0, B) for m in got)  # every sender's copy of MY slice
            else:
                assert all(m["rows"] == (dst * b_, (dst + 1) * b_) and m["cols"] == (0, width) for m in got)
    with pytest.raises(bnd.SBError, match="multiple of K"):
        arr = bnd._layers_array(wl.layers)
        import ctypes
        cfg = bnd.sb_config(32, 32, 3, 4, 2, 4, 0, 0)
        n = ctypes.c_int32()
        st = bnd.sb_exchange_plan(arr, len(wl.layers), ctypes.byref(cfg), None, 0, ctypes.byref(n))
        raise bnd.SBError(st, bnd._lib.sb_partition_last_error().decode())


@pytest.mark.parametrize("N,mp_,b_", [(4, 2, 3), (8, 2, 4), (8, 4, 2), (6, 3, 5)])
def test_exchange_plan_with_several_mp_groups(N, mp_, b_):
    """Group MP Extension: N workers in N / mp groups.  Worker p belongs to group p // mp at offset p % mp; the modulo
    and shard layers' blocks stay inside a group and cover that group's rows only; the conv stack is reduced over all N
    workers, every FC shard over the workers at the same offset of all groups."""
    bnd = binding()
    wl = si.config(5)
    msgs = bnd.exchange_plan(wl.layers, 32, 32, 3, b_, N, mp_)
    G = N // mp_
    fc = [li for li, (k, _) in enumerate(wl.layers) if k in (si.FC_RELU, si.FC)]
    conv = [li for li, (k, _) in enumerate(wl.layers) if k == si.CONV3X3_RELU]
    p2p = [m for m in msgs if m["kind"] in (bnd.SB_X_GATHER_ROWS, bnd.SB_X_GATHER_COLS, bnd.SB_X_REDUCE_COLS, bnd.SB_X_REDUCE_ROWS)]
    assert all(m["src"] // mp_ == m["dst"] // mp_ and m["src"] != m["dst"] for m in p2p)          # nothing crosses a group
    for m in p2p:
        gid = m["dst"] // mp_
        g0, g1 = gid * mp_ * b_, (gid + 1) * mp_ * b_
        if m["kind"] == bnd.SB_X_GATHER_ROWS:
            assert m["rows"] == (m["src"] * b_, (m["src"] + 1) * b_) and g0 <= m["rows"][0] < g1  # owner of row g: worker g // b
        elif m["kind"] == bnd.SB_X_REDUCE_ROWS:
            assert m["rows"] == (m["dst"] * b_, (m["dst"] + 1) * b_)
        else:
            cb = si.shard_bounds(m["width"], mp_)
            who = m["src"] if m["kind"] == bnd.SB_X_GATHER_COLS else m["dst"]
            assert m["rows"] == (g0, g1) and m["cols"] == (cb[who % mp_], cb[who % mp_ + 1])
    for kind, layers_ in [(bnd.SB_X_GATHER_ROWS, fc[:1]), (bnd.SB_X_REDUCE_ROWS, fc[:1]), (bnd.SB_X_GATHER_COLS, fc), (bnd.SB_X_REDUCE_COLS, fc[:-1])]:
        for li in layers_:
            assert len([m for m in p2p if m["kind"] == kind and m["layer"] == li]) == G * mp_ * (mp_ - 1)
    # one group's traffic does not grow with the number of groups (the point of the extension): per worker, the modulo
    # and shard layers receive (mp - 1) / mp of each matrix whatever N is
    one = bnd.exchange_plan(wl.layers, 32, 32, 3, b_, mp_, mp_)
    per_worker = lambda ms, w: sum((m["rows"][1] - m["rows"][0]) * (m["cols"][1] - m["cols"][0]) for m in ms if m["dst"] == w)
    assert per_worker(p2p, N - 1) == per_worker([m for m in one if m["dst"] >= 0], mp_ - 1)
    # parameter reduces
    assert [m["layer"] for m in msgs if m["kind"] == bnd.SB_X_ALLREDUCE] == list(reversed(conv))
    gr = [m for m in msgs if m["kind"] == bnd.SB_X_ALLREDUCE_GROUPS]
    assert [(m["layer"], m["src"]) for m in gr] == [(li, o) for li in reversed(fc) for o in range(mp_)]
    for m in gr:
        cb = si.shard_bounds(m["width"], mp_)
        assert m["cols"] == (cb[m["src"]], cb[m["src"] + 1]) and m["backward"] == 1
    # a single group has no such entry; K = 1 is pure data parallelism: nothing but reduces over all workers, FC layers included
    assert not [m for m in bnd.exchange_plan(wl.layers, 32, 32, 3, b_, mp_, mp_) if m["kind"] == bnd.SB_X_ALLREDUCE_GROUPS]
    dp = bnd.exchange_plan(wl.layers, 32, 32, 3, b_, N, 1)
    assert all(m["kind"] == bnd.SB_X_ALLREDUCE for m in dp) and [m["layer"] for m in dp] == list(reversed(sorted(conv + fc)))
