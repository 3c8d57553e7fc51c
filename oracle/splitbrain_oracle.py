"""CPU oracle for one SplitBrain hybrid-parallel training step.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this module; the
CUDA library never does, and the two share no code.

The oracle *carries out* the partitioned computation the paper describes, step by step, with
explicit loops over the R replicas and the K model shards and explicit copies for every
communication step, on top of the direct-loop layer primitives in sb_oracle.c:

  1. each replica r runs the convolution stack on its own b images           [Design: conv layers
     are replicated, data parallel]
  2. modulo layer, forward: the MP group gathers all replicas' feature rows; row g of the gathered
     matrix belongs to replica g // b (the paper's  remote = b / size  rule)  [Modulo Layer]
  3. each FC layer is split by output column into K shards of 1/K size; shard j computes its own
     columns (ReLU applied per shard, no exchange)                            [Layer Partitioning]
  4. shard layer, forward: the K column slices are concatenated into the full-width input of the
     next layer, and of the log-softmax                                       [Shard Layer]
  5. loss: log-softmax + NLL, mean over the full batch of R*b rows
  6. shard layer, backward: each shard's input gradient covers the full input width; they are
     summed over shards in order j = 0..K-1                                   [Shard Layer]
  7. modulo layer, backward: gradient rows go back to the replica that owns them [Modulo Layer]
  8. each replica back-propagates through its convolution stack; the replicas' weight gradients
     are summed in order r = 0..R-1 (synchronous DP reduce, period 1)
  9. SGD with momentum on every parameter.

Readings taken where the paper is silent (stated in full in the design notes): one synchronous
pass over all R*b rows instead of K sub-iterations with gradients divided by K; R and K are
independent; every FC layer is sharded with boundaries floor(j*out/K).

step_modulo() is the other schedule, the paper's own [Modulo Layer]: the FC stack runs K
sub-iterations on b/K examples of every replica and updates the FC parameters after each with
gradients divided by K; the conv stack back-propagates once, after the K-th.  It is not equal to the
unpartitioned step for K > 1, so its parity is against this algorithm only; it is pinned by K = 1
(identical to step()), by lr = 0 (gradients add up to the synchronous ones), by re-composition
out of forward()/backward() calls on the sub-batches, and by the paper's worked B = 2, K = 2 example.

`bf16=True` switches on the mixed-precision contract of the CUDA library: operands of every
contraction (stored activations, stored activation gradients, the weight copies used in the
contractions) are rounded to bfloat16 (round-to-nearest-even) at the points where the library
stores them; accumulators, bias add, ReLU, logits, loss, dW/db, master weights and momentum stay
in the working precision.

Dropout [Listing 1, case DROPOUT | RELU: a one-to-one functional layer that follows the partitioned width]:
each shard multiplies its own columns by a keep mask and by 1/(1 - p) (the reading taken: the expectation-
preserving form, so that nothing changes at evaluation time).  The mask bit of element (global batch row g,
logical column c) of dropout layer li in iteration t is drawn by the counter-based Philox-4x32-10 generator
(Salmon et al., "Parallel random numbers: as easy as 1, 2, 3", SC'11) at counter (e mod 2^32, e div 2^32, li, t),
e = g*width + c, key = the 64-bit seed: it depends on neither R nor K.  The element is kept iff the first output
word is >= p * 2^32, p given in units of 1/65536.

Parity pins: see tests/test_oracle_*.py (brute-force single-element evaluators, adjoint
identities, finite differences in double, closed forms, R/K invariance, a float64 autograd
re-computation of the unpartitioned network).  Unpinned: nothing in this file (group-MP mapping,
the CCR rule and the paper's "67 %" figure are not implemented).
"""
from __future__ import annotations

import ctypes
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
from oracle import build_oracle  # noqa: E402

CONV, POOL, FC_RELU, FC, LOSS = 1, 2, 3, 4, 5
DROPOUT = 8   # out = drop probability p in units of 1/65536 (1 .. 65535)

_libs = {}


def _lib(real: str):
    if real not in _libs:
        build_oracle.build()
        lib = ctypes.CDLL(build_oracle.lib_path(real))
        _libs[real] = lib
    return _libs[real]


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32/float64 values to the nearest bfloat16 (ties to even); result keeps a's dtype."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16) << 16
    out = r.astype(np.uint32).view(np.float32).reshape(a.shape)
    out = np.where(np.isfinite(f), out, f)
    return out.astype(a.dtype)


def shard_bounds(out: int, K: int):
    return [(j * out) // K for j in range(K + 1)]


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox-4x32 with 10 rounds (Salmon et al., SC'11, section 3.3 and table 2 constants): counter words c0..c3
    (uint32 arrays or scalars, broadcast together), key words k0, k1.  Returns the four output words as uint64
    arrays holding 32-bit values.  One round: with (hi0, lo0) = M0 * c0 and (hi1, lo1) = M1 * c2 as 64-bit
    products, the new counter is (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); the key is bumped by the Weyl
    constants (golden ratio, sqrt(3) - 1) between rounds."""
    M0, M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
    W0, W1 = 0x9E3779B9, 0xBB67AE85
    mask = np.uint64(0xFFFFFFFF)
    c0, c1, c2, c3 = (np.asarray(c, dtype=np.uint64) & mask for c in (c0, c1, c2, c3))
    k0, k1 = int(k0) & 0xFFFFFFFF, int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = M0 * c0            # < 2^64: exact in uint64
        p1 = M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c0, c1, c2, c3 = hi1 ^ c1 ^ np.uint64(k0), lo1, hi0 ^ c3 ^ np.uint64(k1), lo0
        k0 = (k0 + W0) & 0xFFFFFFFF
        k1 = (k1 + W1) & 0xFFFFFFFF
    return c0, c1, c2, c3


def dropout_keep(seed, step, layer, rows, width, units):
    """Keep mask [len(rows), width] of one dropout layer: element (global row g, column c) is kept iff the first
    Philox word at counter (e mod 2^32, e div 2^32, layer, step mod 2^32), e = g*width + c, under the key
    (seed mod 2^32, seed div 2^32) is >= units * 2^16, i.e. with probability 1 - units/65536."""
    assert 0 < units < 65536
    rows = np.asarray(rows, dtype=np.uint64)
    e = rows[:, None] * np.uint64(width) + np.arange(width, dtype=np.uint64)[None, :]
    x0, _, _, _ = philox4x32_10(e & np.uint64(0xFFFFFFFF), e >> np.uint64(32), layer, int(step) & 0xFFFFFFFF,
                                int(seed) & 0xFFFFFFFF, (int(seed) >> 32) & 0xFFFFFFFF)
    return x0 >= np.uint64(units << 16)


def dropout_scale(units):
    """1 / (1 - p) as one float32 division of exactly representable integers."""
    return np.float32(65536.0) / np.float32(65536 - units)


class Prims:
    """ctypes front-end of the C primitives for one precision ('float' or 'double')."""

    def __init__(self, real: str = "float"):
        self.real = real
        self.dt = np.float32 if real == "float" else np.float64
        self.lib = _lib(real)
        self.creal = ctypes.c_float if real == "float" else ctypes.c_double
        assert self.lib.orc_real_bytes() == np.dtype(self.dt).itemsize

    def _a(self, a):
        return np.ascontiguousarray(a, dtype=self.dt)

    def conv_fwd(self, x, w, bias, relu=True):
        x, w, bias = self._a(x), self._a(w), self._a(bias)
        N, H, W, Cin = x.shape
        Cout = w.shape[0]
        assert w.shape == (Cout, 3, 3, Cin)
        y = np.empty((N, H, W, Cout), self.dt)
        self.lib.orc_conv3x3_fwd(_p(x), _p(w), _p(bias), _p(y), N, H, W, Cin, Cout, int(relu))
        return y

    def conv_dgrad(self, dy, w):
        dy, w = self._a(dy), self._a(w)
        N, H, W, Cout = dy.shape
        Cin = w.shape[3]
        dx = np.empty((N, H, W, Cin), self.dt)
        self.lib.orc_conv3x3_dgrad(_p(dy), _p(w), _p(dx), N, H, W, Cin, Cout)
        return dx

    def conv_wgrad(self, x, dy):
        x, dy = self._a(x), self._a(dy)
        N, H, W, Cin = x.shape
        Cout = dy.shape[3]
        dw = np.empty((Cout, 3, 3, Cin), self.dt)
        db = np.empty((Cout,), self.dt)
        self.lib.orc_conv3x3_wgrad(_p(x), _p(dy), _p(dw), _p(db), N, H, W, Cin, Cout)
        return dw, db

    def pool_fwd(self, x):
        x = self._a(x)
        N, H, W, C = x.shape
        p = np.empty((N, H // 2, W // 2, C), self.dt)
        idx = np.empty((N, H // 2, W // 2, C), np.uint8)
        self.lib.orc_maxpool2_fwd(_p(x), _p(p), _p(idx), N, H, W, C)
        return p, idx

    def pool_bwd(self, dp, idx):
        dp = self._a(dp)
        N, Ho, Wo, C = dp.shape
        dx = np.empty((N, 2 * Ho, 2 * Wo, C), self.dt)
        self.lib.orc_maxpool2_bwd(_p(dp), _p(np.ascontiguousarray(idx)), _p(dx), N, 2 * Ho, 2 * Wo, C)
        return dx

    def fc_fwd(self, X, Wt, b, relu):
        X, Wt, b = self._a(X), self._a(Wt), self._a(b)
        B, d_in = X.shape
        out_j = Wt.shape[0]
        Y = np.empty((B, out_j), self.dt)
        self.lib.orc_fc_fwd(_p(X), _p(Wt), _p(b), _p(Y), B, d_in, out_j, int(relu))
        return Y

    def fc_bwd(self, X, Wt, dY):
        X, Wt, dY = self._a(X), self._a(Wt), self._a(dY)
        B, d_in = X.shape
        out_j = Wt.shape[0]
        dW = np.empty((out_j, d_in), self.dt)
        db = np.empty((out_j,), self.dt)
        dX = np.empty((B, d_in), self.dt)
        self.lib.orc_fc_bwd(_p(X), _p(Wt), _p(dY), _p(dW), _p(db), _p(dX), B, d_in, out_j)
        return dW, db, dX

    def softmax_xent(self, Z, labels, scale):
        Z = self._a(Z)
        labels = np.ascontiguousarray(labels, dtype=np.int32)
        B, C = Z.shape
        row = np.empty((B,), self.dt)
        dZ = np.empty((B, C), self.dt)
        self.lib.orc_softmax_xent(_p(Z), _p(labels), _p(row), _p(dZ), B, C, self.creal(scale))
        return row, dZ

    def sgd(self, w, v, g, lr, mu):
        assert w.dtype == self.dt and v.dtype == self.dt and w.flags.c_contiguous and v.flags.c_contiguous
        g = self._a(g)
        self.lib.orc_sgd_momentum(_p(w), _p(v), _p(g), ctypes.c_size_t(w.size), self.creal(lr), self.creal(mu))


class OracleModel:
    """The partitioned network: one copy of the (replicated, always in-sync) conv parameters,
    K shards of every FC layer, momentum buffers of the same shapes."""

    def __init__(self, layers, H, W, C, b, R, K, real="float", bf16=False, loss_B=None):
        self.layers = list(layers)
        self.H, self.W, self.C, self.b, self.R, self.K = H, W, C, b, R, K
        self.B = b * R
        # loss_B: size of the batch the mean loss is taken over.  It defaults to this model's own batch; a
        # test that follows a few sampled images of a larger batch sets it to that batch size, so that the
        # per-row gradients (softmax - onehot)/loss_B are the ones those rows have inside the large batch
        # (every row's forward and activation-gradient computation is independent of the other rows).
        self.loss_B = loss_B if loss_B is not None else self.B
        self.P = Prims(real)
        self.dt = self.P.dt
        self.bf16 = bf16
        self.params = [None] * len(layers)   # conv: {'w','b'}; fc: [ {'w','b'} per shard ]
        self.mom = [None] * len(layers)
        self.bounds = [None] * len(layers)   # fc: shard column boundaries
        self.grads = [None] * len(layers)
        self.dropout_seed, self.dropout_step = 0, 0   # key and iteration counter of the dropout masks

    # ---- helpers -------------------------------------------------------------------------
    def _q(self, a):
        """Storage rounding of the mixed-precision mode (identity otherwise)."""
        return round_bf16(a) if self.bf16 else a

    def set_dropout(self, seed, step=0):
        """Key of the dropout masks and the iteration number the next forward pass draws them for."""
        self.dropout_seed, self.dropout_step = int(seed), int(step)

    def load_params(self, full_params):
        """Take the logical (unpartitioned) parameters and split every FC layer by output column
        into K shards of 1/K size [Layer Partitioning]; momentum starts at zero."""
        for li, (kind, out) in enumerate(self.layers):
            p = full_params[li]
            if kind == CONV:
                self.params[li] = {"w": np.array(p["w"], self.dt), "b": np.array(p["b"], self.dt)}
                self.mom[li] = {"w": np.zeros_like(self.params[li]["w"]), "b": np.zeros_like(self.params[li]["b"])}
            elif kind in (FC_RELU, FC):
                cb = shard_bounds(out, self.K)
                self.bounds[li] = cb
                self.params[li] = [{"w": np.array(p["w"][cb[j]:cb[j + 1]], self.dt),
                                    "b": np.array(p["b"][cb[j]:cb[j + 1]], self.dt)} for j in range(self.K)]
                self.mom[li] = [{"w": np.zeros_like(s["w"]), "b": np.zeros_like(s["b"])} for s in self.params[li]]

    def full_params(self):
        """Logical parameters reassembled from the shards (for comparisons across partitionings)."""
        return self._assemble(self.params)

    def full_grads(self):
        return self._assemble(self.grads)

    def full_mom(self):
        return self._assemble(self.mom)

    def _assemble(self, src):
        out = []
        for li, (kind, _) in enumerate(self.layers):
            if kind == CONV:
                out.append({"w": src[li]["w"].copy(), "b": src[li]["b"].copy()})
            elif kind in (FC_RELU, FC):
                out.append({"w": np.concatenate([s["w"] for s in src[li]], 0),
                            "b": np.concatenate([s["b"] for s in src[li]], 0)})
            else:
                out.append(None)
        return out

    # ---- forward -------------------------------------------------------------------------
    def forward(self, x_list, labels_list):
        """x_list: R arrays [b,H,W,C]; labels_list: R int arrays [b].  Returns the mean loss."""
        P, R, b = self.P, self.R, self.b
        assert len(x_list) == R and len(labels_list) == R
        nl = len(self.layers)
        self.x_in = [self._q(np.array(x, self.dt)) for x in x_list]
        self.conv_out = [[None] * nl for _ in range(R)]   # per replica, per conv-side layer output
        self.pool_idx = [[None] * nl for _ in range(R)]
        self.fc_in = [None] * nl                          # full-width input of each FC layer [B,in]
        self.fc_out = [None] * nl                         # full-width output (after the shard layer)
        self.drop_keep = [None] * nl                      # dropout layers: the keep mask [B,width]
        first_fc = next(i for i, (k, _) in enumerate(self.layers) if k in (FC_RELU, FC))
        self.first_fc = first_fc
        # 1. data-parallel convolution stack, one replica at a time
        feats = []
        for r in range(R):
            a = self.x_in[r]
            for li in range(first_fc):
                kind, _ = self.layers[li]
                if kind == CONV:
                    w = self._q(self.params[li]["w"])
                    a = self._q(P.conv_fwd(a, w, self.params[li]["b"], relu=True))
                elif kind == POOL:
                    a, self.pool_idx[r][li] = P.pool_fwd(a)
                else:
                    raise ValueError("conv-side layer expected")
                self.conv_out[r][li] = a
            feats.append(a.reshape(b, -1))                # flatten in (h, w, c) order
        self.feat_shape = a.shape
        # 2. modulo layer forward: gather; row g <- replica g // b, local row g % b
        D = feats[0].shape[1]
        X = np.empty((self.B, D), self.dt)
        for g in range(self.B):
            X[g, :] = feats[g // b][g % b, :]
        labels = np.empty((self.B,), np.int32)
        for g in range(self.B):
            labels[g] = labels_list[g // b][g % b]
        self.labels = labels
        # 3./4. sharded FC layers with a shard layer (column concat) after each
        for li in range(first_fc, nl):
            kind, out = self.layers[li]
            if kind in (FC_RELU, FC):
                self.fc_in[li] = X
                cb = self.bounds[li]
                Y = np.empty((self.B, out), self.dt)
                for j in range(self.K):
                    sh = self.params[li][j]
                    Yj = P.fc_fwd(X, self._q(sh["w"]), sh["b"], relu=(kind == FC_RELU))
                    Y[:, cb[j]:cb[j + 1]] = Yj            # shard layer: all-gather of column slices
                if kind == FC_RELU:
                    Y = self._q(Y)                        # stored activation; logits stay unrounded
                self.fc_out[li] = Y
                X = Y
            elif kind == DROPOUT:
                # one-to-one layer on the partitioned width: shard j masks and rescales its own columns of the layer
                # below (an FC + ReLU), before the shard layer gathers them
                assert self.layers[li - 1][0] == FC_RELU, "dropout follows an FC + ReLU layer"
                cb = self.bounds[li - 1]
                width = X.shape[1]
                keep = dropout_keep(self.dropout_seed, self.dropout_step, li, np.arange(self.B), width, out)
                scale = dropout_scale(out)
                Y = np.empty_like(X)
                for j in range(self.K):
                    Xj, kj = X[:, cb[j]:cb[j + 1]], keep[:, cb[j]:cb[j + 1]]
                    Y[:, cb[j]:cb[j + 1]] = self._q(np.where(kj, Xj * self.dt(scale), self.dt(0)))
                self.drop_keep[li] = keep
                self.fc_out[li] = Y
                X = Y
            elif kind == LOSS:
                # 5. log-softmax + NLL, mean over the full batch
                self.logits = X
                self.row_loss, self.dZ = P.softmax_xent(X, labels, 1.0 / self.loss_B)
                self.loss = self.dt(np.sum(self.row_loss, dtype=self.dt) / self.dt(self.B))
        if any(k == DROPOUT for k, _ in self.layers):
            self.dropout_step += 1                        # the next forward pass draws fresh masks
        return self.loss

    # ---- backward ------------------------------------------------------------------------
    def backward(self):
        P, R, b, K = self.P, self.R, self.b, self.K
        nl = len(self.layers)
        self.d_pre = [None] * nl      # FC layers: gradient w.r.t. the pre-activation output [B,out]
        self.d_fc_in = [None] * nl    # FC layers: gradient w.r.t. the (full-width) input, unmasked
        dY = self._q(self.dZ)         # gradient of the loss w.r.t. the last FC's output
        for li in range(nl - 2, self.first_fc - 1, -1):
            kind, out = self.layers[li]
            if kind == DROPOUT:
                # dY is the gradient w.r.t. this layer's output: the kept elements carry it down times 1/(1 - p); the
                # layer below is an FC + ReLU, whose mask and storage rounding follow
                self.d_pre[li] = dY
                dIn = np.where(self.drop_keep[li], dY * self.dt(dropout_scale(out)), self.dt(0))
                dY = self._q(dIn * (self.fc_out[li - 1] > 0))
                continue
            cb = self.bounds[li]
            self.d_pre[li] = dY
            X = self.fc_in[li]
            g = []
            dX = np.zeros_like(X)
            for j in range(K):                            # 6. shard-layer backward: sum over shards
                sh = self.params[li][j]
                dYj = np.ascontiguousarray(dY[:, cb[j]:cb[j + 1]])
                dWj, dbj, dXj = P.fc_bwd(X, self._q(sh["w"]), dYj)
                g.append({"w": dWj, "b": dbj})
                dX = dX + dXj
            self.grads[li] = g
            self.d_fc_in[li] = dX
            if li > self.first_fc and self.layers[li - 1][0] == DROPOUT:
                dY = self._q(dX)                          # stored gradient w.r.t. the dropout layer's output
            elif li > self.first_fc:
                # the layer below is an FC+ReLU: mask by its stored output, then store
                dY = self._q(dX * (self.fc_out[li - 1] > 0))
        # 7. modulo layer backward: rows back to their owners
        dfeat = [np.empty((b,) + self.feat_shape[1:], self.dt) for _ in range(R)]
        for g_ in range(self.B):
            dfeat[g_ // b][g_ % b] = dX[g_].reshape(self.feat_shape[1:])
        # 8. per-replica conv backward + DP reduce in replica order
        self.d_conv = [[None] * nl for _ in range(R)]  # conv: d wrt pre-activation; pool: d wrt pool output
        rep_grads = []
        for r in range(R):
            d = dfeat[r]                                  # gradient w.r.t. the output of layer li
            gr = {}
            for li in range(self.first_fc - 1, -1, -1):
                kind, _ = self.layers[li]
                below = self.conv_out[r][li - 1] if li > 0 else self.x_in[r]
                if kind == POOL:
                    d = self._q(d)
                    self.d_conv[r][li] = d
                    d = P.pool_bwd(d, self.pool_idx[r][li])
                else:
                    d = self._q(d * (self.conv_out[r][li] > 0))   # ReLU'(0) = 0
                    self.d_conv[r][li] = d
                    dw, db = P.conv_wgrad(below, d)
                    gr[li] = {"w": dw, "b": db}
                    if li > 0:
                        d = P.conv_dgrad(d, self._q(self.params[li]["w"]))
            rep_grads.append(gr)
        for li in range(self.first_fc):
            if self.layers[li][0] == CONV:
                gw = np.zeros_like(self.params[li]["w"])
                gb = np.zeros_like(self.params[li]["b"])
                for r in range(R):
                    gw = gw + rep_grads[r][li]["w"]
                    gb = gb + rep_grads[r][li]["b"]
                self.grads[li] = {"w": gw, "b": gb}

    # ---- update --------------------------------------------------------------------------
    def sgd_step(self, lr, mu):
        for li, (kind, _) in enumerate(self.layers):
            if kind == CONV:
                for k in ("w", "b"):
                    self.P.sgd(self.params[li][k], self.mom[li][k], self.grads[li][k], lr, mu)
            elif kind in (FC_RELU, FC):
                for j in range(self.K):
                    for k in ("w", "b"):
                        self.P.sgd(self.params[li][j][k], self.mom[li][j][k], self.grads[li][j][k], lr, mu)

    def step(self, x_list, labels_list, lr, mu):
        loss = self.forward(x_list, labels_list)
        self.backward()
        self.sgd_step(lr, mu)
        return loss

    # ---- the modulo layer's own schedule [Modulo Layer] ------------------------------------
    def modulo_rows(self, k):
        """Rows (in gather order g = r*b + i) that sub-iteration k sends through the FC stack: every replica's k-th
        slice of b/K local examples, replica-major -- row p of the sub-batch comes from replica p // (b/K)."""
        bk = self.b // self.K
        return np.array([r * self.b + k * bk + i for r in range(self.R) for i in range(bk)], dtype=np.int64)

    def step_modulo(self, x_list, labels_list, lr, mu):
        """One iteration in the paper's schedule: the conv stack runs once on the whole local batches, then the FC
        stack runs K sub-iterations, each on a distinct b/K examples of every replica; the FC parameters are
        updated after every sub-iteration with gradients divided by K, the conv parameters once at the end.

        Normalisation: every row's loss gradient is (softmax - onehot)/B, B = R*b.  For the FC parameters that is
        the mean over the sub-batch divided by K (the paper's compensation); for the conv stack it is what the
        synchronous iteration uses, so with K = 1 this is step().  Returns the mean of the B row losses (each
        taken with the FC parameters of its own sub-iteration)."""
        P, R, b, K = self.P, self.R, self.b, self.K
        assert b % K == 0, "the modulo schedule needs b divisible by K"
        nl = len(self.layers)
        first_fc = next(i for i, (k, _) in enumerate(self.layers) if k in (FC_RELU, FC))
        assert first_fc > 0, "the modulo layer sits between a conv-side stack and the FC stack"
        self.first_fc = first_fc
        # 1. conv stack forward, all rows, once (as in forward())
        self.x_in = [self._q(np.array(x, self.dt)) for x in x_list]
        self.conv_out = [[None] * nl for _ in range(R)]
        self.pool_idx = [[None] * nl for _ in range(R)]
        feats = []
        for r in range(R):
            a = self.x_in[r]
            for li in range(first_fc):
                kind, _ = self.layers[li]
                if kind == CONV:
                    a = self._q(P.conv_fwd(a, self._q(self.params[li]["w"]), self.params[li]["b"], relu=True))
                else:
                    a, self.pool_idx[r][li] = P.pool_fwd(a)
                self.conv_out[r][li] = a
            feats.append(a.reshape(b, -1))
        self.feat_shape = a.shape
        D = feats[0].shape[1]
        X_all = np.empty((self.B, D), self.dt)
        labels_all = np.empty((self.B,), np.int32)
        for g in range(self.B):
            X_all[g, :] = feats[g // b][g % b, :]
            labels_all[g] = labels_list[g // b][g % b]
        dX_all = np.zeros((self.B, D), self.dt)
        row_loss_all = np.zeros((self.B,), self.dt)
        self.mod_fc_grads = []            # per sub-iteration: the FC gradients that were applied (for tests)
        # 2. K sub-iterations of the FC stack
        for k in range(K):
            rows = self.modulo_rows(k)
            X = np.ascontiguousarray(X_all[rows])
            labels = np.ascontiguousarray(labels_all[rows])
            fc_in, fc_out, drop_keep = {}, {}, {}
            for li in range(first_fc, nl):
                kind, out = self.layers[li]
                if kind in (FC_RELU, FC):
                    fc_in[li] = X
                    cb = self.bounds[li]
                    Y = np.empty((X.shape[0], out), self.dt)
                    for j in range(K):
                        sh = self.params[li][j]
                        Y[:, cb[j]:cb[j + 1]] = P.fc_fwd(X, self._q(sh["w"]), sh["b"], relu=(kind == FC_RELU))
                    if kind == FC_RELU:
                        Y = self._q(Y)
                    fc_out[li] = Y
                    X = Y
                elif kind == DROPOUT:
                    # the masks of an iteration belong to the examples (global rows), whichever sub-iteration carries them
                    cb = self.bounds[li - 1]
                    keep = dropout_keep(self.dropout_seed, self.dropout_step, li, rows, X.shape[1], out)
                    Y = np.empty_like(X)
                    for j in range(K):
                        Y[:, cb[j]:cb[j + 1]] = self._q(np.where(keep[:, cb[j]:cb[j + 1]], X[:, cb[j]:cb[j + 1]] * self.dt(dropout_scale(out)), self.dt(0)))
                    drop_keep[li] = keep
                    fc_out[li] = Y
                    X = Y
                else:
                    row_loss, dZ = P.softmax_xent(X, labels, 1.0 / self.B)
                    row_loss_all[rows] = row_loss
            dY = self._q(dZ)
            g_k = {}
            for li in range(nl - 2, first_fc - 1, -1):
                if self.layers[li][0] == DROPOUT:
                    dIn = np.where(drop_keep[li], dY * self.dt(dropout_scale(self.layers[li][1])), self.dt(0))
                    dY = self._q(dIn * (fc_out[li - 1] > 0))
                    continue
                cb = self.bounds[li]
                Xin = fc_in[li]
                g = []
                dX = np.zeros_like(Xin)
                for j in range(K):
                    sh = self.params[li][j]
                    dWj, dbj, dXj = P.fc_bwd(Xin, self._q(sh["w"]), np.ascontiguousarray(dY[:, cb[j]:cb[j + 1]]))
                    g.append({"w": dWj, "b": dbj})
                    dX = dX + dXj
                g_k[li] = g
                if li > first_fc and self.layers[li - 1][0] == DROPOUT:
                    dY = self._q(dX)
                elif li > first_fc:
                    dY = self._q(dX * (fc_out[li - 1] > 0))
            dX_all[rows] = dX
            self.mod_fc_grads.append(g_k)
            for li, g in g_k.items():     # FC update of this sub-iteration
                self.grads[li] = g
                for j in range(K):
                    for key in ("w", "b"):
                        P.sgd(self.params[li][j][key], self.mom[li][j][key], g[j][key], lr, mu)
        self.row_loss = row_loss_all
        self.loss = self.dt(np.sum(row_loss_all, dtype=self.dt) / self.dt(self.B))
        if any(k_ == DROPOUT for k_, _ in self.layers):
            self.dropout_step += 1                        # one iteration = all K sub-iterations
        # 3. modulo layer backward + conv stack backward on all rows, DP reduce, conv update (as in backward())
        dfeat = [np.empty((b,) + self.feat_shape[1:], self.dt) for _ in range(R)]
        for g_ in range(self.B):
            dfeat[g_ // b][g_ % b] = dX_all[g_].reshape(self.feat_shape[1:])
        self.mod_dfeat = dfeat
        rep_grads = []
        for r in range(R):
            d = dfeat[r]
            gr = {}
            for li in range(first_fc - 1, -1, -1):
                kind, _ = self.layers[li]
                below = self.conv_out[r][li - 1] if li > 0 else self.x_in[r]
                if kind == POOL:
                    d = P.pool_bwd(self._q(d), self.pool_idx[r][li])
                else:
                    d = self._q(d * (self.conv_out[r][li] > 0))
                    dw, db = P.conv_wgrad(below, d)
                    gr[li] = {"w": dw, "b": db}
                    if li > 0:
                        d = P.conv_dgrad(d, self._q(self.params[li]["w"]))
            rep_grads.append(gr)
        for li in range(first_fc):
            if self.layers[li][0] == CONV:
                gw = np.zeros_like(self.params[li]["w"])
                gb = np.zeros_like(self.params[li]["b"])
                for r in range(R):
                    gw = gw + rep_grads[r][li]["w"]
                    gb = gb + rep_grads[r][li]["b"]
                self.grads[li] = {"w": gw, "b": gb}
                for key in ("w", "b"):
                    P.sgd(self.params[li][key], self.mom[li][key], self.grads[li][key], lr, mu)
        return self.loss


def from_workload(wl, real="float", bf16=False, loss_B=None) -> OracleModel:
    return OracleModel(wl.layers, wl.H, wl.W, wl.C, wl.b, wl.R, wl.K, real=real, bf16=bf16, loss_B=loss_B)
