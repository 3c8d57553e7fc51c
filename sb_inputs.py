"""Seeded synthetic inputs and workload definitions shared by the CPU oracle tests and the GPU tests.

This module generates *inputs only*: network descriptions (layer lists and shapes), images,
labels and initial parameters.  It contains none of the training arithmetic (no convolution,
no GEMM, no loss, no optimiser), so both the oracle and the CUDA library can be fed from it
without sharing any computation.

Every tensor is drawn from a counter-based Philox stream keyed by (seed, tensor id) over the
*logical* (unpartitioned) tensor, so that a given weight or pixel has the same value for every
replica count R and shard count K.  That property is what makes the partition-invariance tests
(the paper's Layer Partitioning paragraph: the sharded network must evaluate the same output
error as the complete local model) meaningful.

Layouts: images NHWC float32; conv weights [Cout][3][3][Cin]; FC weights [out][in] with the
input index running over the flattened (h, w, c) feature map.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

# Layer kinds (same integer codes as the C header's sb_layer_kind).
CONV3X3_RELU = 1
MAXPOOL2 = 2
FC_RELU = 3
FC = 4
SOFTMAX_XENT = 5
FC_RELU_WHOLE = 6   # FC + ReLU that the partitioning keeps whole on every worker
FC_WHOLE = 7
DROPOUT = 8         # out = drop probability in units of 1/65536; follows an FC + ReLU layer

SEED_WEIGHTS = 2112
SEED_DATA = 15317


@dataclass
class Workload:
    """A network plus its partitioning: R replicas of b images, K column shards per FC layer."""

    name: str
    layers: List[Tuple[int, int]]  # (kind, out) ; out = Cout / out-features / classes, 0 for pool
    H: int
    W: int
    C: int
    b: int  # images per replica
    R: int
    K: int
    classes: int = field(init=False)

    def __post_init__(self):
        assert self.layers[-1][0] == SOFTMAX_XENT
        self.classes = self.layers[-1][1]

    @property
    def B(self) -> int:
        return self.b * self.R

    def with_partition(self, R: int, K: int, name: str | None = None) -> "Workload":
        """Same network and same total batch, different logical partitioning."""
        assert self.B % R == 0
        return Workload(name or f"{self.name}_R{R}K{K}", list(self.layers), self.H, self.W, self.C,
                        self.B // R, R, K)

    def with_batch(self, b: int, name: str | None = None) -> "Workload":
        return Workload(name or f"{self.name}_b{b}", list(self.layers), self.H, self.W, self.C,
                        b, self.R, self.K)


def layer_shapes(wl: Workload):
    """Walk the layer list and return one dict per layer with its input/output geometry.

    conv : {'kind','H','W','Cin','Cout'}          (H, W preserved: 3x3, stride 1, zero pad 1)
    pool : {'kind','H','W','C'}                   (input H, W; output H/2, W/2)
    fc   : {'kind','in','out','relu'}
    dropout : {'kind','width','units'}            (units = drop probability * 65536)
    loss : {'kind','classes'}
    """
    H, W, C = wl.H, wl.W, wl.C
    feat = None
    out = []
    for kind, o in wl.layers:
        if kind == CONV3X3_RELU:
            assert feat is None, "conv after FC"
            out.append(dict(kind=kind, H=H, W=W, Cin=C, Cout=o))
            C = o
        elif kind == MAXPOOL2:
            assert feat is None and H % 2 == 0 and W % 2 == 0
            out.append(dict(kind=kind, H=H, W=W, C=C))
            H //= 2
            W //= 2
        elif kind in (FC_RELU, FC, FC_RELU_WHOLE, FC_WHOLE):
            if feat is None:
                feat = H * W * C
            kind = FC_RELU if kind in (FC_RELU, FC_RELU_WHOLE) else FC      # (shapes and initial values do not depend on the split)
            out.append({"kind": kind, "in": feat, "out": o, "relu": kind == FC_RELU})
            feat = o
        elif kind == DROPOUT:
            assert feat is not None and 0 < o < 65536
            out.append(dict(kind=kind, width=feat, units=o))
        elif kind == SOFTMAX_XENT:
            assert feat == o, "loss width must equal last FC width"
            out.append(dict(kind=kind, classes=o))
        else:
            raise ValueError(f"unknown layer kind {kind}")
    return out


def shard_bounds(out: int, K: int):
    """Column-shard boundaries c_0..c_K with c_j = floor(j*out/K) (uneven shards allowed)."""
    return [(j * out) // K for j in range(K + 1)]


def vgg16_layers(fc_in_hw: int, classes: int, fc_width: int = 4096):
    widths = [(64, 2), (128, 2), (256, 3), (512, 3), (512, 3)]
    layers = []
    for w, reps in widths:
        layers += [(CONV3X3_RELU, w)] * reps + [(MAXPOOL2, 0)]
    layers += [(FC_RELU, fc_width), (FC_RELU, fc_width), (FC, classes), (SOFTMAX_XENT, classes)]
    return layers


def tiny_layers():
    return [(CONV3X3_RELU, 16), (MAXPOOL2, 0), (CONV3X3_RELU, 32), (MAXPOOL2, 0),
            (FC_RELU, 64), (FC, 10), (SOFTMAX_XENT, 10)]


def paper_vgg_variant_layers():
    """The 7-conv / 3-FC CIFAR network of the paper's Table 1 (pool placement inferred from
    FC0's 4096 = 256*4*4 inputs: three 2x2 pools on 32x32 images)."""
    L = [(CONV3X3_RELU, 64), (CONV3X3_RELU, 64), (MAXPOOL2, 0),
         (CONV3X3_RELU, 128), (CONV3X3_RELU, 128), (MAXPOOL2, 0),
         (CONV3X3_RELU, 256), (CONV3X3_RELU, 256), (CONV3X3_RELU, 256), (MAXPOOL2, 0),
         (FC_RELU, 1024), (FC_RELU, 1024), (FC, 10), (SOFTMAX_XENT, 10)]
    return L


def config(i: int) -> Workload:
    """The benchmark configurations, in order."""
    if i == 0:
        return Workload("cfg0_tiny", tiny_layers(), 32, 32, 3, 4, 2, 2)
    if i == 1:
        return Workload("cfg1_vgg16_cifar_b128", vgg16_layers(1, 10), 32, 32, 3, 32, 4, 4)
    if i == 2:
        return Workload("cfg2_vgg16_cifar_b256", vgg16_layers(1, 10), 32, 32, 3, 32, 8, 8)
    if i == 3:
        return Workload("cfg3_vgg16_imagenet_b64", vgg16_layers(7, 1000), 224, 224, 3, 16, 4, 4)
    if i == 5:
        # the paper's own evaluation network (Table 1), one MP group of four workers: mp = 4, 32 images per worker
        return Workload("cfg5_paper_vgg_cifar_b128", paper_vgg_variant_layers(), 32, 32, 3, 32, 4, 4)
    raise ValueError("config 4 is the FC sweep: see fc_sweep_case()")


def _gen(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed & 0xFFFFFFFFFFFFFFFF, tensor_id]))


def make_batch(wl: Workload, seed: int = SEED_DATA):
    """Images ~ N(0,1) [B,H,W,C] float32 and labels uniform in [0, classes) int32, over the whole
    batch; replica r owns rows [r*b, (r+1)*b)."""
    x = _gen(seed, 1).standard_normal((wl.B, wl.H, wl.W, wl.C), dtype=np.float32)
    y = _gen(seed, 2).integers(0, wl.classes, size=(wl.B,), dtype=np.int64).astype(np.int32)
    return x, y


def split_replicas(a: np.ndarray, R: int):
    """Rows of a whole-batch array as a list of R per-replica arrays (contiguous copies)."""
    b = a.shape[0] // R
    return [np.ascontiguousarray(a[r * b:(r + 1) * b]) for r in range(R)]


def make_params(wl: Workload, seed: int = SEED_WEIGHTS, bias_std: float = 0.0):
    """He-normal weights (std sqrt(2/fan_in); fan_in = 9*Cin for conv, `in` for FC) and zero
    biases for the logical, unpartitioned network: a list with one entry per layer, None for
    layers without parameters, else {'w': ..., 'b': ...} in float32.

    bias_std > 0 draws N(0, bias_std^2) biases instead of zeros; tests use it so that a bias
    handled wrongly cannot hide behind a zero.
    """
    params = []
    for li, s in enumerate(layer_shapes(wl)):
        if s["kind"] == CONV3X3_RELU:
            fan_in = 9 * s["Cin"]
            w = _gen(seed, 100 + 2 * li).standard_normal((s["Cout"], 3, 3, s["Cin"]), dtype=np.float32)
            nb = s["Cout"]
        elif s["kind"] in (FC_RELU, FC):
            fan_in = s["in"]
            w = _gen(seed, 100 + 2 * li).standard_normal((s["out"], s["in"]), dtype=np.float32)
            nb = s["out"]
        else:
            params.append(None)
            continue
        w *= np.float32(np.sqrt(2.0 / fan_in))
        if bias_std > 0:
            bb = (_gen(seed, 101 + 2 * li).standard_normal((nb,), dtype=np.float32) * np.float32(bias_std))
        else:
            bb = np.zeros((nb,), dtype=np.float32)
        params.append({"w": w, "b": bb})
    return params


def fc_sweep_case(B: int, seed: int = SEED_WEIGHTS, d_in: int = 25088, d_out: int = 4096):
    """Inputs of the sharded-FC sweep: W [out][in] ~ N(0, 2/in), X [B][in] ~ N(0,1), dY [B][out] ~ N(0,1)."""
    w = _gen(seed, 900).standard_normal((d_out, d_in), dtype=np.float32) * np.float32(np.sqrt(2.0 / d_in))
    x = _gen(seed, 901 + B).standard_normal((B, d_in), dtype=np.float32)
    dy = _gen(seed, 5901 + B).standard_normal((B, d_out), dtype=np.float32)
    return w, x, dy


def param_count(wl: Workload):
    """(conv weights, conv biases, fc weights, fc biases) element counts of the logical network."""
    cw = cb = fw = fb = 0
    for s in layer_shapes(wl):
        if s["kind"] == CONV3X3_RELU:
            cw += 9 * s["Cin"] * s["Cout"]
            cb += s["Cout"]
        elif s["kind"] in (FC_RELU, FC):
            fw += s["in"] * s["out"]
            fb += s["out"]
    return cw, cb, fw, fb
