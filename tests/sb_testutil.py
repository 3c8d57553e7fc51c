"""Shared helpers for the parity tests: run the same seeded workload through the oracle and through
the CUDA library (C ABI via the ctypes binding) and compare tensors."""
from __future__ import annotations

import numpy as np

import sb_inputs as si


def maxrel(a, ref):
    a = np.asarray(a, np.float64)
    ref = np.asarray(ref, np.float64)
    assert a.shape == ref.shape, (a.shape, ref.shape)
    d = float(np.max(np.abs(a - ref))) if a.size else 0.0
    return d / (float(np.max(np.abs(ref))) + 1e-30)


def frob(a, ref):
    a = np.asarray(a, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.linalg.norm(a - ref) / (np.linalg.norm(ref) + 1e-30))


def outlier_fraction(a, ref, tol):
    a = np.asarray(a, np.float64)
    ref = np.asarray(ref, np.float64)
    return float(np.mean(np.abs(a - ref) > tol * (np.max(np.abs(ref)) + 1e-30)))


class Checks:
    """Collects (name, value, bound) comparisons so that one run reports every violation, not just the first.
    `log` keeps everything that was measured (a probe can print it); finish() asserts that nothing exceeded its bound."""

    def __init__(self):
        self.log = []

    def le(self, name, value, bound):
        self.log.append((name, float(value), float(bound)))

    def worst(self, prefix):
        vals = [v for n, v, _ in self.log if str(n).startswith(prefix)]
        return max(vals) if vals else 0.0

    def finish(self):
        bad = [(n, v, b) for n, v, b in self.log if not v <= b]
        assert not bad, "parity bounds exceeded: " + "; ".join(f"{n}: {v:.3e} > {b:.1e}" for n, v, b in bad[:12])


def all_split(wl):
    """The same workload with every FC layer split K ways (an FC layer kept whole computes the same function: the oracle,
    which splits every FC layer, serves as the reference for both)."""
    kinds = {si.FC_RELU_WHOLE: si.FC_RELU, si.FC_WHOLE: si.FC}
    return si.Workload(wl.name, [(kinds.get(k, k), o) for k, o in wl.layers], wl.H, wl.W, wl.C, wl.b, wl.R, wl.K)


def oracle_model(wl, params, bf16, real="float"):
    from oracle import splitbrain_oracle as so
    m = so.from_workload(all_split(wl), real=real, bf16=bf16)
    m.load_params(params)
    return m


def gpu_model(wl, params, precision, flags=0):
    from paper_2112_15317_b200 import binding as sb
    m = sb.Model.from_workload(wl, precision=precision, flags=flags)
    m.load_params(params, si.shard_bounds)
    return m


def device_batch(wl, x, y, bf16):
    """Per-replica device tensors of the images (activation dtype) and labels."""
    import torch
    xs = [torch.from_numpy(a).cuda() for a in si.split_replicas(x, wl.R)]
    if bf16:
        xs = [t.to(torch.bfloat16) for t in xs]
    ys = [torch.from_numpy(a).cuda() for a in si.split_replicas(y, wl.R)]
    return xs, ys
