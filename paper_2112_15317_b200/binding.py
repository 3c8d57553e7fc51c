"""ctypes binding of libsplitbrain.so: argument marshalling only.

Module-level functions carry the names of the C entry points (include/splitbrain.h) and return
the sb_status code unchanged.  `Model` is a convenience wrapper that owns the torch arena tensor,
converts numpy/torch arguments to pointers and raises SBError on a non-zero status; every step of
the training iteration itself runs inside the library's CUDA kernels.  There is no CPU fallback:
importing this module without the built library raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int32, c_int64, c_size_t, c_void_p

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsplitbrain.so")

SB_OK = 0
SB_FP32, SB_BF16 = 0, 1
SB_CONV3X3_RELU, SB_MAXPOOL2, SB_FC_RELU, SB_FC, SB_SOFTMAX_XENT, SB_FC_RELU_WHOLE, SB_FC_WHOLE, SB_DROPOUT = 1, 2, 3, 4, 5, 6, 7, 8
SB_NODE_LAYER, SB_NODE_MODULO, SB_NODE_SHARD = 0, 1, 2
SB_X_GATHER_ROWS, SB_X_GATHER_COLS, SB_X_REDUCE_COLS, SB_X_REDUCE_ROWS, SB_X_ALLREDUCE, SB_X_ALLREDUCE_GROUPS = 1, 2, 3, 4, 5, 6
SB_FLAG_INPUT_GRAD, SB_FLAG_FORCE_SIMT, SB_FLAG_PROFILE_LAYERS, SB_FLAG_FORCE_PAIR, SB_FLAG_MODULO_SCHEDULE, SB_FLAG_NO_HALO, SB_FLAG_FORCE_PERSIST = 1, 2, 4, 8, 16, 32, 64
(SB_T_WEIGHT, SB_T_BIAS, SB_T_GRAD_W, SB_T_GRAD_B, SB_T_MOM_W, SB_T_MOM_B, SB_T_ACT, SB_T_DACT,
 SB_T_POOL_IDX, SB_T_ROW_LOSS, SB_T_INPUT_GRAD, SB_T_SHADOW_W) = range(12)
SB_DT_F32, SB_DT_BF16, SB_DT_U8, SB_DT_I32 = 0, 1, 2, 3
STATUS_NAMES = {0: "SB_OK", 1: "SB_ERR_INVALID_ARG", 2: "SB_ERR_SHAPE", 3: "SB_ERR_UNSUPPORTED",
                4: "SB_ERR_ARENA_TOO_SMALL", 5: "SB_ERR_CUDA", 6: "SB_ERR_STATE", 7: "SB_ERR_TIMEOUT"}


class sb_layer(ctypes.Structure):
    _fields_ = [("kind", c_int32), ("out", c_int32)]


class sb_config(ctypes.Structure):
    _fields_ = [("H", c_int32), ("W", c_int32), ("C", c_int32), ("batch_per_replica", c_int32),
                ("R", c_int32), ("K", c_int32), ("precision", c_int32), ("flags", c_int32)]


class sb_plan_node(ctypes.Structure):
    _fields_ = [("node", c_int32), ("layer", c_int32), ("shards", c_int32), ("reserved", c_int32), ("dim", c_int64), ("dimF", c_int64)]


class sb_exchange_msg(ctypes.Structure):
    _fields_ = [("kind", c_int32), ("layer", c_int32), ("pass_", c_int32), ("src", c_int32), ("dst", c_int32), ("reserved", c_int32),
                ("row0", c_int64), ("row1", c_int64), ("col0", c_int64), ("col1", c_int64), ("width", c_int64)]


class sb_profile_entry(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char * 32), ("launches", c_int32), ("ms_total", c_float),
                ("flops", ctypes.c_double), ("bytes", ctypes.c_double)]


class SBError(RuntimeError):
    def __init__(self, status, msg):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {msg}")
        self.status = status


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2112_15317_b200.build_ext` "
            "(nvcc, sm_100a).  There is no CPU fallback.")
    lib = ctypes.CDLL(LIB_PATH)
    P = POINTER
    sigs = {
        "sb_model_bytes": [P(sb_layer), c_int32, P(sb_config), P(c_size_t)],
        "sb_model_create": [P(sb_layer), c_int32, P(sb_config), c_void_p, c_size_t, P(c_void_p)],
        "sb_model_destroy": [c_void_p],
        "sb_forward": [c_void_p, P(c_void_p), P(c_void_p), c_void_p],
        "sb_backward": [c_void_p, c_void_p],
        "sb_graph_step": [c_void_p, P(c_void_p), P(c_void_p), c_float, c_float, c_void_p],
        "sb_modulo_step": [c_void_p, P(c_void_p), P(c_void_p), c_float, c_float, c_void_p],
        "sb_debug_wait_probe": [c_void_p, c_int32, c_void_p],
        "sb_debug_poison": [c_void_p, c_void_p],
        "sb_debug_check_guards": [c_void_p, c_void_p, P(c_int32), P(c_int64)],
        "sb_sgd_step": [c_void_p, c_float, c_float, c_void_p],
        "sb_loss": [c_void_p, c_void_p, P(c_float)],
        "sb_train_step_host": [c_void_p, c_void_p, c_void_p, c_float, c_float, c_void_p, P(c_float)],
        "sb_prefetch_host": [c_void_p, c_void_p, c_void_p],
        "sb_train_step_host_async": [c_void_p, c_void_p, c_void_p, c_float, c_float, c_void_p],
        "sb_train_step_host_wait": [c_void_p, c_void_p, P(c_float)],
        "sb_tensor": [c_void_p, c_int32, c_int32, c_int32, P(c_void_p), P(c_int64), P(c_int32)],
        "sb_tensor_read": [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_size_t],
        "sb_tensor_write": [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_size_t],
        "sb_refresh_shadow": [c_void_p, c_void_p],
        "sb_dropout_seed": [c_void_p, ctypes.c_uint64, ctypes.c_uint64, c_void_p],
        "sb_forward_layers": [c_void_p, c_int32, c_int32, P(c_void_p), P(c_void_p), c_void_p],
        "sb_backward_layers": [c_void_p, c_int32, c_int32, c_void_p],
        "sb_param_bytes": [c_void_p, c_int32, P(c_size_t)],
        "sb_launch_count": [c_void_p, P(c_int64)],
        "sb_conv_in_wgrad_static": [c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_int32, c_int32, c_void_p],
        "sb_partition": [P(sb_layer), c_int32, P(sb_config), P(sb_plan_node), c_int32, P(c_int32)],
        "sb_exchange_plan": [P(sb_layer), c_int32, P(sb_config), P(sb_exchange_msg), c_int32, P(c_int32)],
        "sb_profile_begin": [c_void_p, c_void_p],
        "sb_profile_end": [c_void_p, c_void_p, P(sb_profile_entry), c_int32, P(c_int32)],
    }
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = c_int32
    lib.sb_last_error.argtypes = []
    lib.sb_last_error.restype = c_char_p
    lib.sb_static_last_error.argtypes = []
    lib.sb_static_last_error.restype = c_char_p
    lib.sb_partition_last_error.argtypes = []
    lib.sb_partition_last_error.restype = c_char_p
    return lib, sigs


_lib, _SIGS = _load()
EXPORTED = sorted(list(_SIGS) + ["sb_last_error", "sb_static_last_error", "sb_partition_last_error"])

# Same-named module-level entry points (raw status codes).
sb_model_bytes = _lib.sb_model_bytes
sb_model_create = _lib.sb_model_create
sb_model_destroy = _lib.sb_model_destroy
sb_forward = _lib.sb_forward
sb_backward = _lib.sb_backward
sb_graph_step = _lib.sb_graph_step
sb_modulo_step = _lib.sb_modulo_step
sb_debug_wait_probe = _lib.sb_debug_wait_probe
sb_debug_poison = _lib.sb_debug_poison
sb_debug_check_guards = _lib.sb_debug_check_guards
sb_sgd_step = _lib.sb_sgd_step
sb_loss = _lib.sb_loss
sb_train_step_host = _lib.sb_train_step_host
sb_prefetch_host = _lib.sb_prefetch_host
sb_train_step_host_async = _lib.sb_train_step_host_async
sb_train_step_host_wait = _lib.sb_train_step_host_wait
sb_tensor = _lib.sb_tensor
sb_tensor_read = _lib.sb_tensor_read
sb_tensor_write = _lib.sb_tensor_write
sb_refresh_shadow = _lib.sb_refresh_shadow
sb_dropout_seed = _lib.sb_dropout_seed
sb_forward_layers = _lib.sb_forward_layers
sb_backward_layers = _lib.sb_backward_layers
sb_param_bytes = _lib.sb_param_bytes
sb_launch_count = _lib.sb_launch_count
sb_conv_in_wgrad_static = _lib.sb_conv_in_wgrad_static
sb_profile_begin = _lib.sb_profile_begin
sb_profile_end = _lib.sb_profile_end
sb_partition = _lib.sb_partition
sb_exchange_plan = _lib.sb_exchange_plan


def partition(layers, H, W, C, K):
    """The transformed network of sb_partition as a list of dicts (host-only; no GPU needed)."""
    arr = _layers_array(layers)
    cfg = sb_config(H, W, C, 1, K, K, SB_FP32, 0)
    n = c_int32()
    st = sb_partition(arr, len(layers), byref(cfg), None, 0, byref(n))
    if st != SB_OK:
        raise SBError(st, _lib.sb_partition_last_error().decode())
    out = (sb_plan_node * n.value)()
    st = sb_partition(arr, len(layers), byref(cfg), out, n.value, byref(n))
    if st != SB_OK:
        raise SBError(st, _lib.sb_partition_last_error().decode())
    return [dict(node=o.node, layer=o.layer, shards=o.shards, dim=o.dim, dimF=o.dimF) for o in out]


def exchange_plan(layers, H, W, C, b, N, mp=None):
    """The exchange schedule of N workers in MP groups of mp (default: one group of N) from sb_exchange_plan, as a list
    of dicts (host-only)."""
    arr = _layers_array(layers)
    cfg = sb_config(H, W, C, b, N, N if mp is None else mp, SB_FP32, 0)
    n = c_int32()
    st = sb_exchange_plan(arr, len(layers), byref(cfg), None, 0, byref(n))
    if st != SB_OK:
        raise SBError(st, _lib.sb_partition_last_error().decode())
    out = (sb_exchange_msg * max(n.value, 1))()
    st = sb_exchange_plan(arr, len(layers), byref(cfg), out, n.value, byref(n))
    if st != SB_OK:
        raise SBError(st, _lib.sb_partition_last_error().decode())
    return [dict(kind=o.kind, layer=o.layer, backward=o.pass_, src=o.src, dst=o.dst, rows=(o.row0, o.row1), cols=(o.col0, o.col1),
                 width=o.width) for o in out[:n.value]]


def sb_last_error() -> str:
    return _lib.sb_last_error().decode()


def sb_static_last_error() -> str:
    return _lib.sb_static_last_error().decode()


def conv_in_wgrad_static(x, dy, dw, db, precision):
    """Input-layer conv weight/bias gradient with the library's built-in scratch (no allocation anywhere).
    x [B,H,W,Cin], dy [B,H,W,Cout]: device tensors of the precision's dtype; dw [Cout,3,3,Cin], db [Cout]: float
    device tensors that receive the result.  Enqueues on torch's current stream."""
    import torch
    B, H, W, Cin = x.shape
    Cout = dy.shape[3]
    st = _lib.sb_conv_in_wgrad_static(c_void_p(x.data_ptr()), c_void_p(dy.data_ptr()), c_void_p(dw.data_ptr()),
                                      c_void_p(db.data_ptr()), B, H, W, Cin, Cout, precision,
                                      c_void_p(torch.cuda.current_stream().cuda_stream))
    if st != SB_OK:
        raise SBError(st, sb_static_last_error())


def _check(status):
    if status != SB_OK:
        raise SBError(status, sb_last_error())


def _layers_array(layers):
    arr = (sb_layer * len(layers))()
    for i, (k, o) in enumerate(layers):
        arr[i].kind, arr[i].out = int(k), int(o)
    return arr


_NP_DT = {SB_DT_F32: np.float32, SB_DT_BF16: np.uint16, SB_DT_U8: np.uint8, SB_DT_I32: np.int32}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16) with round-to-nearest-even, via torch (data marshalling)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16).copy()


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32)


class Model:
    """Owns the device arena (a torch uint8 tensor) and the sb_model handle."""

    def __init__(self, layers, H, W, C, b, R, K, precision=SB_BF16, flags=0, device="cuda:0"):
        import torch
        self.torch = torch
        self.layers = [(int(k), int(o)) for k, o in layers]
        self.cfg = sb_config(H, W, C, b, R, K, precision, flags)
        self.R, self.K, self.b, self.B = R, K, b, R * b
        self.bf16 = precision == SB_BF16
        self.device = torch.device(device)
        self._larr = _layers_array(self.layers)
        need = c_size_t(0)
        _check(sb_model_bytes(self._larr, len(self.layers), byref(self.cfg), byref(need)))
        self.arena_bytes = need.value
        torch.cuda.set_device(self.device)
        self.arena = torch.empty(need.value + 256, dtype=torch.uint8, device=self.device)
        base = (self.arena.data_ptr() + 255) // 256 * 256
        h = c_void_p()
        _check(sb_model_create(self._larr, len(self.layers), byref(self.cfg), c_void_p(base), need.value, byref(h)))
        self.h = h
        self._keep = None

    def close(self):
        if self.h:
            sb_model_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def from_workload(wl, precision=SB_BF16, flags=0, device="cuda:0"):
        return Model(wl.layers, wl.H, wl.W, wl.C, wl.b, wl.R, wl.K, precision, flags, device)

    def _stream(self):
        return c_void_p(self.torch.cuda.current_stream().cuda_stream)

    def _ptr_arrays(self, xs, labels):
        xp = lp = None
        if xs is not None:
            assert len(xs) == self.R
            xp = (c_void_p * self.R)(*[c_void_p(t.data_ptr()) for t in xs])
        if labels is not None:
            assert len(labels) == self.R
            lp = (c_void_p * self.R)(*[c_void_p(t.data_ptr()) for t in labels])
        self._keep = (xs, labels)
        return xp, lp

    # ---- the iteration -----------------------------------------------------------------------
    def forward(self, xs, labels):
        """xs: R device tensors [b,H,W,C] (float32 or bfloat16 to match the precision); labels: R int32 [b]."""
        xp, lp = self._ptr_arrays(xs, labels)
        _check(sb_forward(self.h, xp, lp, self._stream()))

    def backward(self):
        _check(sb_backward(self.h, self._stream()))

    def graph_step(self, xs, labels, lr, momentum):
        """forward + backward + sgd_step as one CUDA-graph launch (captured by the library on the second call)."""
        xp, lp = self._ptr_arrays(xs, labels)
        _check(sb_graph_step(self.h, xp, lp, c_float(lr), c_float(momentum), self._stream()))

    def modulo_step(self, xs, labels, lr, momentum):
        """One iteration in the modulo layer's sub-iteration schedule (model created with SB_FLAG_MODULO_SCHEDULE)."""
        xp, lp = self._ptr_arrays(xs, labels)
        _check(sb_modulo_step(self.h, xp, lp, c_float(lr), c_float(momentum), self._stream()))

    def debug_wait_probe(self, limit_ms=20):
        """Enqueue the bounded-wait self-test; the next loss() raises SB_ERR_TIMEOUT."""
        _check(sb_debug_wait_probe(self.h, c_int32(limit_ms), self._stream()))

    def sgd_step(self, lr, momentum):
        _check(sb_sgd_step(self.h, c_float(lr), c_float(momentum), self._stream()))

    def loss(self) -> float:
        v = c_float()
        _check(sb_loss(self.h, self._stream(), byref(v)))
        return v.value

    def train_step_host(self, host_x, host_labels, lr, momentum) -> float:
        """host_x / host_labels: CPU torch tensors (pinned for async copies) or numpy arrays."""
        v = c_float()
        px = host_x.data_ptr() if hasattr(host_x, "data_ptr") else host_x.ctypes.data
        pl = host_labels.data_ptr() if hasattr(host_labels, "data_ptr") else host_labels.ctypes.data
        _check(sb_train_step_host(self.h, c_void_p(px), c_void_p(pl), c_float(lr), c_float(momentum), self._stream(), byref(v)))
        return v.value

    def prefetch_host(self, host_x, host_labels):
        """Start the host->device copy of a later iteration's inputs (consumed by the next train_step_host on the same buffers)."""
        px = host_x.data_ptr() if hasattr(host_x, "data_ptr") else host_x.ctypes.data
        pl = host_labels.data_ptr() if hasattr(host_labels, "data_ptr") else host_labels.ctypes.data
        _check(sb_prefetch_host(self.h, c_void_p(px), c_void_p(pl)))

    def train_step_host_async(self, host_x, host_labels, lr, momentum):
        """Launch an iteration on a staged batch without waiting; collect its loss with train_step_host_wait()."""
        px = host_x.data_ptr() if hasattr(host_x, "data_ptr") else host_x.ctypes.data
        pl = host_labels.data_ptr() if hasattr(host_labels, "data_ptr") else host_labels.ctypes.data
        _check(sb_train_step_host_async(self.h, c_void_p(px), c_void_p(pl), c_float(lr), c_float(momentum), self._stream()))

    def train_step_host_wait(self) -> float:
        """Loss of the oldest iteration in flight (blocks until it has finished)."""
        v = c_float()
        _check(sb_train_step_host_wait(self.h, self._stream(), byref(v)))
        return v.value

    def forward_layers(self, first, last, xs=None, labels=None):
        xp, lp = self._ptr_arrays(xs, labels)
        _check(sb_forward_layers(self.h, first, last, xp, lp, self._stream()))

    def backward_layers(self, last, first):
        _check(sb_backward_layers(self.h, last, first, self._stream()))

    def refresh_shadow(self):
        _check(sb_refresh_shadow(self.h, self._stream()))

    def dropout_seed(self, seed, iteration=0):
        _check(sb_dropout_seed(self.h, ctypes.c_uint64(seed), ctypes.c_uint64(iteration), self._stream()))

    # ---- introspection -----------------------------------------------------------------------
    def tensor_info(self, what, layer, part=0):
        p = c_void_p()
        shape = (c_int64 * 4)()
        dt = c_int32()
        _check(sb_tensor(self.h, what, layer, part, byref(p), shape, byref(dt)))
        return p.value, tuple(shape), dt.value

    def read(self, what, layer, part=0, squeeze=True) -> np.ndarray:
        """Tensor as numpy; bfloat16 tensors come back converted to float32."""
        _, shape, dt = self.tensor_info(what, layer, part)
        a = np.empty(shape, _NP_DT[dt])
        _check(sb_tensor_read(self.h, what, layer, part, c_void_p(a.ctypes.data), a.nbytes))
        if dt == SB_DT_BF16:
            a = bf16_bits_to_f32(a)
        if squeeze:
            while a.ndim > 1 and a.shape[-1] == 1:
                a = a[..., 0]
        return a

    def write(self, what, layer, part, value: np.ndarray):
        """value: float array (converted to the tensor's dtype, RNE for bfloat16) or uint8."""
        _, shape, dt = self.tensor_info(what, layer, part)
        n = int(np.prod(shape))
        assert value.size == n, (value.shape, shape)
        if dt == SB_DT_BF16:
            a = f32_to_bf16_bits(np.asarray(value, np.float32).reshape(-1))
        else:
            a = np.ascontiguousarray(np.asarray(value).reshape(-1), dtype=_NP_DT[dt])
        _check(sb_tensor_write(self.h, what, layer, part, c_void_p(a.ctypes.data), a.nbytes))

    def load_params(self, full_params, bounds_fn):
        """Logical (unpartitioned) parameters -> replicated conv tensors and K FC shards.
        bounds_fn(out, K) gives the shard boundaries (data marshalling only)."""
        for li, ((kind, out), p) in enumerate(zip(self.layers, full_params)):
            if kind == SB_CONV3X3_RELU:
                self.write(SB_T_WEIGHT, li, 0, p["w"])
                self.write(SB_T_BIAS, li, 0, p["b"])
            elif kind in (SB_FC_RELU, SB_FC, SB_FC_RELU_WHOLE, SB_FC_WHOLE):
                K = self.K if kind in (SB_FC_RELU, SB_FC) else 1       # a layer kept whole has one shard
                cb = bounds_fn(out, K)
                for j in range(K):
                    self.write(SB_T_WEIGHT, li, j, p["w"][cb[j]:cb[j + 1]])
                    self.write(SB_T_BIAS, li, j, p["b"][cb[j]:cb[j + 1]])
        self.refresh_shadow()
        self.torch.cuda.synchronize()

    def gather_params(self, what_w, what_b):
        """Reassemble logical tensors (weights, grads or momentum) from the shards, as numpy."""
        out = []
        for li, (kind, _) in enumerate(self.layers):
            if kind == SB_CONV3X3_RELU:
                out.append({"w": self.read(what_w, li, 0, squeeze=False), "b": self.read(what_b, li, 0)})
            elif kind in (SB_FC_RELU, SB_FC, SB_FC_RELU_WHOLE, SB_FC_WHOLE):
                K = self.K if kind in (SB_FC_RELU, SB_FC) else 1
                ws = [self.read(what_w, li, j, squeeze=False)[:, :, 0, 0] for j in range(K)]
                bs = [self.read(what_b, li, j, squeeze=False)[:, 0, 0, 0] for j in range(K)]
                out.append({"w": np.concatenate(ws, 0), "b": np.concatenate(bs, 0)})
            else:
                out.append(None)
        return out

    def debug_poison(self):
        _check(sb_debug_poison(self.h, self._stream()))

    def debug_check_guards(self):
        """(number of damaged guard regions, arena offset of the first damaged byte or -1)"""
        n, off = c_int32(), c_int64()
        _check(sb_debug_check_guards(self.h, self._stream(), byref(n), byref(off)))
        return n.value, off.value

    def param_bytes(self, shard=0) -> int:
        v = c_size_t()
        _check(sb_param_bytes(self.h, shard, byref(v)))
        return v.value

    def profile_begin(self):
        _check(sb_profile_begin(self.h, self._stream()))

    def profile_end(self):
        """Per kernel class: {'name', 'launches', 'ms_total', 'flops', 'bytes'} (algorithmic work)."""
        arr = (sb_profile_entry * 256)()
        n = c_int32()
        _check(sb_profile_end(self.h, self._stream(), arr, 256, byref(n)))
        return [dict(name=arr[i].name.decode(), launches=arr[i].launches, ms_total=arr[i].ms_total,
                     flops=arr[i].flops, bytes=arr[i].bytes) for i in range(n.value)]

    def launch_count(self) -> int:
        v = c_int64()
        _check(sb_launch_count(self.h, byref(v)))
        return v.value
