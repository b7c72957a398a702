"""Python binding of libchoco (the CHOCO-Gossip / CHOCO-SGD step on one B200).

Argument marshalling only: every function forwards to the C entry point of the same
name in ``libchoco.so`` (declared in ``include/choco.h``); all arithmetic runs in the
library's CUDA kernels.  PyTorch tensors are used for device memory and streams.
There is no CPU path: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libchoco.so")

Q_IDENTITY, Q_TOPK, Q_RANDK, Q_QSGD, Q_SIGN = 0, 1, 2, 3, 4
Q_KINDS = {"identity": Q_IDENTITY, "topk": Q_TOPK, "randk": Q_RANDK, "qsgd": Q_QSGD, "sign": Q_SIGN}

EXPORTS = [
    "choco_init", "choco_destroy", "choco_gossip_step", "choco_sgd_step",
    "choco_sgd_momentum_step", "choco_sgd_step_host", "choco_invalidate", "choco_set_carry",
    "choco_get_step", "choco_set_graphs", "choco_set_rescue", "choco_set_select_blocks", "choco_set_nesterov",
    "choco_set_step", "choco_message_bytes", "choco_get_message", "choco_read_message",
    "choco_consensus_error", "choco_consensus_error_noalloc",
    "choco_get_stats", "choco_profile_enable", "choco_profile_set_stride", "choco_profile_read", "choco_strerror",
    "choco_last_cuda_error", "choco_debug_set_wait_polls", "choco_debug_set_candidate_slot",
    "choco_layers_init", "choco_layers_destroy", "choco_layers_gossip_step", "choco_layers_sgd_step",
    "choco_layers_sgd_momentum_step", "choco_layers_message_bytes", "choco_layers_get_layer",
    "choco_layers_invalidate", "choco_layers_set_step", "choco_layers_set_nesterov", "choco_layers_set_graphs", "choco_layers_combined_steps",
]


ERR_TIMEOUT = -8


class ChocoError(RuntimeError):
    """A libchoco call returned a negative status; `code` holds it."""

    def __init__(self, message: str, code: int = 0):
        super().__init__(message)
        self.code = code


class choco_params(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("s", ctypes.c_int32), ("bucket", ctypes.c_int32),
                ("qsgd_biased", ctypes.c_int32), ("k", ctypes.c_int64)]


class choco_stats(ctypes.Structure):
    _fields_ = [("steps", ctypes.c_uint64), ("prepared_rows", ctypes.c_uint64),
                ("recompressed_rows", ctypes.c_uint64), ("exact_rows", ctypes.c_uint64),
                ("kernel_launches", ctypes.c_uint64), ("device_timeouts", ctypes.c_uint64),
                ("graph_replays", ctypes.c_uint64), ("rescued_rows", ctypes.c_uint64)]


_lib = None


def load() -> ctypes.CDLL:
    """dlopen libchoco.so; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ChocoError(f"{LIB_PATH} is missing: run `python -m paper_1907_09356_b200.build` "
                             "(there is no fallback implementation)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, u64, f32 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64,
                                  ctypes.c_float)
        lib.choco_init.argtypes = [ctypes.POINTER(vp), i32, i64, i64, vp, vp, vp,
                                   ctypes.POINTER(choco_params), u64]
        lib.choco_destroy.argtypes = [vp]
        lib.choco_gossip_step.argtypes = [vp, vp, vp, vp, f32, vp]
        lib.choco_sgd_step.argtypes = [vp, vp, vp, vp, vp, f32, f32, vp]
        lib.choco_sgd_momentum_step.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, f32, f32, vp]
        lib.choco_sgd_step_host.argtypes = [vp, vp, vp, vp, vp, f32, f32, vp]
        lib.choco_invalidate.argtypes = [vp]
        lib.choco_set_carry.argtypes = [vp, i32]
        lib.choco_set_graphs.argtypes = [vp, i32]
        lib.choco_set_rescue.argtypes = [vp, i32]
        lib.choco_set_select_blocks.argtypes = [vp, i32]
        lib.choco_set_nesterov.argtypes = [vp, i32]
        lib.choco_debug_set_candidate_slot.argtypes = [vp, i32]
        lib.choco_get_step.argtypes = [vp, ctypes.POINTER(u64)]
        lib.choco_set_step.argtypes = [vp, u64]
        lib.choco_message_bytes.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        lib.choco_get_message.argtypes = [vp, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(i64)]
        lib.choco_read_message.argtypes = [vp, i32, i32, vp, i64, ctypes.POINTER(i64), vp]
        lib.choco_consensus_error.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_double), vp]
        lib.choco_consensus_error_noalloc.argtypes = [vp, i32, i64, i64, vp, vp]
        lib.choco_get_stats.argtypes = [vp, ctypes.POINTER(choco_stats), vp]
        lib.choco_profile_enable.argtypes = [vp, i32]
        lib.choco_profile_set_stride.argtypes = [vp, i32]
        lib.choco_profile_read.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double), vp]
        lib.choco_strerror.argtypes = [ctypes.c_int]
        lib.choco_strerror.restype = ctypes.c_char_p
        lib.choco_last_cuda_error.argtypes = [vp]
        lib.choco_debug_set_wait_polls.argtypes = [vp, ctypes.c_uint32]
        lib.choco_layers_init.argtypes = [ctypes.POINTER(vp), i32, i32, vp, i64, vp, vp, vp,
                                          ctypes.POINTER(choco_params), i64, i64, u64]
        lib.choco_layers_destroy.argtypes = [vp]
        lib.choco_layers_gossip_step.argtypes = [vp, vp, vp, vp, f32, vp]
        lib.choco_layers_sgd_step.argtypes = [vp, vp, vp, vp, vp, f32, f32, vp]
        lib.choco_layers_sgd_momentum_step.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, f32, f32, vp]
        lib.choco_layers_message_bytes.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        lib.choco_layers_get_layer.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(i64),
                                               ctypes.POINTER(i64)]
        lib.choco_layers_invalidate.argtypes = [vp]
        lib.choco_layers_set_step.argtypes = [vp, u64]
        lib.choco_layers_set_nesterov.argtypes = [vp, i32]
        lib.choco_layers_set_graphs.argtypes = [vp, i32, ctypes.POINTER(u64)]
        lib.choco_layers_combined_steps.argtypes = [vp, ctypes.POINTER(u64)]
        for name in EXPORTS:
            if name not in ("choco_strerror",):
                getattr(lib, name).restype = ctypes.c_int
        _lib = lib
    return _lib


def _check(rc: int, ctx=None) -> None:
    if rc != 0:
        lib = load()
        msg = lib.choco_strerror(rc).decode()
        if ctx is not None and rc == -4:
            msg += f" (cudaError {lib.choco_last_cuda_error(ctx)})"
        raise ChocoError(f"libchoco: {msg} [{rc}]", rc)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


# --------------------------------------------------------------------------- C names


def choco_init(n: int, d: int, ld: int, w_row_ptr, w_col, w_val, kind, k: int = 0, s: int = 16,
               bucket: int = 0, qsgd_biased: bool = True, seed: int = 0):
    """W as host numpy arrays (int32, int32, float32).  Returns the context handle."""
    import numpy as np
    rp = np.ascontiguousarray(w_row_ptr, dtype=np.int32)
    col = np.ascontiguousarray(w_col, dtype=np.int32)
    val = np.ascontiguousarray(w_val, dtype=np.float32)
    p = choco_params(Q_KINDS[kind] if isinstance(kind, str) else int(kind), int(s), int(bucket),
                     1 if qsgd_biased else 0, int(k))
    ctx = ctypes.c_void_p()
    _check(load().choco_init(ctypes.byref(ctx), n, d, ld, rp.ctypes.data, col.ctypes.data,
                             val.ctypes.data, ctypes.byref(p), seed))
    return ctx


def choco_destroy(ctx) -> None:
    _check(load().choco_destroy(ctx))


def choco_gossip_step(ctx, X, Xhat, S, gamma: float, stream=None) -> None:
    _check(load().choco_gossip_step(ctx, _ptr(X), _ptr(Xhat), _ptr(S), gamma, _stream(stream)), ctx)


def choco_sgd_step(ctx, X, Xhat, S, G, eta: float, gamma: float, stream=None) -> None:
    _check(load().choco_sgd_step(ctx, _ptr(X), _ptr(Xhat), _ptr(S), _ptr(G), eta, gamma,
                                 _stream(stream)), ctx)


def choco_sgd_momentum_step(ctx, X, Xhat, S, G, M, eta: float, gamma: float, lam: float,
                            beta: float, stream=None) -> None:
    _check(load().choco_sgd_momentum_step(ctx, _ptr(X), _ptr(Xhat), _ptr(S), _ptr(G), _ptr(M), eta,
                                          gamma, lam, beta, _stream(stream)), ctx)


def choco_sgd_step_host(ctx, X, Xhat, S, G, eta: float, gamma: float, stream=None) -> None:
    """X, Xhat, S, G: host tensors (CPU torch tensors or numpy arrays), updated in place."""
    def hp(a):
        if a is None:
            return None
        return a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data
    _check(load().choco_sgd_step_host(ctx, hp(X), hp(Xhat), hp(S), hp(G), eta, gamma,
                                      _stream(stream)), ctx)


def choco_invalidate(ctx) -> None:
    _check(load().choco_invalidate(ctx))


def choco_set_carry(ctx, enable: bool) -> None:
    _check(load().choco_set_carry(ctx, 1 if enable else 0))


def choco_set_graphs(ctx, enable: bool) -> None:
    _check(load().choco_set_graphs(ctx, 1 if enable else 0), ctx)


def choco_set_rescue(ctx, enable: bool) -> None:
    _check(load().choco_set_rescue(ctx, 1 if enable else 0), ctx)


def choco_set_select_blocks(ctx, blocks: int) -> None:
    _check(load().choco_set_select_blocks(ctx, blocks), ctx)


def choco_debug_set_candidate_slot(ctx, slot: int) -> None:
    _check(load().choco_debug_set_candidate_slot(ctx, slot), ctx)


def choco_set_nesterov(ctx, enable: bool) -> None:
    _check(load().choco_set_nesterov(ctx, 1 if enable else 0), ctx)


def choco_get_step(ctx) -> int:
    t = ctypes.c_uint64()
    _check(load().choco_get_step(ctx, ctypes.byref(t)))
    return t.value


def choco_set_step(ctx, t: int) -> None:
    _check(load().choco_set_step(ctx, t))


def choco_message_bytes(ctx) -> tuple[int, int]:
    a, b = ctypes.c_int64(), ctypes.c_int64()
    _check(load().choco_message_bytes(ctx, ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def choco_get_message(ctx, worker: int, plane: int) -> tuple[int, int]:
    """(device pointer, size in bytes) of one plane of a worker's last message."""
    p, nb = ctypes.c_void_p(), ctypes.c_int64()
    _check(load().choco_get_message(ctx, worker, plane, ctypes.byref(p), ctypes.byref(nb)))
    return (p.value or 0), nb.value


def choco_read_message(ctx, worker: int, plane: int, stream=None):
    """One plane of a worker's last message, copied to the host as a numpy uint8 array."""
    import numpy as np
    _, size = choco_get_message(ctx, worker, plane)
    out = np.empty(size, dtype=np.uint8)
    nb = ctypes.c_int64()
    if size:
        _check(load().choco_read_message(ctx, worker, plane, out.ctypes.data, size,
                                         ctypes.byref(nb), _stream(stream)), ctx)
    return out


def choco_consensus_error(ctx, X, stream=None) -> float:
    out = ctypes.c_double()
    _check(load().choco_consensus_error(ctx, _ptr(X), ctypes.byref(out), _stream(stream)), ctx)
    return out.value


def choco_consensus_error_noalloc(X, n: int, d: int, ld: int, out_dev, stream=None) -> None:
    """Consensus distance into `out_dev` (a device tensor holding one float64) without any
    allocation by the library: for callers that must not allocate device memory, e.g. while
    a pool or a capture session owns allocation.  d is limited to 4 194 304; asynchronous."""
    _check(load().choco_consensus_error_noalloc(_ptr(X), n, d, ld, _ptr(out_dev), _stream(stream)))


def choco_get_stats(ctx, stream=None) -> dict:
    st = choco_stats()
    _check(load().choco_get_stats(ctx, ctypes.byref(st), _stream(stream)), ctx)
    return {f: getattr(st, f) for f, _ in choco_stats._fields_}


def choco_debug_set_wait_polls(ctx, polls: int) -> None:
    """Test hook: polls a kernel spends on its first wait for staged copies (0 = give up at once)."""
    _check(load().choco_debug_set_wait_polls(ctx, polls), ctx)


def choco_profile_enable(ctx, max_steps: int) -> None:
    _check(load().choco_profile_enable(ctx, max_steps), ctx)


def choco_profile_set_stride(ctx, stride: int) -> None:
    _check(load().choco_profile_set_stride(ctx, stride), ctx)


def choco_profile_read(ctx, stream=None) -> tuple[int, float]:
    """(steps recorded, total milliseconds spent in the update kernel over them)."""
    n, ms = ctypes.c_int32(), ctypes.c_double()
    _check(load().choco_profile_read(ctx, ctypes.byref(n), ctypes.byref(ms), _stream(stream)), ctx)
    return n.value, ms.value


def choco_layers_init(n: int, layer_off, ld: int, w_row_ptr, w_col, w_val, kind, a_num: int = 1,
                      a_den: int = 1, s: int = 16, bucket: int = 0, qsgd_biased: bool = True,
                      seed: int = 0):
    """Per-layer compression: layer_off is a host array of n_layers + 1 offsets; top-k and
    random-k keep max(1, floor(a_num / a_den * d_l)) entries of layer l."""
    import numpy as np
    off = np.ascontiguousarray(layer_off, dtype=np.int64)
    rp = np.ascontiguousarray(w_row_ptr, dtype=np.int32)
    col = np.ascontiguousarray(w_col, dtype=np.int32)
    val = np.ascontiguousarray(w_val, dtype=np.float32)
    p = choco_params(Q_KINDS[kind] if isinstance(kind, str) else int(kind), int(s), int(bucket),
                     1 if qsgd_biased else 0, 0)
    h = ctypes.c_void_p()
    _check(load().choco_layers_init(ctypes.byref(h), n, len(off) - 1, off.ctypes.data, ld, rp.ctypes.data,
                                    col.ctypes.data, val.ctypes.data, ctypes.byref(p), a_num, a_den, seed))
    return h


def choco_layers_destroy(layers) -> None:
    _check(load().choco_layers_destroy(layers))


def choco_layers_gossip_step(layers, X, Xhat, S, gamma: float, stream=None) -> None:
    _check(load().choco_layers_gossip_step(layers, _ptr(X), _ptr(Xhat), _ptr(S), gamma, _stream(stream)))


def choco_layers_sgd_step(layers, X, Xhat, S, G, eta: float, gamma: float, stream=None) -> None:
    _check(load().choco_layers_sgd_step(layers, _ptr(X), _ptr(Xhat), _ptr(S), _ptr(G), eta, gamma,
                                        _stream(stream)))


def choco_layers_sgd_momentum_step(layers, X, Xhat, S, G, M, eta: float, gamma: float, lam: float,
                                   beta: float, stream=None) -> None:
    _check(load().choco_layers_sgd_momentum_step(layers, _ptr(X), _ptr(Xhat), _ptr(S), _ptr(G), _ptr(M),
                                                 eta, gamma, lam, beta, _stream(stream)))


def choco_layers_message_bytes(layers) -> tuple[int, int]:
    a, b = ctypes.c_int64(), ctypes.c_int64()
    _check(load().choco_layers_message_bytes(layers, ctypes.byref(a), ctypes.byref(b)))
    return a.value, b.value


def choco_layers_get_layer(layers, layer: int):
    """(context handle of the layer, its first coordinate, its length)."""
    c, o, n = ctypes.c_void_p(), ctypes.c_int64(), ctypes.c_int64()
    _check(load().choco_layers_get_layer(layers, layer, ctypes.byref(c), ctypes.byref(o), ctypes.byref(n)))
    return c, o.value, n.value


def choco_layers_set_graphs(layers, enable: int = -1) -> int:
    """Turn the CUDA-graph replay of steady-state steps off (0) / on (1), or leave it (-1);
    returns the number of steps replayed so far."""
    n = ctypes.c_uint64()
    _check(load().choco_layers_set_graphs(layers, enable, ctypes.byref(n)))
    return n.value


def choco_layers_combined_steps(layers) -> int:
    """Step calls so far that were enqueued as launches over all layers at once."""
    n = ctypes.c_uint64()
    _check(load().choco_layers_combined_steps(layers, ctypes.byref(n)))
    return n.value


def choco_layers_invalidate(layers) -> None:
    _check(load().choco_layers_invalidate(layers))


def choco_layers_set_step(layers, t: int) -> None:
    _check(load().choco_layers_set_step(layers, t))


def choco_layers_set_nesterov(layers, enable: bool) -> None:
    _check(load().choco_layers_set_nesterov(layers, 1 if enable else 0))


# --------------------------------------------------------------------------- convenience


@dataclasses.dataclass
class Choco:
    """Owns a context; `w` is any object with n, row_ptr, col, val (host arrays)."""

    w: object
    d: int
    kind: str
    k: int = 0
    s: int = 16
    bucket: int = 0
    qsgd_biased: bool = True
    seed: int = 0
    ld: int = 0

    def __post_init__(self):
        self.ld = self.ld or self.d
        self.ctx = choco_init(self.w.n, self.d, self.ld, self.w.row_ptr, self.w.col, self.w.val,
                              self.kind, self.k, self.s, self.bucket, self.qsgd_biased, self.seed)

    def gossip_step(self, X, Xhat, S, gamma, stream=None):
        choco_gossip_step(self.ctx, X, Xhat, S, gamma, stream)

    def sgd_step(self, X, Xhat, S, G, eta, gamma, stream=None):
        choco_sgd_step(self.ctx, X, Xhat, S, G, eta, gamma, stream)

    def sgd_momentum_step(self, X, Xhat, S, G, M, eta, gamma, lam, beta, stream=None):
        choco_sgd_momentum_step(self.ctx, X, Xhat, S, G, M, eta, gamma, lam, beta, stream)

    def close(self):
        if getattr(self, "ctx", None) is not None:
            choco_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
