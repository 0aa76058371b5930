"""Python binding of the ResIST CUDA library (libresist.so): argument marshalling only.

Every step of the path (partition scatter, sub-ResNet forward/backward, SGD update, reassembly,
evaluation) runs in the library's CUDA kernels; torch supplies device memory and streams.
There is no CPU fallback: importing works without a GPU, but creating a context does not.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

RESIST_OK = 0
F32, BF16 = 0, 1
CONV_AUTO, CONV_CUDA_CORES, CONV_TCGEN05, CONV_WARP_MMA, CONV_WARP_MMA_UNFUSED = 0, 1, 2, 3, 4
MOMENTUM_RESTART, MOMENTUM_KEEP = 0, 1
_STATUS = {0: "RESIST_OK", -1: "RESIST_EINVAL", -2: "RESIST_ESTATE", -3: "RESIST_ENOMEM", -4: "RESIST_ECUDA",
           -5: "RESIST_ETIMEOUT", -6: "RESIST_EUNSUPPORTED"}


class ResistError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{_STATUS.get(code, code)}: {msg}")
        self.code = code


class _Block(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "stage", "cin", "cmid", "cout", "stride", "has_projection", "partitionable")]


class _Arch(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("in_h", "in_w", "in_c", "classes", "stem_k", "stem_stride", "stem_cout",
                                           "stem_bn_relu", "stem_maxpool", "num_blocks")] + [("blocks", C.POINTER(_Block))]


class _Opts(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("momentum", C.c_float), ("weight_decay", C.c_float), ("bn_eps", C.c_float),
                ("bn_momentum", C.c_float), ("min_depth", C.c_int32), ("momentum_policy", C.c_int32),
                ("conv_backend", C.c_int32), ("bn_stat_period", C.c_int32)]


_ALLOC_FN = C.CFUNCTYPE(C.c_void_p, C.c_void_p, C.c_size_t)
_FREE_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_void_p)


class _Allocator(C.Structure):
    _fields_ = [("alloc", _ALLOC_FN), ("release", _FREE_FN), ("user", C.c_void_p)]


class _ProfileEntry(C.Structure):
    _fields_ = [("name", C.c_char * 32), ("launches", C.c_int64), ("operations", C.c_int64), ("ms", C.c_double),
                ("bytes", C.c_double), ("flops", C.c_double)]


class _StepInfo(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("kernel_launches", "conv_flops", "tensor_core_convs", "cuda_core_convs",
                                           "workspace_bytes")]


_lib = None


def lib():
    """Loads (building if stale) libresist.so.  Raises if it cannot be built or loaded."""
    global _lib
    if _lib is None:
        so = _build.build()
        L = C.CDLL(so)
        P, I, F, U64 = C.c_void_p, C.c_int32, C.c_float, C.c_uint64
        L.resist_init.argtypes = [C.POINTER(_Arch), C.POINTER(_Opts), U64, C.POINTER(_Allocator), C.POINTER(P)]
        L.resist_destroy.argtypes = [P]
        L.resist_partition.argtypes = [P, U64, I, P, P]
        L.resist_local_step.argtypes = [P, I, P, P, I, F, P, P]
        L.resist_local_step_grouped.argtypes = [P, P, P, I, F, P, P]
        L.resist_aggregate.argtypes = [P, P]
        L.resist_eval.argtypes = [P, P, P, I, P, P, P, P]
        L.resist_param_count.argtypes = [P, C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.resist_get_params.argtypes = [P, I, P, P]
        L.resist_set_params.argtypes = [P, P, P]
        L.resist_get_grads.argtypes = [P, I, P]
        L.resist_get_logits.argtypes = [P, I, P]
        L.resist_get_shadow.argtypes = [P, I, P]
        L.resist_debug_set_wait_status.argtypes = [I]
        L.resist_micro_mma_rate.argtypes = [I, I, I, I, I, C.POINTER(C.c_double)]
        L.resist_get_step_info.argtypes = [P, C.POINTER(_StepInfo)]
        L.resist_splitmix64.argtypes = [U64, C.c_int64, P]
        L.resist_splitmix64.restype = None
        L.resist_set_profiling.argtypes = [P, I]
        L.resist_get_profile.argtypes = [P, P, I, P]
        L.resist_conv2d.argtypes = [I, I, I, P, P, P, P, I, I, I, I, I, I, I, F, P, P]
        L.resist_conv2d_bn_relu.argtypes = [I, I, P, P, P, P, I, I, I, I, I, I, I, F, P, P, P, P, P, P, P, P, P, P, F, F, P, P]
        L.resist_bn_relu_forward.argtypes = [I, P, P, P, P, P, P, P, C.c_int64, I, F, F, P]
        L.resist_bn_relu_backward.argtypes = [I, P, P, P, P, P, P, P, P, P, C.c_int64, I, P]
        L.resist_layer_last_error.restype = C.c_char_p
        L.resist_bn_relu_forward_noalloc.argtypes = [I, P, P, P, P, P, P, P, C.c_int64, I, F, F, P]
        L.resist_noalloc_last_error.restype = C.c_char_p
        L.resist_last_error.argtypes = [P]
        L.resist_last_error.restype = C.c_char_p
        _lib = L
    return _lib


EXPORTS = ["resist_init", "resist_destroy", "resist_partition", "resist_local_step", "resist_local_step_grouped",
           "resist_aggregate", "resist_eval", "resist_param_count", "resist_get_params", "resist_set_params",
           "resist_get_grads", "resist_get_logits", "resist_get_shadow", "resist_debug_set_wait_status", "resist_micro_mma_rate", "resist_get_step_info", "resist_splitmix64", "resist_last_error",
           "resist_set_profiling", "resist_get_profile", "resist_conv2d", "resist_conv2d_bn_relu", "resist_bn_relu_forward", "resist_bn_relu_backward", "resist_layer_last_error",
           "resist_bn_relu_forward_noalloc", "resist_noalloc_last_error"]


def resist_splitmix64(seed: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.uint64)
    lib().resist_splitmix64(seed & 0xFFFFFFFFFFFFFFFF, n, out.ctypes.data)
    return out


def _stream_handle(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def _odim(h, k, s):
    return (h + 2 * ((k - 1) // 2) - k) // s + 1


def _layer_check(rc):
    if rc != RESIST_OK:
        raise ResistError(rc, lib().resist_layer_last_error().decode())


def _dt(t: torch.Tensor) -> int:
    return {torch.float32: F32, torch.bfloat16: BF16}[t.dtype]


def resist_conv2d(mode: int, act: torch.Tensor, wgt: torch.Tensor, geom, add: Optional[torch.Tensor] = None,
                  scale: float = 1.0, backend: int = CONV_AUTO, stream=None):
    """geom = (N, H, W, C, K, ksz, stride) of the forward convolution.  Returns (out, family) with family 0 = CUDA cores, 1 = tcgen05, 2 = warp-level MMA."""
    N, H, W, Cc, K, ksz, stride = geom
    P, Q = _odim(H, ksz, stride), _odim(W, ksz, stride)
    if mode == 0:
        out = torch.empty(N, P, Q, K, dtype=act.dtype, device=act.device)
    elif mode == 1:
        out = torch.empty(N, H, W, Cc, dtype=act.dtype, device=act.device)
    else:
        out = torch.empty(K, ksz, ksz, Cc, dtype=torch.float32, device=act.device)
    used = C.c_int32(0)
    _layer_check(lib().resist_conv2d(mode, _dt(act), backend, act.data_ptr(), wgt.data_ptr(),
                                     add.data_ptr() if add is not None else None, out.data_ptr(), N, H, W, Cc, K, ksz,
                                     stride, scale, C.addressof(used), _stream_handle(stream)))
    return out, int(used.value)


def micro_mma_rate(n: int, layout: int, reps: int = 4096, issuers: int = 1, alternate: int = 0) -> float:
    """SM clocks per tcgen05 MMA of shape 128 x n x 16 (see resist.h)."""
    out = C.c_double(0.0)
    rc = lib().resist_micro_mma_rate(n, layout, reps, issuers, alternate, C.byref(out))
    if rc:
        raise ResistError(rc, "resist_micro_mma_rate failed")
    return float(out.value)


def resist_conv2d_bn_relu(mode: int, act: torch.Tensor, wgt: torch.Tensor, geom, gamma, beta, stat=None, x=None, add=None, bn_add=None,
                          run_mean=None, run_var=None, scale: float = 1.0, eps=1e-5, momentum=0.1, backend: int = CONV_AUTO, stream=None):
    """The convolution and the BN+ReLU that consumes its output, as one call (see resist.h).  mode 0 returns (y, a, stat, family);
    mode 1 returns (da, dx, dgamma, dbeta, family)."""
    N, H, W, Cc, K, ksz, stride = geom
    P, Q = _odim(H, ksz, stride), _odim(W, ksz, stride)
    dev = act.device
    ptr = lambda t: t.data_ptr() if t is not None else None
    used = C.c_int32(0)
    if mode == 0:
        out = torch.empty(N, P, Q, K, dtype=act.dtype, device=dev)
        stat = torch.zeros(4 * K, dtype=torch.float32, device=dev)
        dg = db = None
    else:
        out = torch.empty(N, H, W, Cc, dtype=act.dtype, device=dev)
        dg, db = torch.zeros(Cc, dtype=torch.float32, device=dev), torch.zeros(Cc, dtype=torch.float32, device=dev)
    bn_out = torch.empty_like(out)
    _layer_check(lib().resist_conv2d_bn_relu(mode, backend, act.data_ptr(), wgt.data_ptr(), ptr(add), out.data_ptr(), N, H, W, Cc, K, ksz, stride,
                                             scale, ptr(x), gamma.data_ptr(), beta.data_ptr(), stat.data_ptr(), ptr(run_mean), ptr(run_var),
                                             ptr(bn_add), bn_out.data_ptr(), ptr(dg), ptr(db), eps, momentum, C.addressof(used),
                                             _stream_handle(stream)))
    if mode == 0:
        return out, bn_out, stat, int(used.value)
    return out, bn_out, dg, db, int(used.value)


def resist_bn_relu_forward(x: torch.Tensor, gamma, beta, run_mean=None, run_var=None, eps=1e-5, momentum=0.1, stream=None):
    Cc = x.shape[-1]
    m = x.numel() // Cc
    a = torch.empty_like(x)
    stat = torch.zeros(4 * Cc, dtype=torch.float32, device=x.device)
    _layer_check(lib().resist_bn_relu_forward(_dt(x), x.data_ptr(), gamma.data_ptr(), beta.data_ptr(), a.data_ptr(),
                                              stat.data_ptr(), run_mean.data_ptr() if run_mean is not None else None,
                                              run_var.data_ptr() if run_var is not None else None, m, Cc, eps, momentum,
                                              _stream_handle(stream)))
    return a, stat


def resist_bn_relu_forward_noalloc(x: torch.Tensor, gamma, beta, a: torch.Tensor, stat: torch.Tensor, run_mean=None,
                                   run_var=None, eps=1e-5, momentum=0.1, stream=None):
    """resist_bn_relu_forward without any device allocation: the caller passes the output `a` (shape of x) and
    `stat` (float32 [4*C]) too, and the reduction scratch is a fixed array inside the library (see the header for
    its limit).  Enqueues on the stream and returns; calls must not overlap on the GPU."""
    Cc = x.shape[-1]
    m = x.numel() // Cc
    rc = lib().resist_bn_relu_forward_noalloc(_dt(x), x.data_ptr(), gamma.data_ptr(), beta.data_ptr(), a.data_ptr(),
                                              stat.data_ptr(), run_mean.data_ptr() if run_mean is not None else None,
                                              run_var.data_ptr() if run_var is not None else None, m, Cc, eps, momentum,
                                              _stream_handle(stream))
    if rc != RESIST_OK:
        raise ResistError(rc, lib().resist_noalloc_last_error().decode())


def resist_bn_relu_backward(x, da, gamma, beta, stat, add=None, stream=None):
    Cc = x.shape[-1]
    m = x.numel() // Cc
    dx = torch.empty_like(x)
    dg = torch.empty(Cc, dtype=torch.float32, device=x.device)
    db = torch.empty(Cc, dtype=torch.float32, device=x.device)
    _layer_check(lib().resist_bn_relu_backward(_dt(x), x.data_ptr(), da.data_ptr(), gamma.data_ptr(), beta.data_ptr(),
                                               stat.data_ptr(), add.data_ptr() if add is not None else None, dx.data_ptr(),
                                               dg.data_ptr(), db.data_ptr(), m, Cc, _stream_handle(stream)))
    return dx, dg, db


class Context:
    """A global ResNet plus its S working copies on one GPU (resist_ctx)."""

    def __init__(self, arch_int32: np.ndarray, dtype: int = F32, momentum: float = 0.9, weight_decay: float = 0.0,
                 bn_eps: float = 1e-5, bn_momentum: float = 0.1, min_depth: int = 0,
                 momentum_policy: int = MOMENTUM_RESTART, conv_backend: int = CONV_AUTO, seed: int = 0,
                 device: str = "cuda:0", bn_stat_period: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("the ResIST library needs a CUDA device; there is no CPU path")
        self._lib = lib()
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        a = np.asarray(arch_int32, dtype=np.int32)
        nb = int(a[9])
        self._blocks = (_Block * max(nb, 1))()
        for i in range(nb):
            for j, (name, _) in enumerate(_Block._fields_):
                setattr(self._blocks[i], name, int(a[10 + 8 * i + j]))
        arch = _Arch(*[int(v) for v in a[:10]], C.cast(self._blocks, C.POINTER(_Block)))
        opts = _Opts(dtype, momentum, weight_decay, bn_eps, bn_momentum, min_depth, momentum_policy, conv_backend, bn_stat_period)
        # device memory comes from torch's caching allocator
        self._held = {}

        def _alloc(_user, nbytes):
            try:
                t = torch.empty(int(nbytes), dtype=torch.uint8, device=self.device)
            except RuntimeError:
                return None
            self._held[t.data_ptr()] = t
            return t.data_ptr()

        def _free(_user, ptr):
            self._held.pop(ptr, None)

        self._alloc_cb, self._free_cb = _ALLOC_FN(_alloc), _FREE_FN(_free)
        self._allocator = _Allocator(self._alloc_cb, self._free_cb, None)
        self._ctx = C.c_void_p()
        rc = self._lib.resist_init(C.byref(arch), C.byref(opts), seed & 0xFFFFFFFFFFFFFFFF, C.byref(self._allocator),
                                   C.byref(self._ctx))
        if rc != RESIST_OK:
            raise ResistError(rc, self._lib.resist_last_error(None).decode())
        self.dtype = dtype
        self.classes = int(a[3])
        self.num_blocks = nb
        n, nbuf = C.c_int64(), C.c_int64()
        self._lib.resist_param_count(self._ctx, C.byref(n), C.byref(nbuf))
        self.n_params, self.n_buffers = n.value, nbuf.value
        self.S = 0

    # ---- helpers
    def _check(self, rc: int):
        if rc != RESIST_OK:
            raise ResistError(rc, self._lib.resist_last_error(self._ctx).decode())

    def close(self):
        if getattr(self, "_ctx", None) and self._ctx.value:
            self._lib.resist_destroy(self._ctx)
            self._ctx = C.c_void_p()
            self._held.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def act_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == BF16 else torch.float32

    def _images(self, t: torch.Tensor) -> torch.Tensor:
        assert t.is_cuda and t.dtype == self.act_dtype and t.is_contiguous(), "images: contiguous NHWC on the GPU, library dtype"
        return t

    # ---- the protocol
    def partition(self, round_seed: int, S: int, stream=None) -> np.ndarray:
        mask = np.zeros(max(self.num_blocks, 1), dtype=np.uint32)
        self._check(self._lib.resist_partition(self._ctx, round_seed & 0xFFFFFFFFFFFFFFFF, S, mask.ctypes.data,
                                               _stream_handle(stream)))
        self.S = S
        return mask[:self.num_blocks]

    def local_step(self, subnet: int, images: torch.Tensor, labels: torch.Tensor, lr: float,
                   loss_out: Optional[torch.Tensor] = None, stream=None):
        self._images(images)
        assert labels.is_cuda and labels.dtype == torch.int32
        self._check(self._lib.resist_local_step(self._ctx, subnet, images.data_ptr(), labels.data_ptr(), images.shape[0],
                                                lr, loss_out.data_ptr() if loss_out is not None else None,
                                                _stream_handle(stream)))

    def local_step_grouped(self, images: Sequence[torch.Tensor], labels: Sequence[torch.Tensor], lr: float,
                           loss_out: Optional[torch.Tensor] = None, stream=None):
        S = len(images)
        assert S == self.S and len(labels) == S
        ip = (C.c_void_p * S)(*[self._images(t).data_ptr() for t in images])
        lp = (C.c_void_p * S)(*[t.data_ptr() for t in labels])
        self._check(self._lib.resist_local_step_grouped(self._ctx, ip, lp, images[0].shape[0], lr,
                                                        loss_out.data_ptr() if loss_out is not None else None,
                                                        _stream_handle(stream)))

    def aggregate(self, stream=None):
        self._check(self._lib.resist_aggregate(self._ctx, _stream_handle(stream)))

    def eval(self, images: torch.Tensor, labels: Optional[torch.Tensor] = None, stream=None):
        """Returns (logits [B, classes] float32 cuda, loss float tensor [1], correct int32 tensor [1])."""
        self._images(images)
        B = images.shape[0]
        logits = torch.empty(B, self.classes, dtype=torch.float32, device=self.device)
        loss = torch.zeros(1, dtype=torch.float32, device=self.device)
        correct = torch.zeros(1, dtype=torch.int32, device=self.device)
        self._check(self._lib.resist_eval(self._ctx, images.data_ptr(), labels.data_ptr() if labels is not None else None,
                                          B, logits.data_ptr(), loss.data_ptr(), correct.data_ptr(), _stream_handle(stream)))
        return logits, loss, correct

    # ---- taps
    def get_params(self, subnet: int = -1):
        p = np.empty(self.n_params, dtype=np.float32)
        b = np.empty(self.n_buffers, dtype=np.float32)
        self._check(self._lib.resist_get_params(self._ctx, subnet, p.ctypes.data, b.ctypes.data))
        return p, b

    def set_params(self, params: Optional[np.ndarray], buffers: Optional[np.ndarray] = None):
        p = np.ascontiguousarray(params, dtype=np.float32) if params is not None else None
        b = np.ascontiguousarray(buffers, dtype=np.float32) if buffers is not None else None
        assert p is None or p.size == self.n_params
        assert b is None or b.size == self.n_buffers
        self._check(self._lib.resist_set_params(self._ctx, p.ctypes.data if p is not None else None,
                                                b.ctypes.data if b is not None else None))

    def get_grads(self, subnet: int) -> np.ndarray:
        g = np.empty(self.n_params, dtype=np.float32)
        self._check(self._lib.resist_get_grads(self._ctx, subnet, g.ctypes.data))
        return g

    def get_logits(self, subnet: int, B: int) -> np.ndarray:
        out = np.empty((B, self.classes), dtype=np.float32)
        self._check(self._lib.resist_get_logits(self._ctx, subnet, out.ctypes.data))
        return out

    def get_shadow(self, subnet: int) -> np.ndarray:
        """bf16 bit patterns (uint16) of the convolutions' copy of a sub-ResNet's parameters, flat order."""
        out = np.empty(self.n_params, dtype=np.uint16)
        self._check(self._lib.resist_get_shadow(self._ctx, subnet, out.ctypes.data))
        return out

    def set_profiling(self, on: bool):
        self._check(self._lib.resist_set_profiling(self._ctx, 1 if on else 0))

    def get_profile(self) -> dict:
        """{family: dict(launches, operations, ms, bytes, flops)} since the last read; clears the counters."""
        arr = (_ProfileEntry * 96)()
        n = C.c_int32(0)
        self._check(self._lib.resist_get_profile(self._ctx, C.addressof(arr), 96, C.addressof(n)))
        return {arr[i].name.decode(): {"launches": arr[i].launches, "operations": arr[i].operations, "ms": arr[i].ms,
                                       "bytes": arr[i].bytes, "flops": arr[i].flops} for i in range(min(n.value, 96))}

    def step_info(self) -> dict:
        s = _StepInfo()
        self._check(self._lib.resist_get_step_info(self._ctx, C.byref(s)))
        return {n: getattr(s, n) for n, _ in _StepInfo._fields_}


def resist_init(arch_int32: np.ndarray, **kw) -> Context:
    return Context(arch_int32, **kw)
