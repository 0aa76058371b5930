"""ctypes wrapper around the CPU oracle (oracle/resist_oracle.cpp).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package; the
CUDA library never does.  `build()` compiles the C++ file with g++ -O2 into liboracle.so beside it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "resist_oracle.cpp")
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-shared", "-fPIC", "-o", _SO, _SRC])
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.oracle_partition.argtypes = [C.c_void_p, C.c_uint64, C.c_int, C.c_int, C.c_void_p]
        _lib.oracle_splitmix64.argtypes = [C.c_uint64, C.c_int64, C.c_void_p]
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _suf(dtype) -> str:
    return {np.dtype(np.float32): "f32", np.dtype(np.float64): "f64"}[np.dtype(dtype)]


def splitmix64(seed: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.uint64)
    lib().oracle_splitmix64(C.c_uint64(seed & 0xFFFFFFFFFFFFFFFF), n, _p(out))
    return out


def param_count(arch: np.ndarray):
    n, nb = C.c_int64(), C.c_int64()
    lib().oracle_param_count(_p(arch), C.byref(n), C.byref(nb))
    return n.value, nb.value


def block_ranges(arch: np.ndarray) -> np.ndarray:
    nb = int(arch[9])
    out = np.empty((nb, 4), dtype=np.int64)
    lib().oracle_block_ranges(_p(arch), _p(out))
    return out


def partition(arch: np.ndarray, round_seed: int, S: int, min_depth: int = 0) -> np.ndarray:
    """member_mask[num_blocks] (uint32): bit s set = block is in sub-ResNet s."""
    mask = np.zeros(int(arch[9]), dtype=np.uint32)
    rc = lib().oracle_partition(_p(arch), C.c_uint64(round_seed & 0xFFFFFFFFFFFFFFFF), S, min_depth, _p(mask))
    if rc != 0:
        raise ValueError(f"oracle_partition failed: {rc}")
    return mask


def present_of(mask: np.ndarray, s: int) -> np.ndarray:
    return ((mask >> np.uint32(s)) & np.uint32(1)).astype(np.uint8)


def step(arch, present, params, mom, buffers, images, labels, lr=0.1, mu=0.9, wd=0.0, eps=1e-5,
         bn_mom=0.1, quant=0, do_update=True):
    """One local SGD step of a sub-ResNet.  params, mom, buffers are updated IN PLACE (buffers may be
    None: running statistics are then not tracked).  Returns dict(loss, logits, grads)."""
    dt = params.dtype
    suf = _suf(dt)
    B = images.shape[0]
    images = np.ascontiguousarray(images, dtype=dt)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    present = np.ascontiguousarray(present, dtype=np.uint8)
    grads = np.zeros_like(params)
    logits = np.zeros((B, int(arch[3])), dtype=dt)
    loss = C.c_double()
    fn = getattr(lib(), "oracle_step_" + suf)
    rc = fn(_p(arch), _p(present), _p(params), _p(mom), _p(buffers), _p(images), _p(labels), C.c_int(B),
            C.c_double(lr), C.c_double(mu), C.c_double(wd), C.c_double(eps), C.c_double(bn_mom),
            C.c_int(quant), C.c_int(1 if do_update else 0), _p(grads), _p(logits), C.byref(loss))
    if rc != 0:
        raise ValueError(f"oracle_step failed: {rc}")
    return {"loss": loss.value, "logits": logits, "grads": grads}


def evaluate(arch, params, buffers, S, images, labels, eps=1e-5, quant=0):
    dt = params.dtype
    B = images.shape[0]
    images = np.ascontiguousarray(images, dtype=dt)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    logits = np.zeros((B, int(arch[3])), dtype=dt)
    loss, correct = C.c_double(), C.c_int32()
    fn = getattr(lib(), "oracle_eval_" + _suf(dt))
    fn(_p(arch), _p(params), _p(buffers), C.c_int(S), _p(images), _p(labels), C.c_int(B), C.c_double(eps),
       C.c_int(quant), _p(logits), C.byref(loss), C.byref(correct))
    return {"loss": loss.value, "logits": logits, "correct": correct.value}


def aggregate(arch, member_mask, sub_params: Sequence[np.ndarray], sub_buffers: Optional[Sequence[np.ndarray]],
              global_params: np.ndarray, global_buffers: Optional[np.ndarray]):
    """Reassemble the global parameters (in place in global_params / global_buffers)."""
    S = len(sub_params)
    dt = global_params.dtype
    PP = C.c_void_p * S
    sp = PP(*[s.ctypes.data for s in sub_params])
    sb = PP(*[s.ctypes.data for s in sub_buffers]) if sub_buffers is not None else None
    fn = getattr(lib(), "oracle_aggregate_" + _suf(dt))
    member_mask = np.ascontiguousarray(member_mask, dtype=np.uint32)
    fn(_p(arch), _p(member_mask), C.c_int(S), sp, sb, _p(global_params), _p(global_buffers))
    return global_params, global_buffers


# ---- layer routines (exported for the pins and for per-kernel parity tests) --------------------
def _odim(h, k, s):
    return (h + 2 * ((k - 1) // 2) - k) // s + 1


def conv_fwd(a, w, stride=1, add=None, quant=0, scale=1.0):
    N, H, W, Cc = a.shape
    K, k = w.shape[0], w.shape[1]
    y = np.empty((N, _odim(H, k, stride), _odim(W, k, stride), K), dtype=a.dtype)
    getattr(lib(), "oracle_conv_fwd_" + _suf(a.dtype))(
        _p(np.ascontiguousarray(a)), _p(np.ascontiguousarray(w)), _p(add), _p(y), N, H, W, Cc, K, k, stride,
        quant, C.c_double(scale))
    return y


def conv_dgrad(dy, w, in_hw, stride=1, add=None, quant=0):
    N = dy.shape[0]
    K, k, _, Cc = w.shape
    H, W = in_hw
    da = np.empty((N, H, W, Cc), dtype=dy.dtype)
    getattr(lib(), "oracle_conv_dgrad_" + _suf(dy.dtype))(
        _p(np.ascontiguousarray(dy)), _p(np.ascontiguousarray(w)), _p(add), _p(da), N, H, W, Cc, K, k, stride, quant)
    return da


def conv_wgrad(dy, a, k, stride=1):
    N, H, W, Cc = a.shape
    K = dy.shape[3]
    dw = np.empty((K, k, k, Cc), dtype=a.dtype)
    getattr(lib(), "oracle_conv_wgrad_" + _suf(a.dtype))(
        _p(np.ascontiguousarray(dy)), _p(np.ascontiguousarray(a)), _p(dw), N, H, W, Cc, K, k, stride)
    return dw


def bn_relu_fwd(x, gamma, beta, run_mean=None, run_var=None, eps=1e-5, mom=0.1, quant=0):
    Cc = x.shape[-1]
    m = x.size // Cc
    a = np.empty_like(x)
    mean = np.empty(Cc, dtype=np.float64)
    invstd = np.empty(Cc, dtype=np.float64)
    getattr(lib(), "oracle_bn_relu_fwd_" + _suf(x.dtype))(
        _p(np.ascontiguousarray(x)), _p(gamma), _p(beta), _p(a), _p(mean), _p(invstd), _p(run_mean), _p(run_var),
        C.c_int64(m), Cc, C.c_double(eps), C.c_double(mom), quant)
    return a, mean, invstd


def bn_relu_bwd(da, x, gamma, beta, mean, invstd, add=None, quant=0):
    Cc = x.shape[-1]
    m = x.size // Cc
    dx = np.empty_like(x)
    dg = np.empty(Cc, dtype=x.dtype)
    db = np.empty(Cc, dtype=x.dtype)
    getattr(lib(), "oracle_bn_relu_bwd_" + _suf(x.dtype))(
        _p(np.ascontiguousarray(da)), _p(np.ascontiguousarray(x)), _p(gamma), _p(beta), _p(mean), _p(invstd),
        _p(add), _p(dx), _p(dg), _p(db), C.c_int64(m), Cc, quant)
    return dx, dg, db


def maxpool_fwd(x):
    N, H, W, Cc = x.shape
    y = np.empty((N, _odim(H, 3, 2), _odim(W, 3, 2), Cc), dtype=x.dtype)
    arg = np.empty(y.shape, dtype=np.int32)
    getattr(lib(), "oracle_maxpool_fwd_" + _suf(x.dtype))(_p(np.ascontiguousarray(x)), _p(y), _p(arg), N, H, W, Cc)
    return y, arg


def maxpool_bwd(dy, arg, in_hw):
    N, _, _, Cc = dy.shape
    H, W = in_hw
    dx = np.empty((N, H, W, Cc), dtype=dy.dtype)
    getattr(lib(), "oracle_maxpool_bwd_" + _suf(dy.dtype))(_p(np.ascontiguousarray(dy)), _p(arg), _p(dx), N, H, W, Cc)
    return dx
