"""ctypes wrapper of the plain-C CPU oracle (``saem_oracle.c``): TEST INFRASTRUCTURE.

Argument marshalling only; every number comes from the C file.  The shared object is built with
gcc on first use (``build()``), without -ffast-math.  Nothing here imports the CUDA package's
binding, and the CUDA package never imports this module.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "saem_oracle.c")
_LIB = os.path.join(_HERE, "libsaem_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile saem_oracle.c -> libsaem_oracle.so (gcc -O2 -fopenmp)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.saem_oracle_max_threads.restype = C.c_int
    return _lib


def max_threads() -> int:
    return int(_load().saem_oracle_max_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _ptr_array(mats: Sequence[Optional[np.ndarray]]):
    arr = (C.c_void_p * len(mats))()
    for i, m in enumerate(mats):
        if m is not None:
            assert m.dtype == np.uint16 and m.flags.c_contiguous
            arr[i] = m.ctypes.data
    return arr


def router_logits(x: np.ndarray, w_router: np.ndarray) -> np.ndarray:
    """float64 logits[T, E] of a bias-free linear router from bf16 bit patterns x[T, d], w_router[E, d]."""
    x = np.ascontiguousarray(x, dtype=np.uint16)
    w_router = np.ascontiguousarray(w_router, dtype=np.uint16)
    T, d = x.shape
    E = w_router.shape[0]
    out = np.empty((T, E), np.float64)
    _load().saem_oracle_router_logits(_p(x), _p(w_router), T, E, d, _p(out))
    return out


def route(logits: np.ndarray, k: int, renorm: bool = True):
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, E = logits.shape
    idx = np.empty((T, k), np.int32)
    w = np.empty((T, k), np.float64)
    _load().saem_oracle_route(_p(logits), T, E, k, int(renorm), _p(idx), _p(w))
    return idx, w


def repack(topk_idx: np.ndarray, x: Optional[np.ndarray], n_experts: int):
    topk_idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, k = topk_idx.shape
    d = 0
    xp = None
    if x is not None:
        x = np.ascontiguousarray(x, dtype=np.uint16)
        d = x.shape[1]
        xp = np.empty((T * k, d), np.uint16)
    counts = np.empty(n_experts, np.int32)
    offsets = np.empty(n_experts + 1, np.int32)
    perm = np.empty(T * k, np.int32)
    inv = np.empty(T * k, np.int32)
    _load().saem_oracle_repack(_p(topk_idx), _p(x), T, n_experts, k, d, _p(counts), _p(offsets),
                               _p(perm), _p(inv), _p(xp))
    return counts, offsets, perm, inv, xp


def expert_ffn(x_packed: np.ndarray, offsets: np.ndarray, gate, up, down, acc_fp32: bool = False):
    x_packed = np.ascontiguousarray(x_packed, dtype=np.uint16)
    offsets = np.ascontiguousarray(offsets, dtype=np.int32)
    E = len(offsets) - 1
    P, d = x_packed.shape
    assert offsets[E] == P
    f = next(g.shape[0] for g in gate if g is not None)
    y = np.empty((P, d), np.float64)
    _load().saem_oracle_expert_ffn(_p(x_packed), _p(offsets), E, d, f, _ptr_array(gate), _ptr_array(up),
                                   _ptr_array(down), int(acc_fp32), _p(y))
    return y


def combine(y_packed: np.ndarray, inv_perm: np.ndarray, topk_w: np.ndarray,
            shared_y: Optional[np.ndarray] = None):
    y_packed = np.ascontiguousarray(y_packed, dtype=np.float64)
    inv_perm = np.ascontiguousarray(inv_perm, dtype=np.int32)
    topk_w = np.ascontiguousarray(topk_w, dtype=np.float64)
    T, k = topk_w.shape
    d = y_packed.shape[1]
    if shared_y is not None:
        shared_y = np.ascontiguousarray(shared_y, dtype=np.float64)
    out = np.empty((T, d), np.float64)
    _load().saem_oracle_combine(_p(y_packed), _p(inv_perm), _p(topk_w), T, k, d, _p(shared_y), _p(out))
    return out


def moe_step(logits, x, k, gate, up, down, shared=None, renorm=True, acc_fp32=False):
    """The whole layer step. Returns a dict of every intermediate and ``out``."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    x = np.ascontiguousarray(x, dtype=np.uint16)
    T, E = logits.shape
    d = x.shape[1]
    f = next(g.shape[0] for g in gate if g is not None)
    P = T * k
    r = dict(topk_idx=np.empty((T, k), np.int32), topk_w=np.empty((T, k), np.float64),
             counts=np.empty(E, np.int32), offsets=np.empty(E + 1, np.int32),
             perm=np.empty(P, np.int32), inv_perm=np.empty(P, np.int32),
             x_packed=np.empty((P, d), np.uint16), y_packed=np.empty((P, d), np.float64),
             shared_y=np.empty((T, d), np.float64) if shared else None,
             out=np.empty((T, d), np.float64))
    fs = shared[0].shape[0] if shared else 0
    sg, su, sd = (shared if shared else (None, None, None))
    _load().saem_oracle_moe_step(
        _p(logits), _p(x), T, E, k, d, f, int(renorm), _ptr_array(gate), _ptr_array(up), _ptr_array(down),
        fs, _p(sg), _p(su), _p(sd), int(acc_fp32),
        _p(r["topk_idx"]), _p(r["topk_w"]), _p(r["counts"]), _p(r["offsets"]), _p(r["perm"]),
        _p(r["inv_perm"]), _p(r["x_packed"]), _p(r["y_packed"]), _p(r["shared_y"]), _p(r["out"]))
    return r
