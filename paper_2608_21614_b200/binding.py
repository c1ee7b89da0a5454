"""ctypes binding of libsaem.so: the same names as ``include/saem.h``, argument marshalling only.

Every step of the path runs in the library's CUDA kernels; PyTorch is used here for device
memory, pinned host memory and streams.  Importing this module loads the library and raises if it
cannot be found or built -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

SAEM_OK = 0
SAEM_ERR_INVALID_ARG, SAEM_ERR_SHAPE, SAEM_ERR_ALIGNMENT, SAEM_ERR_WORKSPACE = 1, 2, 3, 4
SAEM_ERR_NOT_RESIDENT, SAEM_ERR_SLOT_BUSY, SAEM_ERR_TIMEOUT, SAEM_ERR_CUDA, SAEM_ERR_UNSUPPORTED = 5, 6, 7, 8, 9
SAEM_MAX_EXPERTS = 128
SAEM_TEMP = -2
SAEM_HOST_MAPPED = -3
SAEM_OUT_F32, SAEM_OUT_BF16 = 0, 1
SAEM_FFN_AUTO, SAEM_FFN_SCALAR, SAEM_FFN_TENSOR, SAEM_FFN_TENSOR_PAIRS, SAEM_FFN_DECODE_FUSED = 0, 1, 2, 3, 4


class saem_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "d_model", "d_ff", "n_experts", "top_k", "max_tokens", "n_layers", "slots_per_layer", "temp_slots",
        "renorm", "out_dtype", "ffn_path", "n_shared")]


class SaemError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (status %d)" % (where, saem_status_string(code), code))


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path) or _build.stale():
        path = _build.build()           # raises if nvcc is missing or the build fails
    lib = C.CDLL(path)
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    cfgp = C.POINTER(saem_config)
    sig = {
        "saem_version": (C.c_int, []),
        "saem_status_string": (C.c_char_p, [i32]),
        "saem_slot_bytes": (sz, [cfgp]),
        "saem_slot_region_bytes": (sz, [cfgp]),
        "saem_workspace_bytes": (sz, [cfgp]),
        "saem_create": (i32, [cfgp, vp, sz, vp, sz, C.POINTER(vp)]),
        "saem_destroy": (None, [vp]),
        "saem_pack_expert_host": (i32, [cfgp, vp, vp, vp, vp]),
        "saem_route": (i32, [vp, vp, i32, vp, vp, vp]),
        "saem_route_fused": (i32, [vp, vp, vp, i32, vp, vp, vp, vp]),
        "saem_repack": (i32, [vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]),
        "saem_expert_ffn": (i32, [vp, i32, vp, vp, i32, vp, i32, vp, vp]),
        "saem_combine": (i32, [vp, vp, vp, vp, i32, vp, vp, vp]),
        "saem_moe_step": (i32, [vp, vp, i32, vp, vp, i32, vp, vp]),
        "saem_moe_step_host": (i32, [vp, vp, i32, vp, vp, i32, vp, vp]),
        "saem_moe_step_host_async": (i32, [vp, vp, i32, vp, vp, i32, vp, vp]),
        "saem_step_buffer": (vp, [vp, i32]),
        "saem_cache_load": (i32, [vp, i32, i32, i32, vp, vp]),
        "saem_cache_evict": (i32, [vp, i32, i32]),
        "saem_cache_map_host": (i32, [vp, i32, i32, vp]),
        "saem_cache_query": (i32, [vp, i32, i32, C.POINTER(i32), C.POINTER(i32)]),
        "saem_cache_wait": (i32, [vp, i32, i32, vp]),
        "saem_last_device_status": (i32, [vp, C.POINTER(i32)]),
        "saem_launch_count": (C.c_longlong, [vp]),
        "saem_expert_ffn_static": (i32, [vp, vp, i32, i32, i32, i32, vp, vp, vp]),
        "saem_selftest_bounded_wait": (i32, [vp, i32, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    return lib


_lib = _load()
EXPORTS = ("saem_version saem_status_string saem_slot_bytes saem_slot_region_bytes saem_workspace_bytes "
           "saem_create saem_destroy saem_pack_expert_host saem_route saem_route_fused saem_repack saem_expert_ffn saem_combine "
           "saem_moe_step saem_moe_step_host saem_moe_step_host_async saem_step_buffer saem_cache_load saem_cache_evict saem_cache_map_host saem_cache_query "
           "saem_cache_wait saem_last_device_status saem_launch_count saem_expert_ffn_static saem_selftest_bounded_wait").split()


def library_path() -> str:
    return _build.LIB


def _ptr(t) -> Optional[int]:
    """Device/host address of a torch tensor, numpy array, int or None."""
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


def _stream(s) -> Optional[int]:
    if s is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(s, torch.cuda.Stream):
        return s.cuda_stream or None
    return int(s) or None


def _check(code: int, where: str) -> None:
    if code != SAEM_OK:
        raise SaemError(code, where)


# ------------------------------------------------------------------------- the C ABI, same names
def saem_version() -> int:
    return _lib.saem_version()


def saem_status_string(code: int) -> str:
    return _lib.saem_status_string(code).decode()


def saem_slot_bytes(cfg: saem_config) -> int:
    return _lib.saem_slot_bytes(C.byref(cfg))


def saem_slot_region_bytes(cfg: saem_config) -> int:
    return _lib.saem_slot_region_bytes(C.byref(cfg))


def saem_workspace_bytes(cfg: saem_config) -> int:
    return _lib.saem_workspace_bytes(C.byref(cfg))


def saem_create(cfg: saem_config, slot_region, slot_region_bytes: int, workspace, workspace_bytes: int) -> int:
    """Returns the context handle (an integer address). Raises SaemError on failure."""
    out = C.c_void_p()
    _check(_lib.saem_create(C.byref(cfg), _ptr(slot_region), slot_region_bytes, _ptr(workspace), workspace_bytes,
                            C.byref(out)), "saem_create")
    return out.value


def saem_create_status(cfg, slot_region, slot_region_bytes, workspace, workspace_bytes) -> int:
    """saem_create returning the raw status (for error-path tests)."""
    out = C.c_void_p()
    code = _lib.saem_create(C.byref(cfg) if cfg is not None else None, _ptr(slot_region), slot_region_bytes,
                            _ptr(workspace), workspace_bytes, C.byref(out))
    if code == SAEM_OK:
        _lib.saem_destroy(out)
    return code


def saem_destroy(ctx: int) -> None:
    _lib.saem_destroy(ctx)


def saem_pack_expert_host(cfg: saem_config, gate, up, down, packed_out) -> None:
    _check(_lib.saem_pack_expert_host(C.byref(cfg), _ptr(gate), _ptr(up), _ptr(down), _ptr(packed_out)),
           "saem_pack_expert_host")


def saem_route(ctx, logits, T, topk_idx, topk_w, stream=None, check=True) -> int:
    code = _lib.saem_route(ctx, _ptr(logits), T, _ptr(topk_idx), _ptr(topk_w), _stream(stream))
    if check:
        _check(code, "saem_route")
    return code


def saem_route_fused(ctx, x, w_router, T, logits_out, topk_idx, topk_w, stream=None, check=True) -> int:
    code = _lib.saem_route_fused(ctx, _ptr(x), _ptr(w_router), T, _ptr(logits_out), _ptr(topk_idx), _ptr(topk_w),
                                 _stream(stream))
    if check:
        _check(code, "saem_route_fused")
    return code


def saem_repack(ctx, topk_idx, x, T, counts, offsets, perm, inv_perm, x_packed, stream=None, check=True) -> int:
    code = _lib.saem_repack(ctx, _ptr(topk_idx), _ptr(x), T, _ptr(counts), _ptr(offsets), _ptr(perm), _ptr(inv_perm),
                            _ptr(x_packed), _stream(stream))
    if check:
        _check(code, "saem_repack")
    return code


def saem_expert_ffn(ctx, layer, x_packed, offsets, max_rows, expert_subset: Optional[Sequence[int]], y_packed,
                    stream=None, check=True) -> int:
    sub, n = None, 0
    if expert_subset is not None:
        n = len(expert_subset)
        sub = (C.c_int32 * max(n, 1))(*expert_subset)
    code = _lib.saem_expert_ffn(ctx, layer, _ptr(x_packed), _ptr(offsets), max_rows,
                                C.cast(sub, C.c_void_p) if sub is not None else None, n, _ptr(y_packed),
                                _stream(stream))
    if check:
        _check(code, "saem_expert_ffn")
    return code


def saem_combine(ctx, y_packed, inv_perm, topk_w, T, shared_y, out, stream=None, check=True) -> int:
    code = _lib.saem_combine(ctx, _ptr(y_packed), _ptr(inv_perm), _ptr(topk_w), T, _ptr(shared_y), _ptr(out),
                             _stream(stream))
    if check:
        _check(code, "saem_combine")
    return code


def saem_moe_step(ctx, shared_ctx, layer, logits, x, T, out, stream=None, check=True) -> int:
    code = _lib.saem_moe_step(ctx, shared_ctx, layer, _ptr(logits), _ptr(x), T, _ptr(out), _stream(stream))
    if check:
        _check(code, "saem_moe_step")
    return code


def saem_moe_step_host(ctx, shared_ctx, layer, logits_host, x_host, T, out_host, stream=None, check=True) -> int:
    code = _lib.saem_moe_step_host(ctx, shared_ctx, layer, _ptr(logits_host), _ptr(x_host), T, _ptr(out_host),
                                   _stream(stream))
    if check:
        _check(code, "saem_moe_step_host")
    return code


def saem_moe_step_host_async(ctx, shared_ctx, layer, logits_host, x_host, T, out_host, stream=None, check=True) -> int:
    code = _lib.saem_moe_step_host_async(ctx, shared_ctx, layer, _ptr(logits_host), _ptr(x_host), T, _ptr(out_host),
                                         _stream(stream))
    if check:
        _check(code, "saem_moe_step_host_async")
    return code


def saem_step_buffer(ctx, which: int) -> Optional[int]:
    return _lib.saem_step_buffer(ctx, which)


def saem_cache_load(ctx, layer, expert, slot, pinned_packed_expert, copy_stream=None, check=True) -> int:
    code = _lib.saem_cache_load(ctx, layer, expert, slot, _ptr(pinned_packed_expert), _stream(copy_stream))
    if check:
        _check(code, "saem_cache_load")
    return code


def saem_cache_evict(ctx, layer, expert, check=True) -> int:
    code = _lib.saem_cache_evict(ctx, layer, expert)
    if check:
        _check(code, "saem_cache_evict")
    return code


def saem_cache_map_host(ctx, layer, expert, pinned_packed_expert, check=True) -> int:
    code = _lib.saem_cache_map_host(ctx, layer, expert, _ptr(pinned_packed_expert))
    if check:
        _check(code, "saem_cache_map_host")
    return code


def saem_cache_query(ctx, layer, expert):
    slot, ready = C.c_int(), C.c_int()
    _check(_lib.saem_cache_query(ctx, layer, expert, C.byref(slot), C.byref(ready)), "saem_cache_query")
    return slot.value, ready.value


def saem_cache_wait(ctx, layer, expert, consumer_stream=None, check=True) -> int:
    code = _lib.saem_cache_wait(ctx, layer, expert, _stream(consumer_stream))
    if check:
        _check(code, "saem_cache_wait")
    return code


def saem_last_device_status(ctx) -> int:
    code = C.c_int()
    _check(_lib.saem_last_device_status(ctx, C.byref(code)), "saem_last_device_status")
    return code.value


def saem_launch_count(ctx) -> int:
    return int(_lib.saem_launch_count(ctx))


def saem_selftest_bounded_wait(ctx, limit_us: int, stream=None, check=True) -> int:
    code = _lib.saem_selftest_bounded_wait(ctx, limit_us, _stream(stream))
    if check:
        _check(code, "saem_selftest_bounded_wait")
    return code


SAEM_STATIC_SCRATCH_ELEMS = 1 << 20


def saem_expert_ffn_static(x_packed, offsets, n_experts, max_rows, d_model, d_ff, packed_experts, y_packed,
                           stream=None, check=True) -> int:
    """The expert FFN for callers that cannot allocate device memory: no context, no workspace;
    the hidden activations use a fixed 2 MiB array inside the library (max_rows * d_ff elements at
    most SAEM_STATIC_SCRATCH_ELEMS).  Calls that may overlap on the GPU race on that array."""
    code = _lib.saem_expert_ffn_static(_ptr(x_packed), _ptr(offsets), n_experts, max_rows, d_model, d_ff,
                                       _ptr(packed_experts), _ptr(y_packed), _stream(stream))
    if check:
        _check(code, "saem_expert_ffn_static")
    return code


# ------------------------------------------------------------------------- memory plumbing (torch)
def make_config(d_model, d_ff, n_experts, top_k, max_tokens, n_layers=1, slots_per_layer=None, temp_slots=0,
                renorm=1, out_dtype=SAEM_OUT_F32, ffn_path=SAEM_FFN_AUTO, n_shared=0) -> saem_config:
    return saem_config(d_model, d_ff, n_experts, top_k, max_tokens, n_layers,
                       n_experts + n_shared if slots_per_layer is None else slots_per_layer, temp_slots, renorm,
                       out_dtype, ffn_path, n_shared)


class Context:
    """A saem_ctx plus the torch tensors that back its slot region and workspace."""

    def __init__(self, cfg: saem_config, device="cuda:0"):
        self.cfg = cfg
        self.device = torch.device(device)
        self.slot_bytes = saem_slot_bytes(cfg)
        if self.slot_bytes == 0:
            raise SaemError(SAEM_ERR_SHAPE, "saem_slot_bytes")
        region_bytes = saem_slot_region_bytes(cfg)
        ws_bytes = saem_workspace_bytes(cfg)
        with torch.cuda.device(self.device):
            self._slots = torch.empty(region_bytes + 1024, dtype=torch.uint8, device=self.device)
            self._ws = torch.empty(ws_bytes + 1024, dtype=torch.uint8, device=self.device)
            self.slot_ptr = (self._slots.data_ptr() + 1023) // 1024 * 1024
            self.ws_ptr = (self._ws.data_ptr() + 1023) // 1024 * 1024
            self.handle = saem_create(cfg, self.slot_ptr, region_bytes, self.ws_ptr, ws_bytes)

    def close(self):
        if getattr(self, "handle", None):
            saem_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def pack(self, gate: np.ndarray, up: np.ndarray, down: np.ndarray, pinned: bool = True) -> torch.Tensor:
        """Canonical bf16-bit matrices -> one packed expert in (pinned) host memory."""
        out = torch.empty(self.slot_bytes, dtype=torch.uint8, pin_memory=pinned)
        saem_pack_expert_host(self.cfg, np.ascontiguousarray(gate), np.ascontiguousarray(up),
                              np.ascontiguousarray(down), out)
        return out

    def step_tensor(self, which: int, shape, dtype) -> torch.Tensor:
        """A view of one intermediate of the last saem_moe_step (see saem_step_buffer)."""
        typestr = {torch.int32: "<i4", torch.float32: "<f4", torch.uint16: "<u2", torch.int16: "<i2"}[dtype]

        class _Raw:
            __cuda_array_interface__ = {"shape": tuple(int(v) for v in shape), "typestr": typestr,
                                        "data": (saem_step_buffer(self.handle, which), False), "version": 2}
        return torch.as_tensor(_Raw(), device=self.device)
