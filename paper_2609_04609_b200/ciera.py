"""Thin ctypes binding of ``libciera.so``: same names as the C ABI, argument marshalling only.

Every step of the codec runs in the library's CUDA kernels.  torch is used for device memory
and streams, nothing else.  Importing this module loads the library and raises if it has not
been built (``python -m paper_2609_04609_b200.build``): there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

from .workloads import UNIT_DTYPE

BF16 = 0
FP32 = 1
FP16 = 2
DTYPE_CODES = {"bf16": BF16, "fp32": FP32, "fp16": FP16}

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED = -2
ERR_MISALIGNED = -3
ERR_CAPACITY = -4
ERR_CUDA = -5
ERR_TIMEOUT = -6
ERR_CORRUPT = -7
ERR_NOT_BOUND = -8
ERR_TOO_LARGE = -9
NOALLOC_MAX_TILES = 65536

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libciera.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build the CUDA library first (python -m paper_2609_04609_b200.build). "
        "There is no fallback path."
    )
_lib = ctypes.CDLL(_LIB_PATH)

_u64, _u32, _i32, _vp, _sz, _dbl = (ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int, ctypes.c_void_p,
                                    ctypes.c_size_t, ctypes.c_double)


class GainIn(ctypes.Structure):
    _fields_ = [
        ("n_values", _u64), ("dtype", ctypes.c_int32), ("block", _u32), ("q", _dbl),
        ("world_size", ctypes.c_int32), ("overlapped", ctypes.c_int32), ("alpha", _dbl), ("beta", _dbl),
        ("table_bytes", ctypes.POINTER(_dbl)), ("table_secs", ctypes.POINTER(_dbl)), ("n_points", ctypes.c_int32),
        ("t_hash", _dbl), ("t_cmp", _dbl), ("t_decmp", _dbl),
    ]


_SIGS = {
    "ciera_message_capacity": ([_u64, _i32, _u32], _sz),
    "ciera_sm_offset": ([_u64, _u32], _sz),
    "ciera_payload_offset": ([_u64, _i32, _u32], _sz),
    "ciera_message_bytes": ([_u64, _i32, _u32, _u64], _sz),
    "ciera_plan_create": ([_vp, _u32, _i32, _u32, ctypes.POINTER(_vp)], _i32),
    "ciera_plan_destroy": ([_vp], None),
    "ciera_plan_n_units": ([_vp], _u32),
    "ciera_plan_n_tiles": ([_vp], _u32),
    "ciera_plan_tile_values": ([_vp], _u32),
    "ciera_plan_total_values": ([_vp], _u64),
    "ciera_plan_device_bytes": ([_vp], _sz),
    "ciera_plan_host_image": ([_vp], _vp),
    "ciera_plan_workspace_bytes": ([_vp], _sz),
    "ciera_workspace_init": ([_vp, _vp, _vp], _i32),
    "ciera_plan_bind": ([_vp, _vp, _sz, _vp], _i32),
    "ciera_cache_init": ([_vp, _vp, _vp, _vp], _i32),
    "ciera_cache_update": ([_vp, _vp, _vp, _vp], _i32),
    "ciera_encode": ([_vp] * 9, _i32),
    "ciera_encode_noalloc": ([_vp] * 8, _i32),
    "ciera_plan_hash_cache_bytes": ([_vp], _sz),
    "ciera_plan_unit_hash_offset": ([_vp, _u32], _sz),
    "ciera_plan_hashed_workspace_bytes": ([_vp], _sz),
    "ciera_hash_cache_init": ([_vp] * 4, _i32),
    "ciera_encode_hashed": ([_vp] * 9, _i32),
    "ciera_plan_entropy_scratch_bytes": ([_vp], _sz),
    "ciera_entropy_encode": ([_vp] * 5, _i32),
    "ciera_entropy_decode": ([_vp] * 6, _i32),
    "ciera_transport": ([_vp] * 7, _i32),
    "ciera_decode": ([_vp] * 8, _i32),
    "ciera_roundtrip_host": ([_vp, _vp, _sz, _vp, _vp, _vp, _vp], _i32),
    "ciera_should_compress": ([ctypes.POINTER(GainIn), ctypes.POINTER(_dbl), ctypes.POINTER(_i32)], _i32),
    "ciera_select_shards": ([ctypes.POINTER(GainIn), _u32, _u64, _i32, _vp, _vp, _vp, _vp, _vp], _i32),
    "ciera_selftest_bounded_waits": ([_u32, _vp, _vp, _vp, _vp], _i32),
    "ciera_last_cuda_error": ([], _i32),
    "ciera_kernel_launch_count": ([], _u64),
    "ciera_status_string": ([_i32], ctypes.c_char_p),
}
for _name, (_args, _res) in _SIGS.items():
    _f = getattr(_lib, _name)
    _f.argtypes, _f.restype = _args, _res

EXPORTS = tuple(_SIGS)


class CieraError(RuntimeError):
    def __init__(self, where: str, status: int):
        self.status = status
        msg = _lib.ciera_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {_lib.ciera_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


def _check(where: str, status: int) -> None:
    if status != OK:
        raise CieraError(where, status)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    return stream.cuda_stream or None


# ------------------------------------------------------------------------------ sizes (host)


def message_capacity(n: int, dtype: int, block: int) -> int:
    return int(_lib.ciera_message_capacity(n, dtype, block))


def sm_offset(n: int, block: int) -> int:
    return int(_lib.ciera_sm_offset(n, block))


def payload_offset(n: int, dtype: int, block: int) -> int:
    return int(_lib.ciera_payload_offset(n, dtype, block))


def message_bytes(n: int, dtype: int, block: int, payload_bytes: int) -> int:
    return int(_lib.ciera_message_bytes(n, dtype, block, payload_bytes))


def kernel_launch_count() -> int:
    return int(_lib.ciera_kernel_launch_count())


def selftest_bounded_waits(max_polls: int, scratch: torch.Tensor, status: torch.Tensor, report: torch.Tensor,
                           stream=None) -> None:
    """Runs the library's two kinds of bounded device wait with a short limit on things nobody completes
    (see ciera.h): ``status`` receives ERR_TIMEOUT, ``report`` (4 x int32) says which waits gave up."""
    _check("ciera_selftest_bounded_waits",
           _lib.ciera_selftest_bounded_waits(max_polls, _ptr(scratch), _ptr(status), _ptr(report), _stream(stream)))


# ------------------------------------------------------------------------------ plan


class Plan:
    """Owner of a ``ciera_plan`` handle and of the device memory its tile table lives in."""

    def __init__(self, units: np.ndarray, dtype: int, block: int, device: Optional[torch.device] = None):
        units = np.ascontiguousarray(units, dtype=UNIT_DTYPE)
        self.units = units
        self.dtype, self.block = dtype, block
        h = _vp()
        _check("ciera_plan_create",
               _lib.ciera_plan_create(units.ctypes.data if units.size else None, units.size, dtype, block,
                                      ctypes.byref(h)))
        self._h = h
        self.n_units = int(_lib.ciera_plan_n_units(h))
        self.n_tiles = int(_lib.ciera_plan_n_tiles(h))
        self.tile_values = int(_lib.ciera_plan_tile_values(h))
        self.total_values = int(_lib.ciera_plan_total_values(h))
        self.device_bytes = int(_lib.ciera_plan_device_bytes(h))
        self.workspace_bytes = int(_lib.ciera_plan_workspace_bytes(h))
        self.hash_cache_bytes = int(_lib.ciera_plan_hash_cache_bytes(h))
        self.entropy_scratch_bytes = int(_lib.ciera_plan_entropy_scratch_bytes(h))
        self.hashed_workspace_bytes = int(_lib.ciera_plan_hashed_workspace_bytes(h))
        self.table = None
        if device is not None:
            self.bind(device)

    def host_image(self) -> np.ndarray:
        n = self.device_bytes
        if n == 0:
            return np.zeros(0, np.uint8)
        buf = (ctypes.c_uint8 * n).from_address(_lib.ciera_plan_host_image(self._h))
        return np.frombuffer(buf, np.uint8).copy()

    def bind(self, device) -> "Plan":
        self.table = torch.empty(self.device_bytes, dtype=torch.uint8, device=device)
        with torch.cuda.device(self.table.device):
            _check("ciera_plan_bind",
                   _lib.ciera_plan_bind(self._h, self.table.data_ptr(), self.table.numel(), _stream(None)))
        return self

    def new_workspace(self) -> torch.Tensor:
        """A fresh workspace, zero-filled through ``ciera_workspace_init`` as the sender calls expect it."""
        ws = torch.empty(max(self.workspace_bytes, 16), dtype=torch.uint8, device=self.table.device)
        workspace_init(self, ws)
        return ws

    @property
    def handle(self):
        return self._h

    def __del__(self):
        h = getattr(self, "_h", None)
        if h:
            _lib.ciera_plan_destroy(h)
            self._h = None


# ------------------------------------------------------------------------------ device calls


def workspace_init(plan: "Plan", workspace: torch.Tensor, stream=None) -> None:
    """Zero-fills a workspace: once after allocating it, and again after a call that reported a device-side error."""
    with torch.cuda.device(workspace.device):
        _check("ciera_workspace_init", _lib.ciera_workspace_init(plan.handle, _ptr(workspace), _stream(stream)))


def cache_init(plan: Plan, cache: torch.Tensor, weights: Optional[torch.Tensor], stream=None) -> None:
    _check("ciera_cache_init", _lib.ciera_cache_init(plan.handle, _ptr(cache), _ptr(weights), _stream(stream)))


def cache_update(plan: Plan, cache: torch.Tensor, weights: torch.Tensor, stream=None) -> None:
    _check("ciera_cache_update", _lib.ciera_cache_update(plan.handle, _ptr(cache), _ptr(weights), _stream(stream)))


def encode(plan: Plan, weights, sender_cache, messages, wire_bytes, changed_blocks, workspace, status=None,
           stream=None) -> None:
    _check("ciera_encode",
           _lib.ciera_encode(plan.handle, _ptr(weights), _ptr(sender_cache), _ptr(messages), _ptr(wire_bytes),
                             _ptr(changed_blocks), _ptr(workspace), _ptr(status), _stream(stream)))


def encode_noalloc(plan: Plan, weights, sender_cache, messages, wire_bytes, changed_blocks, status=None,
                   stream=None) -> None:
    """``ciera_encode`` without a scratch argument: for callers that can pass the buffers they own
    but cannot allocate one more (see ciera.h).  At most NOALLOC_MAX_TILES tiles per call; calls
    that may overlap on the GPU must not both use it."""
    _check("ciera_encode_noalloc",
           _lib.ciera_encode_noalloc(plan.handle, _ptr(weights), _ptr(sender_cache), _ptr(messages), _ptr(wire_bytes),
                                     _ptr(changed_blocks), _ptr(status), _stream(stream)))


def unit_hash_offset(plan: Plan, unit: int) -> int:
    """Byte offset of the unit's first block in the plan's HashCache."""
    return int(_lib.ciera_plan_unit_hash_offset(plan.handle, unit))


def hash_cache_init(plan: Plan, hash_cache: torch.Tensor, weights: Optional[torch.Tensor], stream=None) -> None:
    _check("ciera_hash_cache_init",
           _lib.ciera_hash_cache_init(plan.handle, _ptr(hash_cache), _ptr(weights), _stream(stream)))


def encode_hashed(plan: Plan, weights, hash_cache, messages, wire_bytes, changed_blocks, workspace, status=None,
                  stream=None) -> None:
    """Sender step with a 128-bit hash per block in place of the exponent cache (blocks of 16 values
    and more); ``workspace`` holds ``plan.hashed_workspace_bytes``."""
    _check("ciera_encode_hashed",
           _lib.ciera_encode_hashed(plan.handle, _ptr(weights), _ptr(hash_cache), _ptr(messages), _ptr(wire_bytes),
                                    _ptr(changed_blocks), _ptr(workspace), _ptr(status), _stream(stream)))


def entropy_encode(plan: Plan, messages, wire_bytes, scratch, stream=None) -> None:
    """rANS-codes the payload of every message in place where that shortens it (after encode)."""
    _check("ciera_entropy_encode",
           _lib.ciera_entropy_encode(plan.handle, _ptr(messages), _ptr(wire_bytes), _ptr(scratch), _stream(stream)))


def entropy_decode(plan: Plan, messages, wire_bytes, scratch, status=None, stream=None) -> None:
    """Restores the raw payload of every message in place (before decode)."""
    _check("ciera_entropy_decode",
           _lib.ciera_entropy_decode(plan.handle, _ptr(messages), _ptr(wire_bytes), _ptr(scratch), _ptr(status),
                                     _stream(stream)))


def transport(plan: Plan, src_messages, dst_messages, wire_bytes, workspace, status=None, stream=None) -> None:
    _check("ciera_transport",
           _lib.ciera_transport(plan.handle, _ptr(src_messages), _ptr(dst_messages), _ptr(wire_bytes),
                                _ptr(workspace), _ptr(status), _stream(stream)))


def decode(plan: Plan, messages, receiver_cache, weights_out, wire_bytes=None, workspace=None, status=None,
           stream=None) -> None:
    _check("ciera_decode",
           _lib.ciera_decode(plan.handle, _ptr(messages), _ptr(receiver_cache), _ptr(weights_out), _ptr(wire_bytes),
                             _ptr(workspace), _ptr(status), _stream(stream)))


class DeviceBuffers(ctypes.Structure):
    _fields_ = [(n, _vp) for n in ("weights_dev", "sender_cache_dev", "msg_send_dev", "msg_recv_dev",
                                   "receiver_cache_dev", "weights_out_dev", "wire_bytes_dev", "changed_blocks_dev",
                                   "workspace_dev", "status_dev")]


def roundtrip_host(plan: Plan, weights_host: torch.Tensor, weights_out_host: torch.Tensor,
                   wire_bytes_host: Optional[torch.Tensor], bufs: DeviceBuffers, stream=None) -> None:
    """Host weights in, host weights out (both CPU tensors, ideally pinned); see ciera.h."""
    nbytes = weights_host.numel() * weights_host.element_size()
    _check("ciera_roundtrip_host",
           _lib.ciera_roundtrip_host(plan.handle, _ptr(weights_host), nbytes, _ptr(weights_out_host),
                                     _ptr(wire_bytes_host), ctypes.addressof(bufs), _stream(stream)))


# ------------------------------------------------------------------------------ gain rule (host)


def _fill_gain_in(gi, keep, n_values, dtype, block, q, world_size=2, alpha=0.0, beta=1.0, table=None, t_hash=0.0,
                  t_cmp=0.0, t_decmp=0.0, overlapped=False):
    gi.n_values, gi.dtype, gi.block, gi.q = n_values, dtype, block, q
    gi.world_size, gi.overlapped, gi.alpha, gi.beta = world_size, int(overlapped), alpha, beta
    gi.t_hash, gi.t_cmp, gi.t_decmp = t_hash, t_cmp, t_decmp
    if table:
        tb = (_dbl * len(table))(*[float(p[0]) for p in table])
        ts = (_dbl * len(table))(*[float(p[1]) for p in table])
        keep.append((tb, ts))  # the arrays must outlive the call
        gi.table_bytes, gi.table_secs, gi.n_points = tb, ts, len(table)
    else:
        gi.n_points = 0


def select_shards(shards, cache_budget_bytes: int, with_sender_cache: bool = False):
    """``shards``: a list of dicts with the keyword arguments of ``should_compress``.  Returns a dict with
    ``ranking``, ``selected``, ``gains``, ``footprints`` (lists) and ``used`` (bytes)."""
    n = len(shards)
    arr = (GainIn * max(n, 1))()
    keep = []
    for gi, sh in zip(arr, shards):
        _fill_gain_in(gi, keep, **sh)
    ranking = (_u32 * max(n, 1))()
    selected = (ctypes.c_uint8 * max(n, 1))()
    gains = (_dbl * max(n, 1))()
    fps = (_u64 * max(n, 1))()
    used = _u64(0)
    _check("ciera_select_shards",
           _lib.ciera_select_shards(arr, n, int(cache_budget_bytes), int(with_sender_cache),
                                    ctypes.cast(ranking, _vp), ctypes.cast(selected, _vp), ctypes.cast(gains, _vp),
                                    ctypes.cast(fps, _vp), ctypes.cast(ctypes.pointer(used), _vp)))
    del keep
    return {"ranking": list(ranking)[:n], "selected": [bool(x) for x in list(selected)[:n]],
            "gains": list(gains)[:n], "footprints": list(fps)[:n], "used": int(used.value)}


def should_compress(n_values: int, dtype: int, block: int, q: float, world_size: int = 2, alpha: float = 0.0,
                    beta: float = 1.0, table=None, t_hash: float = 0.0, t_cmp: float = 0.0, t_decmp: float = 0.0,
                    overlapped: bool = False):
    """Returns (gain_seconds, decision)."""
    gi = GainIn()
    keep = []
    _fill_gain_in(gi, keep, n_values, dtype, block, q, world_size, alpha, beta, table, t_hash, t_cmp, t_decmp, overlapped)
    g = _dbl(0.0)
    d = _i32(0)
    _check("ciera_should_compress", _lib.ciera_should_compress(ctypes.byref(gi), ctypes.byref(g), ctypes.byref(d)))
    del keep
    return float(g.value), bool(d.value)
