"""ctypes front end of the entropy-stage oracle (``rans_oracle.c``) and its application to whole
unit messages.  TEST INFRASTRUCTURE ONLY (see ``ciera_oracle.py``)."""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from . import ciera_oracle as ora

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rans_oracle.c")
_LIB = os.path.join(_HERE, "librans_oracle.so")
SEGMENT = 4096
LANES = 32

_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, u32, vp = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_void_p
        L.rans_normalise.argtypes, L.rans_normalise.restype = [vp, u64, vp], None
        L.rans_encode_step.argtypes, L.rans_encode_step.restype = [vp, u32, u32, vp], ctypes.c_int
        L.rans_coded_bound.argtypes, L.rans_coded_bound.restype = [u64], u64
        L.rans_encode.argtypes, L.rans_encode.restype = [vp, u64, vp], u64
        L.rans_decode.argtypes, L.rans_decode.restype = [vp, u64, u64, vp], ctypes.c_int
        _lib = L
    return _lib


def normalise(hist: np.ndarray) -> np.ndarray:
    hist = np.ascontiguousarray(hist, np.uint64)
    f = np.zeros(256, np.uint16)
    lib().rans_normalise(hist.ctypes.data, int(hist.sum()), f.ctypes.data)
    return f


def encode_step(x: int, f: int, c: int):
    """One encoder step of one lane: returns (new state, emitted word or None)."""
    xs, w = ctypes.c_uint32(x), ctypes.c_uint32(0)
    emitted = lib().rans_encode_step(ctypes.addressof(xs), f, c, ctypes.addressof(w))
    return int(xs.value), (int(w.value) if emitted else None)


def coded_bound(p: int) -> int:
    return int(lib().rans_coded_bound(p))


def encode(raw: np.ndarray) -> np.ndarray:
    raw = np.ascontiguousarray(raw, np.uint8)
    out = np.zeros(max(coded_bound(raw.size), 16), np.uint8)
    n = int(lib().rans_encode(raw.ctypes.data, raw.size, out.ctypes.data))
    return out[:n].copy()


def decode(coded: np.ndarray, p: int) -> np.ndarray:
    coded = np.ascontiguousarray(coded, np.uint8)
    raw = np.zeros(max(p, 1), np.uint8)
    rc = lib().rans_decode(coded.ctypes.data if coded.size else None, coded.size, p, raw.ctypes.data)
    if rc != 0:
        raise ValueError("inconsistent coded section")
    return raw[:p]


# ------------------------------------------------------------------ whole unit messages


def payload_bytes_from_bitmap(msg: np.ndarray, n: int, block: int, dtype: int = 0) -> int:
    """P = total length in bytes of the changed blocks, read off the message's bitmap (a block of L values takes
    L bytes, for fp16 -- five bits per exponent, every block starting on a byte boundary -- ceil(5 L / 8))."""
    nb = ora.num_blocks(n, block)
    flags = np.unpackbits(msg[: ora.bitmap_bytes(n, block)], bitorder="little")[:nb].astype(bool)
    lens = np.minimum(block, n - np.arange(nb, dtype=np.int64) * block)
    return int(sum(ora.block_payload_bytes(int(l), dtype) for l in lens[flags]))


def entropy_encode_message(msg: np.ndarray, n: int, dtype: int, block: int) -> np.ndarray:
    """The sender's entropy stage on one unit's raw message: the payload is replaced by its coded
    section iff that is strictly shorter.  The coder's symbols are the payload's BYTES whatever the precision: for
    fp16 these are the bytes of the packed five-bit exponents as they travel (a reading: the paper names a byte-wise
    general-purpose coder from a vendor library and says nothing about sub-byte symbols)."""
    pay_off = ora.payload_offset(n, dtype, block)
    p = msg.size - pay_off
    if p <= 0:
        return msg.copy()
    coded = encode(msg[pay_off:])
    if coded.size >= p:
        return msg.copy()
    return np.concatenate([msg[:pay_off], coded])


def entropy_decode_message(msg: np.ndarray, n: int, dtype: int, block: int) -> np.ndarray:
    """The receiver's entropy stage: a message shorter than its bitmap implies holds a coded section."""
    pay_off = ora.payload_offset(n, dtype, block)
    p = payload_bytes_from_bitmap(msg, n, block, dtype)
    if msg.size == pay_off + p:
        return msg.copy()
    return np.concatenate([msg[:pay_off], decode(msg[pay_off:], p)])
