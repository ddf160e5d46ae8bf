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
        L.rans_coded_bound_alphabet.argtypes, L.rans_coded_bound_alphabet.restype = [u64, u32], u64
        L.rans_encode_alphabet.argtypes, L.rans_encode_alphabet.restype = [vp, u64, vp, u32], u64
        L.rans_decode_alphabet.argtypes, L.rans_decode_alphabet.restype = [vp, u64, u64, vp, u32], ctypes.c_int
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


def coded_bound(p: int, entries: int = 256) -> int:
    return int(lib().rans_coded_bound_alphabet(p, entries))


def encode(raw: np.ndarray, entries: int = 256) -> np.ndarray:
    """Coded section of the symbols ``raw`` (one per byte, all below ``entries`` = 256 or 32)."""
    raw = np.ascontiguousarray(raw, np.uint8)
    if raw.size and int(raw.max()) >= entries:
        raise ValueError("a symbol does not fit the alphabet")
    out = np.zeros(max(coded_bound(raw.size, entries), 16), np.uint8)
    n = int(lib().rans_encode_alphabet(raw.ctypes.data, raw.size, out.ctypes.data, entries))
    return out[:n].copy()


def decode(coded: np.ndarray, p: int, entries: int = 256) -> np.ndarray:
    coded = np.ascontiguousarray(coded, np.uint8)
    raw = np.zeros(max(p, 1), np.uint8)
    rc = lib().rans_decode_alphabet(coded.ctypes.data if coded.size else None, coded.size, p, raw.ctypes.data, entries)
    if rc != 0:
        raise ValueError("inconsistent coded section")
    return raw[:p]


# ------------------------------------------------------------------ whole unit messages

FP16 = 2


def changed_block_lengths(msg: np.ndarray, n: int, block: int) -> np.ndarray:
    """Lengths in values of the changed blocks, in order, read off the message's bitmap."""
    nb = ora.num_blocks(n, block)
    flags = np.unpackbits(msg[: ora.bitmap_bytes(n, block)], bitorder="little")[:nb].astype(bool)
    lens = np.minimum(block, n - np.arange(nb, dtype=np.int64) * block)
    return lens[flags]


def payload_bytes_from_bitmap(msg: np.ndarray, n: int, block: int, dtype: int = 0) -> int:
    """P = total length in bytes of the changed blocks, read off the message's bitmap (a block of L values takes
    L bytes, for fp16 -- five bits per exponent, every block starting on a byte boundary -- ceil(5 L / 8))."""
    return int(sum(ora.block_payload_bytes(int(l), dtype) for l in changed_block_lengths(msg, n, block)))


def unpack_fp16_payload(payload: np.ndarray, lens: np.ndarray) -> np.ndarray:
    """The five-bit exponents of an fp16 payload, one per byte: block k of ``lens[k]`` values starts on a byte
    boundary, its exponent j lies in bits [5 j, 5 j + 5) of the block's bytes (bit i = byte i >> 3, bit i & 7)."""
    out = np.zeros(int(np.sum(lens)), np.uint8)
    weights = np.array([1, 2, 4, 8, 16], np.uint8)
    at_byte = at_sym = 0
    for length in (int(l) for l in lens):
        nbytes = (5 * length + 7) // 8
        bits = np.unpackbits(payload[at_byte : at_byte + nbytes], bitorder="little")[: 5 * length]
        out[at_sym : at_sym + length] = bits.reshape(length, 5) @ weights
        at_byte += nbytes
        at_sym += length
    if at_byte != payload.size:
        raise ValueError("payload length does not match the changed blocks")
    return out


def pack_fp16_payload(symbols: np.ndarray, lens: np.ndarray) -> np.ndarray:
    """Inverse of ``unpack_fp16_payload``; the unused high bits of a block's last byte are zero."""
    pieces = []
    at_sym = 0
    for length in (int(l) for l in lens):
        s = symbols[at_sym : at_sym + length]
        bits = (s[:, None] >> np.arange(5, dtype=np.uint8)[None, :]) & 1
        pieces.append(np.packbits(bits.reshape(-1).astype(np.uint8), bitorder="little"))
        at_sym += length
    return np.concatenate(pieces) if pieces else np.zeros(0, np.uint8)


def entropy_encode_message(msg: np.ndarray, n: int, dtype: int, block: int) -> np.ndarray:
    """The sender's entropy stage on one unit's raw message: the payload is replaced by its coded
    section iff that is strictly shorter.  The coder's symbols are the exponents of the changed blocks (Algorithm 1:
    ANSEncode of {exp[k] | bitmap[k] = 1}): the payload's bytes for bf16 and fp32; for fp16 the five-bit exponents,
    unpacked to one symbol each, with a table of 32 entries."""
    pay_off = ora.payload_offset(n, dtype, block)
    p = msg.size - pay_off
    if p <= 0:
        return msg.copy()
    if dtype == FP16:
        coded = encode(unpack_fp16_payload(msg[pay_off:], changed_block_lengths(msg, n, block)), 32)
    else:
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
    if dtype == FP16:
        lens = changed_block_lengths(msg, n, block)
        payload = pack_fp16_payload(decode(msg[pay_off:], int(lens.sum()), 32), lens)
    else:
        payload = decode(msg[pay_off:], p)
    return np.concatenate([msg[:pay_off], payload])
