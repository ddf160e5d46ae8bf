"""ctypes front end of the plain-C CPU oracle (``ciera_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's cpu_baseline / reference legs.  Nothing in the product package imports
it, and it imports nothing from the product package.

All arrays are numpy, on the host.  Weights travel as raw bit patterns: ``uint16``
for bf16, ``uint32`` for fp32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

BF16 = 0
FP32 = 1
FP16 = 2

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ciera_oracle.c")
_LIB = os.path.join(_HERE, "libciera_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no tuning flags beyond -O2)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, u32, i32, dbl, vp = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        for name, args in (
            ("ora_num_blocks", [u64, u32]),
            ("ora_bitmap_bytes", [u64, u32]),
            ("ora_sm_bytes", [u64, i32]),
            ("ora_block_payload_bytes", [u64, i32]),
            ("ora_sm_offset", [u64, u32]),
            ("ora_payload_offset", [u64, i32, u32]),
            ("ora_message_capacity", [u64, i32, u32]),
            ("ora_paper_bytes", [u64, i32, u32, u64]),
        ):
            f = getattr(L, name)
            f.argtypes, f.restype = args, u64
        L.ora_split.argtypes, L.ora_split.restype = [vp, u64, i32, vp, vp], None
        L.ora_merge.argtypes, L.ora_merge.restype = [vp, vp, u64, i32, vp], None
        L.ora_cache_init.argtypes, L.ora_cache_init.restype = [vp, vp, u64, i32], None
        L.ora_encode.argtypes = [vp, vp, u64, i32, u32, vp, u64, vp, vp, vp]
        L.ora_encode.restype = i32
        L.ora_decode.argtypes, L.ora_decode.restype = [vp, vp, u64, i32, u32, vp], i32
        L.ora_splitmix64_mix.argtypes, L.ora_splitmix64_mix.restype = [u64], u64
        L.ora_splitmix64_next.argtypes, L.ora_splitmix64_next.restype = [vp], u64
        L.ora_splitmix64_next_with.argtypes, L.ora_splitmix64_next_with.restype = [vp, u64], u64
        L.ora_hash128.argtypes, L.ora_hash128.restype = [vp, u64, vp], None
        L.ora_hash_cache_init.argtypes, L.ora_hash_cache_init.restype = [vp, u64, i32, u32, vp], i32
        L.ora_encode_hashed.argtypes = [vp, vp, u64, i32, u32, vp, u64, vp, vp, vp]
        L.ora_encode_hashed.restype = i32
        L.ora_gain.argtypes = [u64, i32, u32, dbl, i32, dbl, dbl, vp, vp, i32, dbl, dbl, dbl, i32]
        L.ora_gain.restype = dbl
        _lib = L
    return _lib


def _wdtype(dtype: int):
    return np.uint32 if dtype == FP32 else np.uint16


def _ptr(a: np.ndarray) -> int:
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data


def num_blocks(n, block):
    return int(lib().ora_num_blocks(n, block))


def bitmap_bytes(n, block):
    return int(lib().ora_bitmap_bytes(n, block))


def sm_bytes(n, dtype):
    return int(lib().ora_sm_bytes(n, dtype))


def block_payload_bytes(length, dtype):
    return int(lib().ora_block_payload_bytes(length, dtype))


def sm_offset(n, block):
    return int(lib().ora_sm_offset(n, block))


def payload_offset(n, dtype, block):
    return int(lib().ora_payload_offset(n, dtype, block))


def message_capacity(n, dtype, block):
    return int(lib().ora_message_capacity(n, dtype, block))


def paper_bytes(n, dtype, block, payload_bytes):
    return int(lib().ora_paper_bytes(n, dtype, block, payload_bytes))


def split(w_bits: np.ndarray, dtype: int):
    """SplitExpMant: returns (exp uint8[N], sm uint32[N])."""
    w_bits = np.ascontiguousarray(w_bits, dtype=_wdtype(dtype))
    n = w_bits.size
    exp = np.empty(n, np.uint8)
    sm = np.empty(n, np.uint32)
    lib().ora_split(_ptr(w_bits), n, dtype, _ptr(exp), _ptr(sm))
    return exp, sm


def merge(exp: np.ndarray, sm: np.ndarray, dtype: int) -> np.ndarray:
    exp = np.ascontiguousarray(exp, np.uint8)
    sm = np.ascontiguousarray(sm, np.uint32)
    out = np.empty(exp.size, _wdtype(dtype))
    lib().ora_merge(_ptr(exp), _ptr(sm), exp.size, dtype, _ptr(out))
    return out


def cache_init(w_bits, n: int, dtype: int) -> np.ndarray:
    """Exponents of ``w_bits``; all zero when ``w_bits`` is None."""
    cache = np.empty(n, np.uint8)
    if w_bits is None:
        lib().ora_cache_init(_ptr(cache), None, n, dtype)
    else:
        w_bits = np.ascontiguousarray(w_bits, dtype=_wdtype(dtype))
        assert w_bits.size == n
        lib().ora_cache_init(_ptr(cache), _ptr(w_bits), n, dtype)
    return cache


def encode(w_bits: np.ndarray, cache_s: np.ndarray, dtype: int, block: int):
    """One unit, sender side.  ``cache_s`` (uint8[N]) is updated in place.

    Returns (message uint8[wire_bytes], wire_bytes, payload_bytes, changed_blocks).
    """
    w_bits = np.ascontiguousarray(w_bits, dtype=_wdtype(dtype))
    n = w_bits.size
    assert cache_s.dtype == np.uint8 and cache_s.size == n and cache_s.flags["C_CONTIGUOUS"]
    cap = message_capacity(n, dtype, block)
    msg = np.zeros(max(cap, 1), np.uint8)
    wire = ctypes.c_uint64(0)
    pay = ctypes.c_uint64(0)
    chg = ctypes.c_uint32(0)
    rc = lib().ora_encode(_ptr(w_bits), _ptr(cache_s), n, dtype, block, _ptr(msg), cap,
                          ctypes.addressof(wire), ctypes.addressof(pay), ctypes.addressof(chg))
    if rc != 0:
        raise RuntimeError(f"ora_encode failed: {rc}")
    return msg[: wire.value].copy(), int(wire.value), int(pay.value), int(chg.value)


def decode(msg: np.ndarray, cache_r: np.ndarray, dtype: int, block: int) -> np.ndarray:
    """One unit, receiver side.  ``cache_r`` (uint8[N]) is patched in place."""
    n = cache_r.size
    assert cache_r.dtype == np.uint8 and cache_r.flags["C_CONTIGUOUS"]
    msg = np.ascontiguousarray(msg, np.uint8)
    out = np.empty(n, _wdtype(dtype))
    rc = lib().ora_decode(_ptr(msg) if msg.size else None, _ptr(cache_r), n, dtype, block, _ptr(out))
    if rc != 0:
        raise RuntimeError(f"ora_decode failed: {rc}")
    return out


def gain(n, dtype, block, q, world, alpha=0.0, beta=1.0, table=None, t_hash=0.0, t_cmp=0.0, t_decmp=0.0,
         overlapped=False) -> float:
    """g_i of the selective-compression rule; ``table`` = [(bytes, seconds), ...] or None."""
    if table:
        tb = np.array([p[0] for p in table], np.float64)
        ts = np.array([p[1] for p in table], np.float64)
        return float(lib().ora_gain(n, dtype, block, q, world, alpha, beta, _ptr(tb), _ptr(ts), len(table),
                                    t_hash, t_cmp, t_decmp, int(overlapped)))
    return float(lib().ora_gain(n, dtype, block, q, world, alpha, beta, None, None, 0,
                                t_hash, t_cmp, t_decmp, int(overlapped)))


# ------------------------------------------------------------------ hash-based change detection


def splitmix64_stream(seed: int, count: int, gamma: int = None):
    """First ``count`` outputs of the SplitMix64 generator seeded with ``seed`` (``gamma``: an increment
    other than the generator's own)."""
    state = ctypes.c_uint64(seed)
    if gamma is None:
        return [int(lib().ora_splitmix64_next(ctypes.addressof(state))) for _ in range(count)]
    return [int(lib().ora_splitmix64_next_with(ctypes.addressof(state), gamma)) for _ in range(count)]


def splitmix64_mix(z: int) -> int:
    return int(lib().ora_splitmix64_mix(z))


def hash128(exp: np.ndarray):
    """Hash128 of one block of exponent bytes: (H_s1, H_s2)."""
    exp = np.ascontiguousarray(exp, np.uint8)
    out = np.zeros(2, np.uint64)
    lib().ora_hash128(_ptr(exp) if exp.size else None, exp.size, _ptr(out))
    return int(out[0]), int(out[1])


def hash_cache_init(w_bits, n: int, dtype: int, block: int) -> np.ndarray:
    """HashCache of one unit: uint64[2 * S_b]; of all-zero exponents when ``w_bits`` is None."""
    hc = np.zeros(2 * num_blocks(n, block), np.uint64)
    if n == 0:
        return hc
    if w_bits is None:
        rc = lib().ora_hash_cache_init(None, n, dtype, block, _ptr(hc))
    else:
        w_bits = np.ascontiguousarray(w_bits, dtype=_wdtype(dtype))
        assert w_bits.size == n
        rc = lib().ora_hash_cache_init(_ptr(w_bits), n, dtype, block, _ptr(hc))
    assert rc == 0
    return hc


def encode_hashed(w_bits: np.ndarray, hash_cache: np.ndarray, dtype: int, block: int):
    """Like ``encode`` but with HashCache (uint64[2 * S_b], updated in place) on the sender."""
    w_bits = np.ascontiguousarray(w_bits, dtype=_wdtype(dtype))
    n = w_bits.size
    assert hash_cache.dtype == np.uint64 and hash_cache.size == 2 * num_blocks(n, block)
    cap = message_capacity(n, dtype, block)
    msg = np.zeros(max(cap, 1), np.uint8)
    wire, pay, chg = ctypes.c_uint64(0), ctypes.c_uint64(0), ctypes.c_uint32(0)
    rc = lib().ora_encode_hashed(_ptr(w_bits) if n else None, _ptr(hash_cache) if n else None, n, dtype, block, _ptr(msg), cap,
                                 ctypes.addressof(wire), ctypes.addressof(pay), ctypes.addressof(chg))
    assert rc == 0, rc
    return msg[: wire.value].copy(), int(wire.value), int(pay.value), int(chg.value)
