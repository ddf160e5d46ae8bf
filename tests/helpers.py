"""Test helpers that derive IEEE fields from the NUMERIC value of a float (frexp), not
from bit manipulation, plus a differently-structured numpy restatement of the block
bookkeeping.  Used to pin the oracle; shared with nothing outside tests/."""
import numpy as np
import torch

BF16, FP32, FP16 = 0, 1, 2
# (exponent bits, stored mantissa bits, exponent bias) of the three precisions
FORMAT = {BF16: (8, 7, 127), FP32: (8, 23, 127), FP16: (5, 10, 15)}


def bits_to_f64(bits: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == BF16:
        t = torch.from_numpy(bits.astype(np.uint16).view(np.int16).copy()).view(torch.bfloat16)
    elif dtype == FP16:
        return bits.astype(np.uint16).view(np.float16).astype(np.float64)
    else:
        t = torch.from_numpy(bits.astype(np.uint32).view(np.int32).copy()).view(torch.float32)
    return t.to(torch.float64).numpy()


def ieee_fields(bits: np.ndarray, dtype: int):
    """(sign, biased exponent, mantissa or -1 for NaN) from the value, by the IEEE-754 /
    bfloat16 definition: x = (-1)^s 2^(E-bias) (1 + M/2^p) for 1 <= E <= Emax-1,
    x = (-1)^s 2^(1-bias) (M/2^p) for E = 0, E = Emax for inf (M = 0) and NaN (M != 0)
    (bias 127, Emax 255 for bf16 / fp32; bias 15, Emax 31 for fp16)."""
    ebits, p, bias = FORMAT[dtype]
    emax = (1 << ebits) - 1
    x = bits_to_f64(bits, dtype)
    sign = np.signbit(x).astype(np.int64)
    ax = np.abs(x)
    E = np.zeros(x.shape, np.int64)
    M = np.zeros(x.shape, np.int64)
    nan = np.isnan(x)
    inf = np.isinf(x)
    fin = ~(nan | inf)
    sub = fin & (ax < 2.0 ** (1 - bias))
    nor = fin & ~sub
    fr, ex = np.frexp(ax[nor])  # ax = fr * 2^ex, fr in [0.5, 1)
    E[nor] = ex - 1 + bias
    M[nor] = np.rint((fr * 2.0 - 1.0) * (1 << p)).astype(np.int64)
    M[sub] = np.rint(ax[sub] * 2.0 ** (bias - 1) * (1 << p)).astype(np.int64)
    E[inf | nan] = emax
    M[nan] = -1
    return sign, E, M


def shadow_blocks(exp_new: np.ndarray, cache: np.ndarray, block: int):
    """Independent block bookkeeping: (bitmap bytes, payload, cache_after, changed mask)."""
    n = exp_new.size
    nb = -(-n // block)
    diff = np.zeros(nb * block, bool)
    diff[:n] = exp_new != cache
    chg = diff.reshape(nb, block).any(axis=1)
    bitmap = np.packbits(chg, bitorder="little")
    per_value = np.repeat(chg, block)[:n]
    payload = exp_new[per_value]
    cache_after = np.where(per_value, exp_new, cache)
    return bitmap, payload, cache_after, chg


def pack_fields(values: np.ndarray, width: int) -> np.ndarray:
    """Bytes of a section in which value j occupies bits [j * width, (j + 1) * width), bit i of the
    section = byte i >> 3, bit i & 7 (numpy restatement, independent of the oracle's bit loop)."""
    v = np.asarray(values, np.uint64)
    bits = ((v[:, None] >> np.arange(width, dtype=np.uint64)[None, :]) & 1).astype(np.uint8).reshape(-1)
    return np.packbits(bits, bitorder="little")


def shadow_blocks_packed(exp_new: np.ndarray, cache: np.ndarray, block: int, ebits: int):
    """``shadow_blocks`` with e-bit exponents on the wire: every changed block is packed on its own
    and starts on a byte boundary."""
    bitmap, _, cache_after, chg = shadow_blocks(exp_new, cache, block)
    parts = [pack_fields(exp_new[k * block : (k + 1) * block], ebits) for k in np.flatnonzero(chg)]
    payload = np.concatenate(parts) if parts else np.zeros(0, np.uint8)
    return bitmap, payload, cache_after, chg


def parse_golden(path):
    steps, cur = [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line == "[step]":
            cur = {}
            steps.append(cur)
            continue
        k, *v = line.split()
        cur[k] = v
    return steps
