"""Test helpers that derive IEEE fields from the NUMERIC value of a float (frexp), not
from bit manipulation, plus a differently-structured numpy restatement of the block
bookkeeping.  Used to pin the oracle; shared with nothing outside tests/."""
import numpy as np
import torch

BF16, FP32 = 0, 1


def bits_to_f64(bits: np.ndarray, dtype: int) -> np.ndarray:
    if dtype == BF16:
        t = torch.from_numpy(bits.astype(np.uint16).view(np.int16).copy()).view(torch.bfloat16)
    else:
        t = torch.from_numpy(bits.astype(np.uint32).view(np.int32).copy()).view(torch.float32)
    return t.to(torch.float64).numpy()


def ieee_fields(bits: np.ndarray, dtype: int):
    """(sign, biased exponent, mantissa or -1 for NaN) from the value, by the IEEE-754 /
    bfloat16 definition: x = (-1)^s 2^(E-127) (1 + M/2^p) for 1 <= E <= 254,
    x = (-1)^s 2^(-126) (M/2^p) for E = 0, E = 255 for inf (M = 0) and NaN (M != 0)."""
    p = 7 if dtype == BF16 else 23
    x = bits_to_f64(bits, dtype)
    sign = np.signbit(x).astype(np.int64)
    ax = np.abs(x)
    E = np.zeros(x.shape, np.int64)
    M = np.zeros(x.shape, np.int64)
    nan = np.isnan(x)
    inf = np.isinf(x)
    fin = ~(nan | inf)
    sub = fin & (ax < 2.0 ** -126)
    nor = fin & ~sub
    fr, ex = np.frexp(ax[nor])  # ax = fr * 2^ex, fr in [0.5, 1)
    E[nor] = ex - 1 + 127
    M[nor] = np.rint((fr * 2.0 - 1.0) * (1 << p)).astype(np.int64)
    M[sub] = np.rint(ax[sub] * 2.0 ** 126 * (1 << p)).astype(np.int64)
    E[inf | nan] = 255
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
