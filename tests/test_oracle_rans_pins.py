"""Pins of the entropy-stage oracle (rANS coding of the changed exponents; Section 3.1 and
Algorithm 1 name only "ANS").  No GPU.

Fixed from outside: the rANS recurrences on hand-worked steps, exact round trips (the stage is
lossless), the coded size against the empirical entropy of the data (an entropy coder with a
12-bit static model stays within a few per cent of it), and the algebra of the model (sums to
4096, every present symbol keeps a non-zero share).  The coded bytes themselves follow this
build's own layout: parity unpinned for the byte stream."""
import os

import numpy as np
import pytest

from helpers import BF16, FP32
from oracle import rans_oracle as rans
from paper_2609_04609_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "rans_worked_example.txt")


def test_hand_worked_encoder_steps():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 4
    for x, f, c, x_new, word in rows:
        got_x, got_w = rans.encode_step(int(x), int(f), int(c))
        assert got_x == int(x_new)
        assert got_w == (None if word == "-" else int(word))
        # the decoder's step inverts it
        slot = got_x % 4096
        assert int(c) <= slot < int(c) + int(f)
        back = int(f) * (got_x // 4096) + slot - int(c)
        if got_w is not None:
            assert back < 65536
            back = back * 65536 + got_w
        assert back == int(x)


def test_model_sums_to_4096_and_keeps_every_present_symbol():
    rng = np.random.default_rng(1)
    for trial in range(300):
        k = int(rng.integers(1, 257))
        hist = np.zeros(256, np.uint64)
        syms = rng.choice(256, k, replace=False)
        kind = trial % 3
        if kind == 0:
            hist[syms] = rng.integers(1, 10, k)
        elif kind == 1:
            hist[syms] = rng.integers(1, 1_000_000, k)
        else:
            hist[syms] = 1
            hist[syms[0]] = 10_000_000  # one dominant symbol, many rare ones
        f = rans.normalise(hist).astype(np.int64)
        assert f.sum() == 4096
        assert np.array_equal(f > 0, hist > 0)
    # proportionality where nothing is clamped: 3 : 1 gives 3072 : 1024
    hist = np.zeros(256, np.uint64)
    hist[65], hist[66] = 300, 100
    f = rans.normalise(hist)
    assert (f[65], f[66]) == (3072, 1024)


def _exponent_like(rng, n):
    """Bytes distributed like the exponents of N(0, 0.02) weights (a few values around 120)."""
    return np.clip(np.round(rng.normal(120.5, 1.3, n)), 0, 255).astype(np.uint8)


@pytest.mark.parametrize("n", [1, 2, 31, 32, 33, 100, 4095, 4096, 4097, 8192, 10_000, 70_001])
def test_round_trip_and_layout(n):
    rng = np.random.default_rng(n)
    for kind in range(4):
        raw = [_exponent_like(rng, n), rng.integers(0, 256, n).astype(np.uint8), np.full(n, 7, np.uint8),
               rng.choice(np.array([0, 255, 128], np.uint8), n, p=[0.98, 0.01, 0.01])][kind]
        coded = rans.encode(raw)
        assert coded.size <= rans.coded_bound(n)
        assert np.array_equal(rans.decode(coded, n), raw)
        # layout: table, directory of word counts, segments of 32 states + words (+ pad), nothing else
        f = coded[:512].view("<u2").astype(np.int64)
        assert f.sum() == 4096 and np.array_equal(f > 0, np.bincount(raw, minlength=256) > 0)
        nseg = -(-n // rans.SEGMENT)
        nw = coded[512 : 512 + 4 * nseg].view("<u4").astype(np.int64)
        assert coded.size == 512 + 4 * nseg + int((128 + 2 * nw + 2 * (nw & 1)).sum())
        # a damaged section is refused, not mis-decoded silently
        if coded.size > 700 and kind == 0:
            bad = coded.copy()
            bad[600] ^= 0x55
            try:
                out = rans.decode(bad, n)
                assert not np.array_equal(out, raw)
            except ValueError:
                pass


def test_coded_size_is_close_to_the_empirical_entropy():
    rng = np.random.default_rng(9)
    for n in (50_000, 400_000):
        raw = _exponent_like(rng, n)
        p = np.bincount(raw, minlength=256) / n
        h_bits = -(p[p > 0] * np.log2(p[p > 0])).sum() * n
        coded = rans.encode(raw)
        nseg = -(-n // rans.SEGMENT)
        word_bits = 16 * int(coded[512 : 512 + 4 * nseg].view("<u4").sum())
        # what the words do not hold sits in the final lane states: at most 16 bits above the start state each
        assert word_bits + 16 * rans.LANES * nseg >= h_bits * 0.999  # no coder beats the entropy of the data
        assert word_bits <= h_bits * 1.03                            # a 12-bit static model costs a few per cent
        assert coded.size < 0.45 * n                     # about 2.6 bits per exponent byte here


@pytest.mark.parametrize("dtype", [BF16, FP32])
@pytest.mark.parametrize("n,block", [(70_001, 512), (8192, 64), (1000, 16), (40_000, 1)])
def test_message_level_stage_is_lossless_and_never_longer(oracle, dtype, n, block):
    name = "bf16" if dtype == BF16 else "fp32"
    traj = [wl.as_bits(w) for w in wl.trajectory(n, name, 77 + n, 2, "adam")]
    cache = oracle.cache_init(None, n, dtype)  # from empty caches: a large payload on the first step
    for w in traj:
        msg, wire, pay, chg = oracle.encode(w, cache, dtype, block)
        assert rans.payload_bytes_from_bitmap(msg, n, block, dtype) == pay
        coded = rans.entropy_encode_message(msg, n, dtype, block)
        assert coded.size <= msg.size
        assert np.array_equal(rans.entropy_decode_message(coded, n, dtype, block), msg)
        if pay > 20_000:
            assert coded.size < msg.size - pay // 2  # exponents of Gaussian weights compress well


def test_five_bit_packing_by_hand():
    """Exponents 1, 2, 3 of one block: 1 | 2 << 5 | 3 << 10 = 0x0C41, little-endian, one spare bit; two blocks
    of 3 and 1 values start on byte boundaries."""
    lens = np.array([3, 1])
    packed = np.array([0x41, 0x0C, 0x1F], np.uint8)
    assert rans.unpack_fp16_payload(packed, lens).tolist() == [1, 2, 3, 31]
    assert rans.pack_fp16_payload(np.array([1, 2, 3, 31], np.uint8), lens).tolist() == [0x41, 0x0C, 0x1F]
    with pytest.raises(ValueError):
        rans.unpack_fp16_payload(packed, np.array([3]))  # a byte too many for one block of three


def test_the_32_entry_table_is_the_256_entry_one_cut_short():
    """Symbols below 32: the coded section with 32 table entries is the one with 256 entries without the 224
    zero entries (same model, same segments), and decodes to the same symbols; a larger symbol is refused."""
    rng = np.random.default_rng(5)
    for n in (1, 31, 4096, 4097, 50_000):
        raw = np.minimum(rng.geometric(0.3, n) + 9, 31).astype(np.uint8)
        wide, narrow = rans.encode(raw), rans.encode(raw, 32)
        assert narrow.size == wide.size - 448 == rans.coded_bound(n, 32) - (rans.coded_bound(n) - wide.size)
        assert np.array_equal(narrow[:64], wide[:64]) and not wide[64:512].any()
        assert np.array_equal(narrow[64:], wide[512:])
        assert np.array_equal(rans.decode(narrow, n, 32), raw)
    with pytest.raises(ValueError):
        rans.encode(np.array([3, 32], np.uint8), 32)
    bad = rans.encode(np.full(100, 7, np.uint8), 32)
    bad[0] ^= 1  # the table no longer sums to 4096
    with pytest.raises(ValueError):
        rans.decode(bad, 100, 32)


@pytest.mark.parametrize("n,block", [(70_001, 512), (8192, 64), (1000, 32), (40_003, 4096), (5_000, 16), (30_001, 4),
                                     (25_000, 1), (20_003, 8), (9_999, 2)])
def test_message_level_stage_on_fp16_exponents(oracle, n, block):
    """fp16: the payload holds five bits per exponent, every changed block starting on a byte boundary.  The
    symbols the stage codes are the exponents themselves: unpacked they equal the exponent fields of the changed
    blocks' values (taken with the codec oracle's split), packing them again gives the payload back, and the
    stage stays lossless, never lengthens a message and shortens large payloads to well under five bits per
    exponent."""
    FP16 = 2
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "fp16", 177 + n, 2, "adam")]
    cache = oracle.cache_init(None, n, FP16)
    for w in traj:
        msg, wire, pay, chg = oracle.encode(w, cache, FP16, block)
        assert rans.payload_bytes_from_bitmap(msg, n, block, FP16) == pay
        nb = -(-n // block)
        assert pay <= (nb - 1) * ((5 * block + 7) // 8) + (5 * (n - (nb - 1) * block) + 7) // 8
        pay_off = msg.size - pay
        lens = rans.changed_block_lengths(msg, n, block)
        symbols = rans.unpack_fp16_payload(msg[pay_off:], lens)
        exp, _ = oracle.split(w, FP16)
        flags = np.unpackbits(msg[: -(-nb // 8)], bitorder="little")[:nb].astype(bool)
        assert np.array_equal(symbols, exp[np.repeat(flags, block)[:n]])
        assert np.array_equal(rans.pack_fp16_payload(symbols, lens), msg[pay_off:])
        coded = rans.entropy_encode_message(msg, n, FP16, block)
        assert coded.size <= msg.size
        assert np.array_equal(rans.entropy_decode_message(coded, n, FP16, block), msg)
        if pay > 20_000:
            assert coded.size < msg.size - pay // 3  # under 3.4 of the 5 bits
