"""Pins of the CPU oracle against what the paper and IEEE-754 fix (no GPU, no CUDA path).

Each test is aimed at one plausible mistake: a wrong field position (frexp pin), a lost bit
(bijection), a wrong block boundary / bit order / section offset (hand-worked fixtures,
shadow bookkeeping), a dropped term in the byte count or the gain (closed forms).
"""
import os

import numpy as np
import pytest
import torch

from helpers import BF16, FP16, FP32, FORMAT, ieee_fields, pack_fields, parse_golden, shadow_blocks, shadow_blocks_packed
from paper_2609_04609_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ per-value split / merge


def _check_fields(oracle, bits, dtype):
    p = FORMAT[dtype][1]
    sign, E, M = ieee_fields(bits, dtype)
    exp, sm = oracle.split(bits, dtype)
    assert np.array_equal(exp.astype(np.int64), E), "exponent field differs from the IEEE definition"
    assert np.array_equal((sm >> p).astype(np.int64), sign), "sign is not bit m-1 of sm"
    ok = M >= 0
    assert np.array_equal((sm & ((1 << p) - 1)).astype(np.int64)[ok], M[ok]), "mantissa differs"
    assert np.all(sm < (1 << (p + 1)))
    # bijection: nothing is lost (covers NaN payloads, which have no numeric definition)
    assert np.array_equal(oracle.merge(exp, sm, dtype), bits)


def test_split_bf16_every_pattern_matches_ieee_definition(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    _check_fields(oracle, bits, BF16)


def test_split_fp16_every_pattern_matches_ieee_definition(oracle):
    bits = np.arange(65536, dtype=np.uint16)
    _check_fields(oracle, bits, FP16)
    exp, _ = oracle.split(bits, FP16)
    assert exp.max() == 31


def test_split_fp32_random_and_special_patterns_match_ieee_definition(oracle):
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 2**32, size=1 << 21, dtype=np.uint64).astype(np.uint32)
    special = np.array(
        [0x00000000, 0x80000000, 0x00000001, 0x807FFFFF, 0x00800000, 0x7F7FFFFF, 0x7F800000, 0xFF800000,
         0x7FC00000, 0xFFFFFFFF, 0x7F800001, 0x3F800000, 0xBFC00000], dtype=np.uint32)
    # every exponent value with extreme mantissas and both signs
    e = np.arange(256, dtype=np.uint32)
    grid = np.concatenate([(s << 31) | (e << 23) | m for s in (0, 1) for m in (0, 1, 0x400000, 0x7FFFFF)])
    _check_fields(oracle, np.concatenate([bits, special, grid.astype(np.uint32)]), FP32)


def test_split_fp32_every_one_of_the_2_to_32_patterns(tmp_path):
    """All 2^32 binary32 patterns through the oracle's split and merge against the numeric field definition
    (frexpf / ldexpf), in a small C program of the test suite built together with the oracle's source: see
    tests/exhaustive_fp32_fields.c.  About ten seconds on eight cores."""
    import subprocess

    here = os.path.dirname(os.path.abspath(__file__))
    exe = str(tmp_path / "exhaustive_fp32_fields")
    src = [os.path.join(here, "exhaustive_fp32_fields.c"), os.path.join(here, "..", "oracle", "ciera_oracle.c")]
    built = subprocess.run(["gcc", "-O2", "-fopenmp", "-o", exe] + src + ["-lm"])
    if built.returncode != 0:  # no OpenMP runtime on this machine: one thread, about a minute
        subprocess.run(["gcc", "-O2", "-o", exe] + src + ["-lm"], check=True)
    out = subprocess.run([exe], capture_output=True, text=True, timeout=1200)
    assert out.returncode == 0 and out.stdout.strip() == "ok 4294967296", out.stdout + out.stderr


# ------------------------------------------------------------------ hand-worked fixtures


@pytest.mark.parametrize("name", ["bf16_worked_example.txt", "fp32_worked_example.txt",
                                  "small_block_worked_example.txt", "fp16_worked_example.txt"])
def test_hand_worked_examples(oracle, name):
    for st in parse_golden(os.path.join(GOLDEN, name)):
        dtype = {"bf16": BF16, "fp32": FP32, "fp16": FP16}[st["dtype"][0]]
        block = int(st["block"][0])
        w = np.array([int(x, 16) for x in st["weights"]], np.uint32 if dtype == FP32 else np.uint16)
        hexb = lambda key: np.array([int(x, 16) for x in st.get(key, [])], np.uint8)
        cache = hexb("cache_before").copy()
        n = w.size
        msg, wire, pay, chg = oracle.encode(w, cache, dtype, block)
        bm, sm, payload = hexb("bitmap"), hexb("sm"), hexb("payload")
        sm_off = -(-bm.size // 16) * 16
        pay_off = sm_off + -(-sm.size // 16) * 16
        expect = np.zeros(pay_off + payload.size, np.uint8)
        expect[: bm.size] = bm
        expect[sm_off : sm_off + sm.size] = sm
        expect[pay_off:] = payload
        assert np.array_equal(msg, expect)
        assert wire == expect.size and pay == payload.size
        assert chg == int(st["changed_blocks"][0])
        assert np.array_equal(cache, hexb("cache_after"))
        assert oracle.paper_bytes(n, dtype, block, pay) == int(st["paper_bytes"][0])
        # receiver starting from the same cache_before reproduces the weights bit for bit
        cache_r = hexb("cache_before").copy()
        assert np.array_equal(oracle.decode(msg, cache_r, dtype, block), w)
        assert np.array_equal(cache_r, hexb("cache_after"))


# ------------------------------------------------------------------ exhaustive bf16 x cache


def test_exhaustive_bf16_patterns_times_cache_values(oracle):
    """All 256 cache values x all 65 536 bf16 patterns (16.7 M values): the complete
    per-value map, through encode and decode, against numerically derived exponents."""
    pat = np.arange(65536, dtype=np.uint16)
    _, E, _ = ieee_fields(pat, BF16)
    w = np.tile(pat, 256)
    exp_true = np.tile(E.astype(np.uint8), 256)
    cache0 = np.repeat(np.arange(256, dtype=np.uint8), 65536)
    block = 64
    n = w.size
    cache_s = cache0.copy()
    msg, wire, pay, chg = oracle.encode(w, cache_s, BF16, block)
    bitmap, payload, cache_after, chg_mask = shadow_blocks(exp_true, cache0, block)
    sm_off, pay_off = oracle.sm_offset(n, block), oracle.payload_offset(n, BF16, block)
    assert np.array_equal(msg[: bitmap.size], bitmap)
    assert not msg[bitmap.size : sm_off].any()
    assert np.array_equal(msg[pay_off:], payload)
    assert pay == payload.size and chg == int(chg_mask.sum())
    assert np.array_equal(cache_s, cache_after) and np.array_equal(cache_s, exp_true)
    # sm byte = sign<<7 | mantissa, from the numeric fields
    sign, _, M = ieee_fields(pat, BF16)
    ok = M >= 0
    sm_true = (sign << 7 | np.where(ok, M, 0)).astype(np.uint8)
    got = msg[sm_off : sm_off + 65536]
    assert np.array_equal(got[ok], sm_true[ok])
    cache_r = cache0.copy()
    assert np.array_equal(oracle.decode(msg, cache_r, BF16, block), w)
    assert np.array_equal(cache_r, exp_true)


# ------------------------------------------------------------------ byte count and layout


@pytest.mark.parametrize("dtype", [BF16, FP32])
def test_transmitted_bytes_formula_and_shadow_bookkeeping(oracle, dtype):
    """wire content and the paper's count S_{s+m} + S_bm + sum of changed-block lengths
    (Section 3.2), over ragged sizes and every supported kind of block size."""
    rng = np.random.default_rng(11 + dtype)
    m_bytes = 1 if dtype == BF16 else 3
    for n, block in [(1, 64), (5, 2), (63, 64), (64, 64), (65, 64), (1000, 128), (4097, 512), (12345, 4096),
                     (70000, 512), (33, 1), (1024, 16), (2049, 1024), (8193, 1), (10001, 2), (9003, 4),
                     (20001, 8)]:
        hi = 1 << (16 if dtype == BF16 else 32)
        w_prev = rng.integers(0, hi, size=n, dtype=np.uint64).astype(np.uint16 if dtype == BF16 else np.uint32)
        w = w_prev.copy()
        flip = rng.random(n) < 0.02
        w[flip] = rng.integers(0, hi, size=int(flip.sum()), dtype=np.uint64).astype(w.dtype)
        cache0 = oracle.cache_init(w_prev, n, dtype)
        cache = cache0.copy()
        msg, wire, pay, chg = oracle.encode(w, cache, dtype, block)
        _, E, _ = ieee_fields(w, dtype)
        bitmap, payload, cache_after, chg_mask = shadow_blocks(E.astype(np.uint8), cache0, block)
        nb = -(-n // block)
        lens = np.minimum(block, n - np.arange(nb) * block)
        assert pay == int(lens[chg_mask].sum())
        s_bm = -(-nb // 8)
        assert oracle.paper_bytes(n, dtype, block, pay) == n * m_bytes + s_bm + pay
        sm_off = -(-s_bm // 16) * 16
        pay_off = sm_off + -(-(n * m_bytes) // 16) * 16
        assert (oracle.sm_offset(n, block), oracle.payload_offset(n, dtype, block)) == (sm_off, pay_off)
        assert wire == pay_off + pay and msg.size == wire
        assert oracle.message_capacity(n, dtype, block) == pay_off + n
        assert np.array_equal(msg[:s_bm], bitmap)
        assert not msg[s_bm:sm_off].any() and not msg[sm_off + n * m_bytes : pay_off].any()
        assert np.array_equal(msg[pay_off:], payload)
        assert np.array_equal(cache, cache_after)
        cache_r = cache0.copy()
        assert np.array_equal(oracle.decode(msg, cache_r, dtype, block), w)
        assert np.array_equal(cache_r, cache_after)


def test_fp32_sm_is_three_little_endian_bytes(oracle):
    w = np.array([0xBFC00000, 0x12345678], np.uint32)  # second: sign 0, exp 0x24, mant 0x345678
    cache = oracle.cache_init(w, 2, FP32)
    msg, *_ = oracle.encode(w, cache, FP32, 64)
    off = oracle.sm_offset(2, 64)
    assert list(msg[off : off + 6]) == [0x00, 0x00, 0xC0, 0x78, 0x56, 0x34]


# ------------------------------------------------------------------ special cases


@pytest.mark.parametrize("dtype", [BF16, FP32])
def test_special_cases(oracle, dtype):
    rng = np.random.default_rng(3)
    n, block = 5000, 512
    m_bytes = 1 if dtype == BF16 else 3
    hi = 1 << (16 if dtype == BF16 else 32)
    w = rng.integers(0, hi, size=n, dtype=np.uint64).astype(np.uint16 if dtype == BF16 else np.uint32)
    s_bm = -(-(-(-n // block)) // 8)
    # unchanged weights: empty bitmap, empty payload, message is sm only
    cache = oracle.cache_init(w, n, dtype)
    msg, wire, pay, chg = oracle.encode(w, cache, dtype, block)
    assert pay == 0 and chg == 0 and not msg[:s_bm].any()
    assert wire == oracle.payload_offset(n, dtype, block)
    assert oracle.paper_bytes(n, dtype, block, pay) == n * m_bytes + s_bm
    # a cache that is wrong everywhere: payload is exp(W) in order, every bit set
    exp, _ = oracle.split(w, dtype)
    cache = (exp + 1).astype(np.uint8)
    msg, wire, pay, chg = oracle.encode(w, cache, dtype, block)
    assert pay == n and chg == -(-n // block)
    assert np.array_equal(msg[oracle.payload_offset(n, dtype, block) :], exp)
    assert oracle.paper_bytes(n, dtype, block, pay) == n * m_bytes + s_bm + n
    bits = np.unpackbits(msg[:s_bm], bitorder="little")
    assert bits[: -(-n // block)].all() and not bits[-(-n // block) :].any()
    # B >= N: one block
    cache = oracle.cache_init(None, n, dtype)
    msg, wire, pay, chg = oracle.encode(w, cache, dtype, 8192)
    assert chg == 1 and pay == n and msg[0] == 1
    # N = 0: empty message
    e = np.zeros(0, w.dtype)
    msg, wire, pay, chg = oracle.encode(e, np.zeros(0, np.uint8), dtype, block)
    assert (msg.size, wire, pay, chg) == (0, 0, 0, 0)
    assert oracle.decode(msg, np.zeros(0, np.uint8), dtype, block).size == 0


def test_zero_cache_marks_blocks_with_nonzero_exponent_only(oracle):
    # block 0: zeros and subnormals (exponent field 0) ; block 1: one normal value
    w = np.array([0x0000, 0x8000, 0x0001, 0x807F, 0x0000, 0x3F80, 0x0000, 0x0000], np.uint16)
    cache = oracle.cache_init(None, 8, BF16)
    assert not cache.any()
    msg, wire, pay, chg = oracle.encode(w, cache, BF16, 4)
    assert msg[0] == 0b10 and chg == 1 and pay == 4
    assert list(cache) == [0, 0, 0, 0, 0, 0x7F, 0, 0]


# ------------------------------------------------------------------ trajectories


@pytest.mark.parametrize("dtype,model", [("bf16", "gaussian"), ("bf16", "clustered"), ("fp32", "adam")])
def test_round_trip_and_cache_invariant_along_a_trajectory(oracle, dtype, model):
    """decode(encode(W_t, cache), cache) == W_t bitwise for every t, and after each
    step sender cache == receiver cache == exponents(W_t)  (Algorithm 1; Section 4.5)."""
    d = BF16 if dtype == "bf16" else FP32
    n_shards, block = 4, 512
    n = 1024 * 512 // 8
    per = n // n_shards
    traj = [wl.as_bits(w) for w in wl.trajectory(n, dtype, 1235, 3, model)]
    cs = [oracle.cache_init(traj[0][p * per : (p + 1) * per], per, d) for p in range(n_shards)]
    cr = [c.copy() for c in cs]
    total_changed = 0
    for t in range(1, 4):
        for p in range(n_shards):
            w = traj[t][p * per : (p + 1) * per]
            msg, wire, pay, chg = oracle.encode(w, cs[p], d, block)
            out = oracle.decode(msg, cr[p], d, block)
            assert np.array_equal(out, w)
            _, E, _ = ieee_fields(w, d)
            assert np.array_equal(cs[p], cr[p]) and np.array_equal(cs[p], E.astype(np.uint8))
            total_changed += chg
    assert total_changed > 0


def test_bitmap_equals_exponent_change_between_iterations(oracle):
    """The bitmap is exactly 'block holds a value whose exponent field differs between
    iteration t-1 and t' (Section 2.2-2.3 definition of change rates)."""
    n, block = 40000, 64
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 99, 2, "adam")]
    cache = oracle.cache_init(traj[0], n, BF16)
    for t in (1, 2):
        msg, _, _, chg = oracle.encode(traj[t], cache, BF16, block)
        _, e_prev, _ = ieee_fields(traj[t - 1], BF16)
        _, e_now, _ = ieee_fields(traj[t], BF16)
        nb = -(-n // block)
        d = np.zeros(nb * block, bool)
        d[:n] = e_prev != e_now
        want = d.reshape(nb, block).any(1)
        got = np.unpackbits(msg[: -(-nb // 8)], bitorder="little")[:nb].astype(bool)
        assert np.array_equal(got, want) and chg == int(want.sum())


# ------------------------------------------------------------------ change statistics


@pytest.mark.parametrize("c,block", [(0.001, 512), (0.01, 64), (0.003, 256)])
def test_block_change_rate_follows_closed_form(oracle, c, block):
    """i.i.d. element changes at rate c: a block stays reusable with probability (1-c)^B
    (Section 2.3)."""
    n = 1 << 21
    gen = wl.make_generator(5)
    w0 = wl.init_weights(n, "bf16", gen)
    w1 = wl.inject_exponent_changes(w0, gen, c)
    cache = oracle.cache_init(wl.as_bits(w0), n, BF16)
    _, _, pay, chg = oracle.encode(wl.as_bits(w1), cache, BF16, block)
    nb = n // block
    q_expect = 1.0 - (1.0 - c) ** block
    sigma = np.sqrt(q_expect * (1 - q_expect) / nb)
    assert abs(chg / nb - q_expect) < 4 * sigma + 1e-12
    assert pay == chg * block


def test_shard_unchanged_probability_closed_form(oracle):
    """Pr(shard unchanged) = (1-c)^n (Section 2.3), on 4000 one-block units of n = 2000."""
    n_units, n, c = 4000, 2000, 0.001
    gen = wl.make_generator(17)
    w0 = wl.init_weights(n_units * n, "bf16", gen)
    w1 = wl.inject_exponent_changes(w0, gen, c)
    b0, b1 = wl.as_bits(w0), wl.as_bits(w1)
    unchanged = 0
    for u in range(n_units):
        cache = oracle.cache_init(b0[u * n : (u + 1) * n], n, BF16)
        _, _, _, chg = oracle.encode(b1[u * n : (u + 1) * n], cache, BF16, 4096)
        unchanged += chg == 0
    p = (1 - c) ** n
    assert abs(unchanged / n_units - p) < 4 * np.sqrt(p * (1 - p) / n_units)


def test_generators_reach_the_regimes_the_paper_reports(oracle):
    """Post-warm-up regime: >= 96 % of exponents unchanged under the literal update models;
    the clustered model gives block change rate ~ f at B = 512 with a sub-percent element rate."""
    n = 1 << 20
    for model, kw in (("gaussian", {}), ("adam", {}), ("clustered", {"f": 0.22})):
        w0, w1 = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 1234, 1, model, **kw)]
        e0, _ = oracle.split(w0, BF16)
        e1, _ = oracle.split(w1, BF16)
        c = float((e0 != e1).mean())
        assert c < 0.04
        if model == "clustered":
            cache = e0.copy()
            _, _, _, chg = oracle.encode(w1, cache, BF16, 512)
            q = chg / (n // 512)
            assert 0.18 < q < 0.26 and c < 0.01


# ------------------------------------------------------------------ gain formula


def test_gain_hand_computed_cases(oracle):
    for line in open(os.path.join(GOLDEN, "gain_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, dt, n, block, q, world, alpha, beta, th, tc, td, ov, table, want = line.split()
        tbl = None if table == "none" else [tuple(float(x) for x in p.split(":")) for p in table.split(",")]
        got = oracle.gain(int(n), BF16 if dt == "bf16" else FP32, int(block), float(q), int(world), float(alpha),
                          float(beta), tbl, float(th), float(tc), float(td), bool(int(ov)))
        assert got == pytest.approx(float(want), rel=1e-9), name


def test_gain_sign_cases(oracle):
    """q = 1 can never pay (more bytes than raw), gain falls with q, and the sender-side
    terms vanish only when overlapped (Section 3.2)."""
    kw = dict(n=131072, dtype=BF16, block=512, world=16, alpha=1e-5, beta=8e9)
    assert oracle.gain(q=1.0, t_decmp=0.0, overlapped=True, **kw) < 0
    gs = [oracle.gain(q=q, t_decmp=1e-6, overlapped=True, **kw) for q in (0, 0.1, 0.22, 0.5, 0.9, 1.0)]
    assert all(a > b for a, b in zip(gs, gs[1:]))
    g_ov = oracle.gain(q=0.2, t_hash=2e-6, t_cmp=3e-6, t_decmp=1e-6, overlapped=True, **kw)
    g_no = oracle.gain(q=0.2, t_hash=2e-6, t_cmp=3e-6, t_decmp=1e-6, overlapped=False, **kw)
    assert g_ov - g_no == pytest.approx(5e-6, rel=1e-9)
    # a fast link makes every gain non-positive once decompression costs anything real
    fast = dict(kw, beta=1e13, alpha=0.0)
    assert oracle.gain(q=0.22, t_decmp=5e-6, overlapped=True, **fast) < 0


# ------------------------------------------------------------------ fp16: packed sections


def test_exhaustive_fp16_patterns_times_cache_values(oracle):
    """All 32 cache values x all 65 536 fp16 patterns: the complete per-value map through encode and
    decode, against numerically derived fields and a numpy restatement of the bit packing."""
    pat = np.arange(65536, dtype=np.uint16)
    sign, E, M = ieee_fields(pat, FP16)
    w = np.tile(pat, 32)
    exp_true = np.tile(E.astype(np.uint8), 32)
    cache0 = np.repeat(np.arange(32, dtype=np.uint8), 65536)
    block = 64
    n = w.size
    cache_s = cache0.copy()
    msg, wire, pay, chg = oracle.encode(w, cache_s, FP16, block)
    bitmap, payload, cache_after, chg_mask = shadow_blocks_packed(exp_true, cache0, block, 5)
    sm_off, pay_off = oracle.sm_offset(n, block), oracle.payload_offset(n, FP16, block)
    assert np.array_equal(msg[: bitmap.size], bitmap)
    assert np.array_equal(msg[pay_off:], payload) and pay == payload.size and chg == int(chg_mask.sum())
    assert np.array_equal(cache_s, cache_after) and np.array_equal(cache_s, exp_true)
    # sm = sign << 10 | mantissa from the numeric fields (NaN payloads are covered by the round trip)
    ok = M >= 0
    sm_true = np.where(ok, sign << 10 | np.where(ok, M, 0), 0)
    got = msg[sm_off : sm_off + 65536 * 11 // 8]
    want = pack_fields(sm_true, 11)
    # compare value by value where the mantissa has a numeric definition
    got_fields = np.unpackbits(got, bitorder="little").reshape(65536, 11)
    want_fields = np.unpackbits(want, bitorder="little").reshape(65536, 11)
    assert np.array_equal(got_fields[ok], want_fields[ok])
    cache_r = cache0.copy()
    assert np.array_equal(oracle.decode(msg, cache_r, FP16, block), w)
    assert np.array_equal(cache_r, exp_true)


def test_fp16_byte_count_and_layout_over_ragged_sizes(oracle):
    """S_{s+m} = ceil(11 N / 8), every changed block ceil(5 L / 8) bytes, capacity = all blocks changed."""
    rng = np.random.default_rng(23)
    for n, block in [(1, 64), (5, 2), (7, 8), (63, 64), (65, 64), (1000, 128), (4097, 512), (12345, 4096), (33, 1),
                     (8193, 32), (100, 3), (1000, 4), (4099, 1), (777, 8), (2050, 2)]:
        w_prev = rng.integers(0, 1 << 16, size=n, dtype=np.uint64).astype(np.uint16)
        w = w_prev.copy()
        flip = rng.random(n) < 0.05
        w[flip] = rng.integers(0, 1 << 16, size=int(flip.sum()), dtype=np.uint64).astype(np.uint16)
        cache0 = oracle.cache_init(w_prev, n, FP16)
        cache = cache0.copy()
        msg, wire, pay, chg = oracle.encode(w, cache, FP16, block)
        _, E, _ = ieee_fields(w, FP16)
        bitmap, payload, cache_after, chg_mask = shadow_blocks_packed(E.astype(np.uint8), cache0, block, 5)
        nb = -(-n // block)
        lens = np.minimum(block, n - np.arange(nb) * block)
        assert pay == int((-(-(lens[chg_mask] * 5) // 8)).sum()) == payload.size
        s_bm, s_sm = -(-nb // 8), -(-(n * 11) // 8)
        assert oracle.paper_bytes(n, FP16, block, pay) == s_sm + s_bm + pay
        sm_off = -(-s_bm // 16) * 16
        pay_off = sm_off + -(-s_sm // 16) * 16
        assert (oracle.sm_offset(n, block), oracle.payload_offset(n, FP16, block)) == (sm_off, pay_off)
        assert wire == pay_off + pay and msg.size == wire
        assert oracle.message_capacity(n, FP16, block) == pay_off + int((-(-(lens * 5) // 8)).sum())
        assert np.array_equal(msg[:s_bm], bitmap) and np.array_equal(msg[pay_off:], payload)
        assert not msg[s_bm:sm_off].any() and not msg[sm_off + s_sm : pay_off].any()
        assert np.array_equal(cache, cache_after)
        cache_r = cache0.copy()
        assert np.array_equal(oracle.decode(msg, cache_r, FP16, block), w)
        assert np.array_equal(cache_r, cache_after)
