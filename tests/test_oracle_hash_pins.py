"""Pins of the oracle's hash-based change detection (Section 3.1; Algorithm 1, sender).  No GPU.

What is fixed from outside: the SplitMix64 generator's published output streams; the exact
comparison path (already pinned) as the predicate the hash stands for; the algebra of the
construction (every single-word change is detected with certainty, because the output function
is a bijection).  The 128-bit values themselves follow a construction the paper does not print,
so they have no external reference beyond these ("parity unpinned" for the hash values)."""
import numpy as np
import pytest

from helpers import BF16, FP32
from paper_2609_04609_b200 import workloads as wl

MASK = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15
GAMMA2 = 0xD1342543DE82EF95  # the second hash's generator runs on an increment of its own
HASHES = ((0, GAMMA), (0x6A09E667F3BCC908, GAMMA2))  # (seed, increment) of the two 64-bit hashes


def test_splitmix64_published_streams(oracle):
    # first outputs of the reference generator for seed 1234567 and for seed 0
    assert oracle.splitmix64_stream(1234567, 5) == [6457827717110365317, 3203168211198807973, 9817491932198370423,
                                                    4593380528125082431, 16408922859458223821]
    assert oracle.splitmix64_stream(0, 3) == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_zero_blocks_tie_the_hash_to_the_generator_stream(oracle):
    """All-zero exponents: the per-word terms are the generator's own outputs for the seed, so
    H_s = mix(L + sum of the first ceil(L/8) outputs)."""
    for L in (1, 7, 8, 9, 64, 512, 4096, 13):
        m = -(-L // 8)
        for h, (seed, gamma) in zip(oracle.hash128(np.zeros(L, np.uint8)), HASHES):
            acc = sum(oracle.splitmix64_stream(seed, m, gamma)) & MASK
            assert h == oracle.splitmix64_mix((acc + L) & MASK)
    # the increment argument itself: the generator's own increment gives the published stream
    assert oracle.splitmix64_stream(1234567, 5, GAMMA) == oracle.splitmix64_stream(1234567, 5)
    assert GAMMA2 % 2 == 1  # odd: the generator's state runs through all 2^64 values


def test_mix_is_a_bijection_on_samples_and_fixes_zero(oracle):
    """The two multipliers are odd and xor-shifts are invertible: invert mix step by step."""
    def unxorshift(z, s):
        x = z
        for _ in range(64 // s + 1):
            x = z ^ (x >> s)
        return x

    inv1 = pow(0xBF58476D1CE4E5B9, -1, 1 << 64)
    inv2 = pow(0x94D049BB133111EB, -1, 1 << 64)
    rng = np.random.default_rng(1)
    assert oracle.splitmix64_mix(0) == 0
    for z in [1, MASK, GAMMA] + [int(v) for v in rng.integers(0, 1 << 63, 200)]:
        y = oracle.splitmix64_mix(z)
        x = unxorshift(y, 31)
        x = (x * inv2) & MASK
        x = unxorshift(x, 27)
        x = (x * inv1) & MASK
        x = unxorshift(x, 30)
        assert x == z


def test_every_single_byte_change_and_every_word_swap_changes_both_halves(oracle):
    rng = np.random.default_rng(2)
    base = rng.integers(0, 256, 64, dtype=np.uint8)
    h0 = oracle.hash128(base)
    for pos in range(64):
        for delta in (1, 2, 0x80, 0xFF):
            v = base.copy()
            v[pos] ^= delta
            h = oracle.hash128(v)
            assert h[0] != h0[0] and h[1] != h0[1]
    for a in range(8):
        for b in range(a + 1, 8):
            v = base.copy().reshape(8, 8)
            v[[a, b]] = v[[b, a]]
            if not np.array_equal(v.reshape(-1), base):
                h = oracle.hash128(v.reshape(-1))
                assert h[0] != h0[0] and h[1] != h0[1]
    # the length is part of the hash: a block and the same block with a zero byte appended differ
    assert oracle.hash128(base[:56]) != oracle.hash128(np.concatenate([base[:56], np.zeros(1, np.uint8)]))
    assert oracle.hash128(np.zeros(8, np.uint8)) != oracle.hash128(np.zeros(16, np.uint8))
    # the two halves are different functions
    assert h0[0] != h0[1]


def test_no_collisions_among_many_random_blocks(oracle):
    rng = np.random.default_rng(3)
    seen = set()
    for _ in range(20000):
        L = int(rng.choice([16, 64, 100, 512]))
        blk = rng.integers(120, 130, L, dtype=np.uint8)  # exponents cluster in a narrow range
        seen.add((L, blk.tobytes(), oracle.hash128(blk)))
    by_hash = {}
    for L, raw, h in seen:
        assert by_hash.setdefault(h, (L, raw)) == (L, raw)


@pytest.mark.parametrize("dtype", [BF16, FP32])
@pytest.mark.parametrize("n,block", [(5, 2), (1000, 16), (4097, 64), (70001, 512), (12345, 4096), (33, 1), (8192, 256)])
def test_hashed_sender_equals_exact_sender(oracle, dtype, n, block):
    """The hash stands for the predicate "the block's exponents differ from the previous ones":
    message for message, the hashed sender equals the exact-comparison sender over a trajectory
    (also from empty caches), and its HashCache always equals the hashes of the last sent exponents."""
    name = "bf16" if dtype == BF16 else "fp32"
    traj = [wl.as_bits(w) for w in wl.trajectory(n, name, 900 + n, 3, "adam")]
    for from_zero in (False, True):
        cache = oracle.cache_init(None if from_zero else traj[0], n, dtype)
        hc = oracle.hash_cache_init(None if from_zero else traj[0], n, dtype, block)
        for w in traj[1:] + [traj[-1]]:  # the repeated last iterate changes nothing
            m1, wire1, pay1, chg1 = oracle.encode(w, cache, dtype, block)
            m2, wire2, pay2, chg2 = oracle.encode_hashed(w, hc, dtype, block)
            assert (wire1, pay1, chg1) == (wire2, pay2, chg2) and np.array_equal(m1, m2)
            # cache holds the exponents the receiver now has; the hash cache their block hashes
            nb = -(-n // block)
            want = np.array([x for k in range(nb) for x in oracle.hash128(cache[k * block : (k + 1) * block])], np.uint64)
            assert np.array_equal(hc, want)
        assert chg2 == 0


def test_python_restatement_of_the_construction(oracle):
    """An independent restatement in Python integers (guards the C code against width slips)."""
    def mix(z):
        z ^= z >> 30
        z = (z * 0xBF58476D1CE4E5B9) & MASK
        z ^= z >> 27
        z = (z * 0x94D049BB133111EB) & MASK
        return z ^ (z >> 31)

    rng = np.random.default_rng(4)
    for L in (1, 8, 9, 63, 64, 65, 512):
        blk = rng.integers(0, 256, L, dtype=np.uint8)
        want = []
        for seed, gamma in HASHES:
            acc = 0
            for j in range(-(-L // 8)):
                x = int.from_bytes(blk[8 * j : 8 * j + 8].tobytes().ljust(8, b"\0"), "little")
                acc = (acc + mix((seed + (j + 1) * gamma + x) & MASK)) & MASK
            want.append(mix((acc + L) & MASK))
        assert oracle.hash128(blk) == tuple(want)


def test_a_rearrangement_that_collides_one_hash_does_not_collide_the_other(oracle):
    """Why the two hashes run on different increments.  Swapping two words and shifting them by the distance times
    an increment g reproduces the per-word terms of the hash that runs on g -- a genuine collision of that 64-bit
    hash, for every seed.  With a common increment both halves would collide together; with different ones the
    other half tells the blocks apart, so Hash128 still detects the change."""
    rng = np.random.default_rng(6)
    for g, collides, differs in ((GAMMA, 0, 1), (GAMMA2, 1, 0)):
        for _ in range(20):
            words = [int(v) for v in rng.integers(0, 1 << 63, 4)]
            i, j = 0, 2
            moved = list(words)
            moved[i] = (words[j] + (j - i) * g) & MASK
            moved[j] = (words[i] - (j - i) * g) & MASK
            a = np.frombuffer(b"".join(w.to_bytes(8, "little") for w in words), np.uint8)
            b = np.frombuffer(b"".join(w.to_bytes(8, "little") for w in moved), np.uint8)
            assert not np.array_equal(a, b)
            ha, hb = oracle.hash128(a), oracle.hash128(b)
            assert ha[collides] == hb[collides]
            assert ha[differs] != hb[differs]
