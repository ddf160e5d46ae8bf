"""GPU parity of the fp16 path (5-bit exponents and 11-bit sign-plus-mantissa, packed on the wire)
against the oracle: messages, lengths, counts, both caches and the reconstructed weights bit for bit."""
import numpy as np
import pytest
import torch

from harness import OracleTable, compare_caches, compare_recon, compare_step, guard, to_dev_bytes
from paper_2609_04609_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
FP16 = 2
RAGGED = [0, 1, 7, 8, 9, 15, 16, 17, 31, 33, 511, 512, 513, 1000, 4095, 4097, 8191, 8192, 8193, 8208, 16383, 16385,
          20000, 0, 70001, 131072 + 7]


@pytest.fixture(scope="module")
def rt():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_04609_b200 import ciera, runtime

    return ciera, runtime


def _run(rt, sizes, shards, block, traj_fn, zero_cache=False, label=""):
    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors(sizes, shards, "fp16", block, DEV, slack=256))
    table = OracleTable(codec.units, FP16, block, codec.cache_bytes, codec.msg_bytes)
    n = codec.weights_bytes // 2
    traj = traj_fn(n)
    first = None if zero_cache else traj[0]
    codec.init_caches(None if first is None else to_dev_bytes(first, DEV))
    table.init_caches(first)
    compare_caches(codec, table, label + " init")
    stats = []
    for t, w in enumerate(traj[1:], 1):
        codec.step(to_dev_bytes(w, DEV))
        torch.cuda.synchronize()
        codec.check_status()
        exp = table.step(w)
        wire, chg = compare_step(codec, exp, w, f"{label} t={t}")
        compare_caches(codec, table, f"{label} t={t}")
        compare_recon(codec, exp, w, FP16, f"{label} t={t}")
        stats.append((int(chg.sum()), codec.n_blocks()))
    return stats


@pytest.mark.parametrize("block", [1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096])
def test_fp16_ragged_units_every_block_size(rt, block):
    """Units shorter than a block, not multiples of 8 / of the block / of the tile, empty units;
    random bit patterns (NaN, Inf, subnormals, both zeros included)."""
    def traj(n):
        rng = np.random.default_rng(200 + block)
        w0 = rng.integers(0, 1 << 16, n, dtype=np.uint64).astype(np.uint16)
        w1 = w0.copy()
        flip = rng.random(n) < 0.01
        w1[flip] = rng.integers(0, 1 << 16, int(flip.sum()), dtype=np.uint64).astype(np.uint16)
        w3 = rng.integers(0, 1 << 16, n, dtype=np.uint64).astype(np.uint16)
        return [w0, w1, w1.copy(), w3]

    stats = _run(rt, RAGGED, 1, block, traj, label=f"fp16-ragged-B{block}")
    assert stats[1][0] == 0


@pytest.mark.parametrize("block,model,kw", [(512, "adam", {}), (512, "clustered", {"f": 0.22}), (64, "clustered", {"f": 0.5}),
                                            (32, "adam", {}), (16, "adam", {}), (8, "adam", {}), (4, "adam", {}),
                                            (2, "adam", {}), (1, "adam", {}), (1, "clustered", {"f": 0.3})])
def test_fp16_reduced_moe_layer(rt, block, model, kw):
    sizes = [r * c for r, c in wl.olmoe_layer_shapes(2)] + [70_001, 17, 0]
    stats = _run(rt, sizes, 4, block, lambda n: [wl.as_bits(w) for w in wl.trajectory(n, "fp16", 31 + block, 3, model, **kw)],
                 label=f"fp16-moe-B{block}-{model}")
    assert stats[-1][0] > 0
    _run(rt, sizes, 4, block, lambda n: [wl.as_bits(w) for w in wl.trajectory(n, "fp16", 32 + block, 1, model, **kw)],
         zero_cache=True, label=f"fp16-moe-zero-B{block}")


@pytest.mark.parametrize("block,c", [(512, 0.001), (64, 0.01), (4096, 0.3), (32, 0.05), (16, 0.1), (8, 0.01), (2, 0.3), (1, 0.02)])
def test_fp16_long_units_of_many_tiles(rt, block, c):
    def traj(n):
        gen = wl.make_generator(4242 + block)
        w0 = wl.init_weights(n, "fp16", gen)
        w1 = wl.inject_exponent_changes(w0, gen, c)
        w2 = wl.inject_exponent_changes(w1, gen, c)
        return [wl.as_bits(w) for w in (w0, w1, w2)]

    _run(rt, [3_000_000 + 123, 600_000], 1, block, traj, label=f"fp16-long-B{block}")


def test_fp16_sizes_and_limits(rt):
    ciera, runtime = rt
    from oracle import ciera_oracle as ora
    for n in (0, 1, 7, 8, 9, 1000, 131072, 70001):
        for block in (1, 2, 4, 8, 32, 512, 4096):
            assert ciera.payload_offset(n, FP16, block) == ora.payload_offset(n, FP16, block)
            assert ciera.message_capacity(n, FP16, block) == ora.message_capacity(n, FP16, block)
            assert ciera.message_bytes(n, FP16, block, 17) == ora.paper_bytes(n, FP16, block, 17)
    codec = runtime.LayerCodec.from_tensors([1000], 1, "fp16", 8, DEV)  # every block size from 1 value on
    with pytest.raises(ciera.CieraError) as e:
        codec.init_hash_cache(None)
        codec.encode_hashed(codec.weights_out)  # the hashed sender: blocks of 16 values and more
    assert e.value.status == ciera.ERR_UNSUPPORTED
    codec = runtime.LayerCodec.from_tensors([1000], 1, "fp16", 64, DEV)
    codec.init_hash_cache(None)  # the hashed sender and the entropy stage take fp16 (test_gpu_hashed.py, test_gpu_entropy.py)
    # the gain rule charges 5 exponent bits per value
    g16, _ = ciera.should_compress(1 << 20, FP16, 512, 0.25, world_size=8, alpha=0.0, beta=1e9)
    want = 7 * ((1 << 21) - ((1 << 20) * 11 / 8 + 256 + 0.25 * (1 << 20) * 5 / 8)) / 1e9
    assert abs(g16 - want) < 1e-12
    assert abs(g16 - ora.gain(1 << 20, FP16, 512, 0.25, 8, 0.0, 1e9)) < 1e-12
