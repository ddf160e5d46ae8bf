"""GPU parity of the sender with hash-based change detection (ciera_encode_hashed) against the
oracle's hashed sender: messages, lengths, changed-block counts and the HashCache itself, bit for
bit; the unchanged receiver path then reproduces the weights."""
import numpy as np
import pytest
import torch

from harness import guard, sender_scratch_is_clean, to_dev_bytes
from oracle import ciera_oracle as ora
from paper_2609_04609_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
WDT = {0: np.uint16, 1: np.uint32, 2: np.uint16}
VB = {0: 2, 1: 4, 2: 2}
NAME = {0: "bf16", 1: "fp32", 2: "fp16"}
RAGGED = [0, 1, 5, 15, 16, 17, 100, 511, 512, 513, 4095, 4097, 8191, 8192, 8193, 20000, 3 * 8192 + 77, 70001]


@pytest.fixture(scope="module")
def rt():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_04609_b200 import ciera, runtime

    return ciera, runtime


def _run(rt, sizes, n_shards, dtype, block, traj, from_zero=False):
    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors(sizes, n_shards, NAME[dtype], block, DEV, slack=256))
    units = codec.units
    first = None if from_zero else traj[0]

    def unit_w(w, u):
        lo = int(u["weights_off"]) // VB[dtype]
        return w[lo : lo + int(u["n_values"])]

    # oracle state: one HashCache per unit; device state: HashCache + the receiver's exponent cache
    hcs = [ora.hash_cache_init(None if first is None else unit_w(first, u), int(u["n_values"]), dtype, block)
           for u in units]
    first_dev = None if first is None else to_dev_bytes(first, DEV)
    codec.init_hash_cache(first_dev)
    codec.init_caches(first_dev)
    assert codec.plan.hash_cache_bytes == 16 * sum(h.size // 2 for h in hcs)

    def compare_hash_cache(label):
        got = codec.hash_cache.cpu().numpy()
        for i, (u, hc) in enumerate(zip(units, hcs)):
            off = ciera.unit_hash_offset(codec.plan, i)
            assert np.array_equal(got[off : off + 8 * hc.size].view(np.uint64), hc), f"{label}: HashCache of unit {i}"

    compare_hash_cache("init")
    changed_total = []
    for t, w in enumerate(traj[1:], 1):
        wd = to_dev_bytes(w, DEV)
        codec.encode_hashed(wd)
        codec.transport()
        codec.decode()
        torch.cuda.synchronize()
        codec.check_status()
        wire = codec.wire_bytes.cpu().numpy()
        chg = codec.changed_blocks.cpu().numpy()
        ms = codec.msg_send.cpu().numpy()
        for i, (u, hc) in enumerate(zip(units, hcs)):
            m, wb, pb, cb = ora.encode_hashed(unit_w(w, u), hc, dtype, block)
            assert int(wire[i]) == wb and int(chg[i]) == cb, f"t={t} unit {i}: length / changed blocks"
            mo = int(u["msg_off"])
            assert np.array_equal(ms[mo : mo + wb], m), f"t={t} unit {i}: message differs"
        compare_hash_cache(f"t={t}")
        out = codec.weights_out.cpu().numpy().view(WDT[dtype])
        for u in units:
            lo, n = int(u["weights_off"]) // VB[dtype], int(u["n_values"])
            assert np.array_equal(out[lo : lo + n], w[lo : lo + n]), f"t={t}: reconstruction differs"
        codec.canaries.check(f"t={t}")
        assert sender_scratch_is_clean(codec), f"t={t}: scratch not handed back all zero"
        changed_total.append(int(chg.sum()))
    return changed_total


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("block", [16, 32, 64, 128, 256, 512, 1024, 2048, 4096])
def test_hashed_ragged_units_every_block_size(rt, dtype, block):
    n = rt[1].LayerCodec.from_tensors(RAGGED, 1, NAME[dtype], block, DEV).weights_bytes // VB[dtype]
    rng = np.random.default_rng(300 * dtype + block)
    hi = 1 << (32 if dtype == 1 else 16)
    w0 = rng.integers(0, hi, n, dtype=np.uint64).astype(WDT[dtype])
    w1 = w0.copy()
    flip = rng.random(n) < 0.01
    w1[flip] = rng.integers(0, hi, int(flip.sum()), dtype=np.uint64).astype(WDT[dtype])
    w3 = rng.integers(0, hi, n, dtype=np.uint64).astype(WDT[dtype])
    chg = _run(rt, RAGGED, 1, dtype, block, [w0, w1, w1, w3])
    assert chg[1] == 0  # the repeated iterate changes nothing


@pytest.mark.parametrize("dtype,block", [(0, 512), (1, 512), (0, 64), (1, 16), (2, 512), (2, 32)])
def test_hashed_reduced_moe_layer_and_zero_start(rt, dtype, block):
    sizes = [r * c for r, c in wl.olmoe_layer_shapes(2)] + [70_001, 17, 0]
    n = rt[1].LayerCodec.from_tensors(sizes, 4, NAME[dtype], block, DEV).weights_bytes // VB[dtype]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 640 + block, 2, "clustered", f=0.2)]
    chg = _run(rt, sizes, 4, dtype, block, traj)
    assert chg[-1] > 0
    _run(rt, sizes, 4, dtype, block, traj[:2], from_zero=True)


@pytest.mark.parametrize("dtype,block", [(0, 128), (0, 32), (1, 4096), (1, 64), (2, 64), (2, 2048)])
def test_hashed_long_unit_of_many_tiles(rt, dtype, block):
    """One unit of ~3 M values = 367 tiles (its tiles are spread over the thread blocks and find their
    payload offsets by look-back) beside a shorter one; long and short rings of the kernel."""
    sizes = [3_000_000 + 123, 600_000]
    n = rt[1].LayerCodec.from_tensors(sizes, 1, NAME[dtype], block, DEV).weights_bytes // VB[dtype]
    gen = wl.make_generator(77 + block)
    w0 = wl.init_weights(n, NAME[dtype], gen)
    w1 = wl.inject_exponent_changes(w0, gen, 0.002)
    w2 = wl.inject_exponent_changes(w1, gen, 0.2)
    _run(rt, sizes, 1, dtype, block, [wl.as_bits(w) for w in (w0, w1, w2)])


def test_hashed_rejects_fine_blocks(rt):
    ciera, runtime = rt
    codec = runtime.LayerCodec.from_tensors([1000], 1, "bf16", 4, DEV)
    with pytest.raises(ciera.CieraError) as e:
        codec.init_hash_cache(None)
    assert e.value.status == ciera.ERR_UNSUPPORTED


@pytest.mark.parametrize("block", [16, 32, 64, 128, 256, 512, 1024, 4096])
def test_hashed_fp16_ragged_units(rt, block):
    """fp16 through the hashed sender (5-bit exponents and 11-bit sign-plus-mantissa packed on the wire, the
    hash taken over the exponents one byte each, as the caches hold them): ragged units, random bit patterns."""
    n = rt[1].LayerCodec.from_tensors(RAGGED, 1, "fp16", block, DEV).weights_bytes // 2
    rng = np.random.default_rng(900 + block)
    w0 = rng.integers(0, 1 << 16, n, dtype=np.uint64).astype(np.uint16)
    w1 = w0.copy()
    flip = rng.random(n) < 0.01
    w1[flip] = rng.integers(0, 1 << 16, int(flip.sum()), dtype=np.uint64).astype(np.uint16)
    w3 = rng.integers(0, 1 << 16, n, dtype=np.uint64).astype(np.uint16)
    chg = _run(rt, RAGGED, 1, 2, block, [w0, w1, w1, w3])
    assert chg[1] == 0
