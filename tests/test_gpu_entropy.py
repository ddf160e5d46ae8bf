"""GPU parity of the entropy stage (ciera_entropy_encode / ciera_entropy_decode) against the rANS
oracle: coded messages and lengths bit for bit, raw messages restored bit for bit, weights exact."""
import numpy as np
import pytest
import torch

from harness import guard, to_dev_bytes
from oracle import ciera_oracle as ora
from oracle import rans_oracle as rans
from paper_2609_04609_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
WDT = {0: np.uint16, 1: np.uint32, 2: np.uint16}
VB = {0: 2, 1: 4, 2: 2}
NAME = {0: "bf16", 1: "fp32", 2: "fp16"}
RAGGED = [0, 1, 5, 31, 33, 100, 511, 513, 4095, 4096, 4097, 8191, 8193, 20000, 3 * 8192 + 77, 70001, 140_000]


@pytest.fixture(scope="module")
def rt():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_04609_b200 import ciera, runtime

    return ciera, runtime


def _run(rt, sizes, n_shards, dtype, block, traj, from_zero):
    """Every step: encode, entropy-encode, transport, entropy-decode, decode; each stage against the oracle."""
    ciera, runtime = rt
    codec = guard(runtime.LayerCodec.from_tensors(sizes, n_shards, NAME[dtype], block, DEV, slack=256))
    units = codec.units

    def unit_w(w, u):
        lo = int(u["weights_off"]) // VB[dtype]
        return w[lo : lo + int(u["n_values"])]

    first = None if from_zero else traj[0]
    caches = [ora.cache_init(None if first is None else unit_w(first, u), int(u["n_values"]), dtype) for u in units]
    codec.init_caches(None if first is None else to_dev_bytes(first, DEV))
    coded_units = 0
    for t, w in enumerate(traj[1:], 1):
        codec.encode(to_dev_bytes(w, DEV))
        codec.entropy_encode()
        torch.cuda.synchronize()
        wire = codec.wire_bytes.cpu().numpy().copy()
        ms = codec.msg_send.cpu().numpy()
        raws = []
        for i, u in enumerate(units):
            n, mo = int(u["n_values"]), int(u["msg_off"])
            raw, wb, pb, cb = ora.encode(unit_w(w, u), caches[i], dtype, block)
            want = rans.entropy_encode_message(raw, n, dtype, block)
            assert int(wire[i]) == want.size, f"t={t} unit {i}: coded length {int(wire[i])} != {want.size} (raw {wb})"
            assert np.array_equal(ms[mo : mo + want.size], want), f"t={t} unit {i}: coded message differs"
            coded_units += want.size < raw.size
            raws.append(raw)
        codec.transport()
        codec.entropy_decode()
        torch.cuda.synchronize()
        codec.check_status()
        wire2 = codec.wire_bytes.cpu().numpy()
        mr = codec.msg_recv.cpu().numpy()
        for i, u in enumerate(units):
            mo = int(u["msg_off"])
            assert int(wire2[i]) == raws[i].size, f"t={t} unit {i}: restored length"
            assert np.array_equal(mr[mo : mo + raws[i].size], raws[i]), f"t={t} unit {i}: restored message differs"
        codec.decode()
        torch.cuda.synchronize()
        codec.check_status()
        out = codec.weights_out.cpu().numpy().view(WDT[dtype])
        for u in units:
            lo, n = int(u["weights_off"]) // VB[dtype], int(u["n_values"])
            assert np.array_equal(out[lo : lo + n], w[lo : lo + n]), f"t={t}: reconstruction differs"
        codec.canaries.check(f"t={t}")
    return coded_units


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("block", [1, 8, 64, 512, 4096])
def test_entropy_stage_ragged_units(rt, dtype, block):
    """Gaussian-like weights from empty caches (large, compressible payloads), then small steps."""
    n = rt[1].LayerCodec.from_tensors(RAGGED, 1, NAME[dtype], block, DEV).weights_bytes // VB[dtype]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 40 + block, 2, "adam")]
    coded = _run(rt, RAGGED, 1, dtype, block, [traj[0]] + traj, from_zero=True)
    assert coded > 0


def test_entropy_stage_keeps_incompressible_payloads_raw(rt):
    """Random bit patterns: the exponent bytes are uniform, the coded form is longer, the raw form travels."""
    sizes = [70_001, 8192, 100]
    n = rt[1].LayerCodec.from_tensors(sizes, 1, "bf16", 64, DEV).weights_bytes // 2
    rng = np.random.default_rng(5)
    w0 = rng.integers(0, 1 << 16, n, dtype=np.uint64).astype(np.uint16)
    w1 = rng.integers(0, 1 << 16, n, dtype=np.uint64).astype(np.uint16)
    coded = _run(rt, sizes, 1, 0, 64, [w0, w1], from_zero=False)
    assert coded == 0


@pytest.mark.parametrize("dtype", [0, 1])
def test_entropy_stage_reduced_moe_layer(rt, dtype):
    sizes = [r * c for r, c in wl.olmoe_layer_shapes(2)]
    n = rt[1].LayerCodec.from_tensors(sizes, 4, NAME[dtype], 512, DEV).weights_bytes // VB[dtype]
    traj = [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], 4, 2, "clustered", f=0.3)]
    coded = _run(rt, sizes, 4, dtype, 512, traj, from_zero=False)
    assert coded > 0


@pytest.mark.parametrize("block", [1, 2, 4, 8, 16, 32, 64, 512, 4096])
def test_entropy_stage_fp16(rt, block):
    """fp16: the stage codes the five-bit exponents as symbols of their own (unpacked before, packed after the
    coder, 32 table entries); ragged units from empty caches (large payloads), a reduced MoE layer under the
    clustered update, and a unit long enough for the chain of launches."""
    n = rt[1].LayerCodec.from_tensors(RAGGED, 1, "fp16", block, DEV).weights_bytes // 2
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "fp16", 140 + block, 2, "adam")]
    assert _run(rt, RAGGED, 1, 2, block, [traj[0]] + traj, from_zero=True) > 0
    sizes = [r * c for r, c in wl.olmoe_layer_shapes(1)] + [700_001]
    n = rt[1].LayerCodec.from_tensors(sizes, 4, "fp16", block, DEV).weights_bytes // 2
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "fp16", 9 + block, 2, "clustered", f=0.3)]
    _run(rt, sizes, 4, 2, block, traj, from_zero=False)
    n = rt[1].LayerCodec.from_tensors([700_001, 3000], 1, "fp16", block, DEV).weights_bytes // 2
    w = wl.as_bits(next(iter(wl.trajectory(n, "fp16", 11 + block, 0, "adam"))))
    assert _run(rt, [700_001, 3000], 1, 2, block, [w, w], from_zero=True) > 0


def test_entropy_stage_unit_of_many_segments(rt):
    """A unit whose payload has more than 256 segments (more than one chunk of the size scan)."""
    sizes = [1_300_000 + 17, 5000]
    n = rt[1].LayerCodec.from_tensors(sizes, 1, "bf16", 256, DEV).weights_bytes // 2
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 8, 1, "adam")]
    coded = _run(rt, sizes, 1, 0, 256, [traj[0]] + traj, from_zero=True)
    assert coded > 0


def test_entropy_stage_long_and_short_units_mixed(rt):
    """Units above and below 262 144 values in one table (the long ones are spread over several
    thread blocks), a long unit with incompressible exponents among them."""
    sizes = [300_000, 1000, 700_001, 262_144, 262_145, 50_000]
    codec = rt[1].LayerCodec.from_tensors(sizes, 1, "bf16", 128, DEV)
    n = codec.weights_bytes // 2
    traj = [wl.as_bits(w) for w in wl.trajectory(n, "bf16", 21, 2, "adam")]
    lo = int(codec.units[0]["weights_off"]) // 2
    rng = np.random.default_rng(2)
    for w in traj:  # unit 0: arbitrary bit patterns, new ones every step
        w[lo : lo + 300_000] = rng.integers(0, 1 << 16, 300_000, dtype=np.uint64).astype(np.uint16)
    coded = _run(rt, sizes, 1, 0, 128, [traj[0]] + traj, from_zero=True)
    assert coded >= 4


@pytest.mark.parametrize("dtype", [0, 2])
@pytest.mark.parametrize("n_values", [70_001, 600_001])
def test_entropy_decode_flags_a_damaged_section(rt, n_values, dtype):
    ciera, runtime = rt
    sizes = [n_values]
    codec = runtime.LayerCodec.from_tensors(sizes, 1, NAME[dtype], 512, DEV)
    n = codec.weights_bytes // 2
    w = wl.as_bits(next(iter(wl.trajectory(n, NAME[dtype], 3, 0, "adam"))))
    codec.init_caches(None)
    codec.encode(to_dev_bytes(w, DEV))
    codec.entropy_encode()
    codec.transport()
    torch.cuda.synchronize()
    raw_len = ora.message_capacity(n_values, dtype, 512)  # from empty caches every block is changed
    assert int(codec.wire_bytes[0].item()) < raw_len  # the coded form travelled
    off = int(codec.units[0]["msg_off"]) + ora.payload_offset(n_values, dtype, 512)
    nseg = -(-n_values // 4096)
    table = 64 if dtype == 2 else 512
    before = codec.msg_recv.clone()
    codec.msg_recv[off + table + 4 * nseg + 200] ^= 0x5A  # inside the first segment's words
    damaged = codec.msg_recv.clone()
    codec.entropy_decode()
    torch.cuda.synchronize()
    assert int(codec.status.item()) == ciera.ERR_CORRUPT
    assert torch.equal(codec.msg_recv, damaged) and not torch.equal(damaged, before)  # left as received
