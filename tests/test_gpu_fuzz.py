"""Randomised differential test of the whole CUDA path against the oracles: random unit tables
(empty, tiny, ragged and multi-tile units), every block size, both precisions, random update models
and start states; with blocks of 16 values and more also the hashed sender and the entropy stage.
Seeds are fixed: the cases are the same on every run.  CIERA_FUZZ_CASES=<n> in the environment runs n
cases of each kind instead of the default 60 / 20 (a longer soak)."""
import os

import numpy as np
import pytest
import torch

from harness import OracleTable, compare_caches, compare_recon, compare_step, guard, to_dev_bytes
from oracle import ciera_oracle as ora
from oracle import rans_oracle as rans
from paper_2609_04609_b200 import workloads as wl

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
WDT = {0: np.uint16, 1: np.uint32, 2: np.uint16}
VB = {0: 2, 1: 4, 2: 2}
NAME = {0: "bf16", 1: "fp32", 2: "fp16"}
BLOCKS = [1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096]
N_FULL = int(os.environ.get("CIERA_FUZZ_CASES", "60"))
N_HASHED = int(os.environ.get("CIERA_FUZZ_CASES", "20"))


@pytest.fixture(scope="module")
def rt():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2609_04609_b200 import ciera, runtime

    return ciera, runtime


def _random_case(seed):
    rng = np.random.default_rng(seed)
    sizes = []
    for _ in range(int(rng.integers(1, 9))):
        kind = rng.integers(0, 6)
        sizes.append(int([0, rng.integers(1, 40), rng.integers(40, 9000), rng.integers(8000, 8400) ,
                          rng.integers(9000, 80_000), rng.integers(80_000, 400_000)][kind]))
    shards = int(rng.choice([1, 1, 2, 3, 8]))
    dtype = int(rng.integers(0, 3))
    block = int(rng.choice(BLOCKS))
    return rng, sizes, shards, dtype, block


def _trajectory(rng, n, dtype):
    hi = 1 << (32 if dtype == 1 else 16)
    style = int(rng.integers(0, 3))
    if style == 0:  # arbitrary bit patterns, a few values replaced per step
        w0 = rng.integers(0, hi, n, dtype=np.uint64).astype(WDT[dtype])
        out = [w0]
        for _ in range(2):
            w = out[-1].copy()
            flip = rng.random(n) < float(rng.choice([0.0005, 0.01, 0.3]))
            w[flip] = rng.integers(0, hi, int(flip.sum()), dtype=np.uint64).astype(WDT[dtype])
            out.append(w)
        return out
    model = ["adam", "clustered"][style - 1]
    kw = {"f": float(rng.choice([0.05, 0.5]))} if model == "clustered" else {}
    return [wl.as_bits(w) for w in wl.trajectory(n, NAME[dtype], int(rng.integers(1, 1 << 30)), 2, model, **kw)]


@pytest.mark.parametrize("seed", range(N_FULL))
def test_random_tables_full_step(rt, seed):
    ciera, runtime = rt
    rng, sizes, shards, dtype, block = _random_case(1000 + seed)
    codec = guard(runtime.LayerCodec.from_tensors(sizes, shards, NAME[dtype], block, DEV, slack=256))
    table = OracleTable(codec.units, dtype, block, codec.cache_bytes, codec.msg_bytes)
    n = codec.weights_bytes // VB[dtype]
    traj = _trajectory(rng, max(n, 1), dtype)
    from_zero = bool(rng.integers(0, 2))
    codec.init_caches(None if from_zero else to_dev_bytes(traj[0], DEV))
    table.init_caches(None if from_zero else traj[0])
    label = f"seed {seed} sizes {sizes} shards {shards} {NAME[dtype]} B={block}"
    for t, w in enumerate(traj[1:], 1):
        codec.step(to_dev_bytes(w, DEV))
        torch.cuda.synchronize()
        codec.check_status()
        exp = table.step(w)
        compare_step(codec, exp, w, f"{label} t={t}")
        compare_caches(codec, table, f"{label} t={t}")
        compare_recon(codec, exp, w, dtype, f"{label} t={t}")


@pytest.mark.parametrize("seed", range(N_HASHED))
def test_random_tables_hashed_sender_and_entropy_stage(rt, seed):
    ciera, runtime = rt
    rng, sizes, shards, dtype, block = _random_case(5000 + seed)
    block = max(block, 16)
    codec = guard(runtime.LayerCodec.from_tensors(sizes, shards, NAME[dtype], block, DEV, slack=256))
    units = codec.units
    n = codec.weights_bytes // VB[dtype]
    traj = _trajectory(rng, max(n, 1), dtype)

    def unit_w(w, u):
        lo = int(u["weights_off"]) // VB[dtype]
        return w[lo : lo + int(u["n_values"])]

    from_zero = bool(rng.integers(0, 2))
    first = None if from_zero else traj[0]
    first_dev = None if from_zero else to_dev_bytes(traj[0], DEV)
    hcs = [ora.hash_cache_init(None if first is None else unit_w(first, u), int(u["n_values"]), dtype, block)
           for u in units]
    codec.init_hash_cache(first_dev)
    codec.init_caches(first_dev)
    label = f"seed {seed} sizes {sizes} shards {shards} {NAME[dtype]} B={block}"
    for t, w in enumerate(traj[1:], 1):
        codec.encode_hashed(to_dev_bytes(w, DEV))
        codec.entropy_encode()
        torch.cuda.synchronize()
        wire = codec.wire_bytes.cpu().numpy()
        ms = codec.msg_send.cpu().numpy()
        for i, (u, hc) in enumerate(zip(units, hcs)):
            nn, mo = int(u["n_values"]), int(u["msg_off"])
            raw, wb, pb, cb = ora.encode_hashed(unit_w(w, u), hc, dtype, block)
            want = rans.entropy_encode_message(raw, nn, dtype, block)
            assert int(wire[i]) == want.size, f"{label} t={t} unit {i}: length"
            assert np.array_equal(ms[mo : mo + want.size], want), f"{label} t={t} unit {i}: message"
        codec.transport()
        codec.entropy_decode()
        codec.decode()
        torch.cuda.synchronize()
        codec.check_status()
        out = codec.weights_out.cpu().numpy().view(WDT[dtype])
        for u in units:
            lo, nn = int(u["weights_off"]) // VB[dtype], int(u["n_values"])
            assert np.array_equal(out[lo : lo + nn], w[lo : lo + nn]), f"{label} t={t}: reconstruction"
        codec.canaries.check(f"{label} t={t}")
