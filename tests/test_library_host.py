"""CPU checks of the C-ABI library: it loads, exports every symbol the header declares, and its
host-side logic (size rules, plan validation and tile table, gain rule) is right.  No kernel is
launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2609_04609_b200 import build as libbuild
from paper_2609_04609_b200.workloads import UNIT_DTYPE, layout_units

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ciera():
    libbuild.build_library()
    from paper_2609_04609_b200 import ciera as c

    return c


def test_library_exports_every_declared_symbol(ciera):
    header = open(os.path.join(ROOT, "include", "ciera.h")).read()
    declared = set(re.findall(r"CIERA_API[^;(]*?\b(ciera_\w+)\s*\(", header))
    assert len(declared) >= 20
    lib = ctypes.CDLL(libbuild.LIB)
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in ciera.h but not exported"
    assert declared == set(ciera.EXPORTS), "binding and header disagree on the entry points"


@pytest.mark.parametrize("dtype", [0, 1])
def test_size_rules_agree_with_the_oracle(ciera, oracle, dtype):
    for n in [0, 1, 15, 16, 17, 127, 128, 129, 4095, 4096, 4097, 131072, 131073, 16777216 + 5]:
        for block in [1, 2, 16, 64, 512, 4096]:
            assert ciera.sm_offset(n, block) == oracle.sm_offset(n, block)
            assert ciera.payload_offset(n, dtype, block) == oracle.payload_offset(n, dtype, block)
            assert ciera.message_capacity(n, dtype, block) == oracle.message_capacity(n, dtype, block)
            for pay in (0, n // 3, n):
                assert ciera.message_bytes(n, dtype, block, pay) == oracle.paper_bytes(n, dtype, block, pay)


def test_paper_size_definitions_on_the_olmoe_unit(ciera):
    # N = 131072 bf16 values, B = 512: S = 262144, S_e = 131072, S_{s+m} = 131072, S_b = 256, S_bm = 32
    assert ciera.message_bytes(131072, 0, 512, 0) == 131072 + 32
    assert ciera.message_bytes(131072, 1, 512, 5 * 512) == 3 * 131072 + 32 + 2560
    assert ciera.sm_offset(131072, 512) == 32 and ciera.payload_offset(131072, 0, 512) == 32 + 131072


def _units(rows):
    return np.array(rows, dtype=UNIT_DTYPE)


def test_plan_validation(ciera):
    cap = ciera.message_capacity(1000, 0, 512)
    good = _units([(1000, 0, 0, 0, cap)])
    assert ciera.Plan(good, 0, 512).n_tiles == 1
    for block in (1, 2, 4, 8, 16, 4096):
        assert ciera.Plan(_units([(1000, 0, 0, 0, ciera.message_capacity(1000, 0, block))]), 0, block).n_tiles == 1
    for block in (0, 3, 100, 8192):
        with pytest.raises(ciera.CieraError) as e:
            ciera.Plan(good, 0, block)
        assert e.value.status in (ciera.ERR_INVALID_ARG, ciera.ERR_UNSUPPORTED)
    with pytest.raises(ciera.CieraError) as e:
        ciera.Plan(_units([(1000, 8, 0, 0, cap)]), 0, 512)
    assert e.value.status == ciera.ERR_MISALIGNED
    with pytest.raises(ciera.CieraError) as e:
        ciera.Plan(_units([(1000, 0, 0, 0, cap - 1)]), 0, 512)
    assert e.value.status == ciera.ERR_CAPACITY
    with pytest.raises(ciera.CieraError) as e:  # more blocks than a 32-bit count holds
        ciera.Plan(_units([(1 << 33, 0, 0, 0, ciera.message_capacity(1 << 33, 0, 1))]), 0, 1)
    assert e.value.status == ciera.ERR_UNSUPPORTED
    with pytest.raises(ciera.CieraError) as e:
        ciera.Plan(good, 7, 512)
    assert e.value.status == ciera.ERR_INVALID_ARG
    # an unbound plan refuses device work
    p = ciera.Plan(good, 0, 512)
    assert ciera._lib.ciera_encode(p.handle, 16, 16, 16, 16, 16, 16, None, None) == ciera.ERR_NOT_BOUND


def test_plan_tile_table(ciera):
    """Every unit is cut into tiles of 8192 values; the table lists short units (<= 32 tiles) first, longest
    first and otherwise in table order, then the longer units; empty units have no tiles."""
    T = 8192
    sizes = [0, 5, T, T + 1, 3 * T + 17, 0, 40000, 40 * T + 3, 33 * T, 13 * T - 5]
    units, wb, cb, mb = layout_units(sizes, 1, 4, lambda n: ciera.message_capacity(n, 1, 64))
    p = ciera.Plan(units, 1, 64)
    ntiles = [-(-n // T) for n in sizes]
    want_tiles = sum(ntiles)
    assert (p.n_units, p.n_tiles, p.tile_values, p.total_values) == (len(sizes), want_tiles, T, sum(sizes))
    assert p.workspace_bytes >= 8 * want_tiles and p.device_bytes >= 48 * want_tiles
    img = p.host_image()[: 48 * want_tiles].view(np.dtype([("w", "<u8"), ("c", "<u8"), ("m", "<u8"), ("n", "<u8"),
                                                          ("unit", "<u4"), ("j", "<u4"), ("first", "<u4"), ("nt", "<u4")]))
    short = sorted([u for u in range(len(sizes)) if 1 <= ntiles[u] <= 32], key=lambda u: -ntiles[u])
    long_ = [u for u in range(len(sizes)) if ntiles[u] > 32]
    k = 0
    for ui in short + long_:
        u = units[ui]
        for j in range(ntiles[ui]):
            t = img[k]
            assert (t["unit"], t["j"], t["first"], t["nt"], t["n"]) == (ui, j, k - j, ntiles[ui], u["n_values"])
            assert t["w"] == u["weights_off"] + j * T * 4 and t["c"] == u["cache_off"] + j * T
            assert t["m"] == u["msg_off"]
            k += 1
    assert k == want_tiles
    # HashCache: 16 bytes per block, units in table order; the image ends with the index of every tile's first
    # block (8 bytes per tile, in tile-table order, padded to 16 bytes), the runs of tiles in which the short units
    # are handed out (pairs of 32-bit tile numbers) and 16 spare bytes
    nblocks = [-(-n // 64) for n in sizes]
    assert p.hash_cache_bytes == 16 * sum(nblocks)
    base = np.concatenate([[0], np.cumsum(nblocks)])
    assert [ciera.unit_hash_offset(p, u) for u in range(len(sizes))] == [16 * int(b) for b in base[:-1]]
    assert p.hashed_workspace_bytes == p.workspace_bytes
    def expected_runs():
        """Every short unit's first run (all but its last one to four tiles), then every unit's last run."""
        heads, tails, k0 = [], [], 0
        for ui in short:
            nt = ntiles[ui]
            head = nt if nt <= 4 else (nt - 1) // 4 * 4
            heads.append((k0, k0 + head))
            if head < nt:
                tails.append((k0 + head, k0 + nt))
            k0 += nt
        return heads + tails

    runs = expected_runs()
    assert any(hi - lo > 4 for lo, hi in runs) and len(runs) > len(short)  # the table has units of more than four tiles
    image = p.host_image()
    got_runs = image[-(8 * len(runs) + 16):-16].view("<u4").reshape(-1, 2)
    assert [tuple(int(x) for x in r) for r in got_runs] == runs
    units512, _, _, _ = layout_units(sizes, 1, 4, lambda n: ciera.message_capacity(n, 1, 512))
    got512 = ciera.Plan(units512, 1, 512).host_image()[-(8 * len(runs) + 16):-16].view("<u4").reshape(-1, 2)
    assert [tuple(int(x) for x in r) for r in got512] == runs  # the same for every block size
    thash_bytes = (8 * want_tiles + 15) // 16 * 16
    tail = image[-(8 * len(runs) + 16 + thash_bytes):-(8 * len(runs) + 16)][: 8 * want_tiles].view("<u8")
    assert [int(x) for x in tail] == [int(base[t["unit"]]) + int(t["j"]) * (T // 64) for t in img]
    # an empty table is legal
    e = ciera.Plan(np.zeros(0, UNIT_DTYPE), 0, 512)
    assert (e.n_units, e.n_tiles) == (0, 0)


def test_should_compress_matches_hand_computed_cases_and_the_oracle(ciera, oracle):
    path = os.path.join(ROOT, "tests", "golden", "gain_cases.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, dt, n, block, q, world, alpha, beta, th, tc, td, ov, table, want = line.split()
        tbl = None if table == "none" else [tuple(float(x) for x in p.split(":")) for p in table.split(",")]
        g, dec = ciera.should_compress(int(n), 0 if dt == "bf16" else 1, int(block), float(q), int(world),
                                       float(alpha), float(beta), tbl, float(th), float(tc), float(td), bool(int(ov)))
        assert g == pytest.approx(float(want), rel=1e-9), name
        assert dec == (float(want) > 0)
    rng = np.random.default_rng(0)
    for _ in range(200):
        n = int(rng.integers(1, 1 << 24))
        dt = int(rng.integers(0, 2))
        block = int(2 ** rng.integers(0, 13))
        q = float(rng.random())
        kw = dict(world=int(rng.integers(2, 129)), alpha=float(rng.random() * 1e-4), beta=float(10 ** rng.uniform(9, 12)),
                  t_hash=float(rng.random() * 1e-5), t_cmp=float(rng.random() * 1e-5), t_decmp=float(rng.random() * 1e-5),
                  overlapped=bool(rng.integers(0, 2)))
        tbl = None
        if rng.random() < 0.5:
            xs = np.sort(rng.uniform(0, 4 * n, 4))
            tbl = [(float(x), float(1e-5 + x * 1e-10 * (1 + i))) for i, x in enumerate(xs)]
        g, dec = ciera.should_compress(n, dt, block, q, kw["world"], kw["alpha"], kw["beta"], tbl, kw["t_hash"],
                                       kw["t_cmp"], kw["t_decmp"], kw["overlapped"])
        want = oracle.gain(n, dt, block, q, kw["world"], kw["alpha"], kw["beta"], tbl, kw["t_hash"], kw["t_cmp"],
                           kw["t_decmp"], kw["overlapped"])
        assert g == pytest.approx(want, rel=1e-12, abs=1e-18)
        assert dec == (g > 0)
    with pytest.raises(ciera.CieraError):
        ciera.should_compress(100, 0, 512, 1.5)
    with pytest.raises(ciera.CieraError):
        ciera.should_compress(100, 0, 512, 0.5, beta=0.0)


def test_selection_behaviour_described_by_the_paper(ciera):
    """Low block change rate pays on a slow link; on a fast intra-node link with a real
    decompression cost nothing is selected (the paper's 4-GPU Llama-4-Scout case)."""
    n = 131072
    slow = dict(world_size=16, alpha=1e-5, beta=8e9, t_decmp=2e-6, overlapped=True)
    assert ciera.should_compress(n, 0, 512, 0.22, **slow)[1] is True
    assert ciera.should_compress(n, 0, 512, 1.0, **slow)[1] is False
    fast = dict(world_size=4, alpha=0.0, beta=300e9, t_decmp=2e-6, overlapped=True)
    assert ciera.should_compress(n, 0, 512, 0.9, **fast)[1] is False
