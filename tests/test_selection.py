"""Shard selection under a cache budget (Section 3.2): pins of the oracle, and the library's
host function against the oracle.  No GPU."""
import itertools
import os

import numpy as np
import pytest

from oracle import selection as sel

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "selection_worked_example.txt")


def _cases(path):
    cases, cur = [], None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line == "[case]":
            cur = {}
            cases.append(cur)
            continue
        k, *v = line.split()
        cur[k] = v
    return cases


def test_hand_worked_selection():
    for c in _cases(GOLDEN):
        gains = [float(x) * 1e-6 for x in c["gains"]]
        fp = [int(x) for x in c["footprints"]]
        ranking, selected, used = sel.select_shards(gains, fp, int(c["budget"][0]))
        npos = len(c["ranking"])
        assert ranking[:npos] == [int(x) for x in c["ranking"]]
        assert sorted(i for i, s in enumerate(selected) if s) == sorted(int(x) for x in c["selected"])
        assert used == int(c["used"][0])


def test_footprint_formula():
    # M_i = (W - 1) S_e^i with one exponent byte per value
    assert sel.cache_footprint(131072, 16) == 15 * 131072
    assert sel.cache_footprint(131072, 16, with_sender_cache=True) == 16 * 131072
    assert sel.cache_footprint(0, 8) == 0


def test_budget_extremes_and_sign_rule():
    rng = np.random.default_rng(3)
    for _ in range(50):
        n = int(rng.integers(1, 12))
        g = rng.normal(0, 1, n).tolist()
        m = rng.integers(1, 1000, n).tolist()
        _, s_all, used = sel.select_shards(g, m, sum(m))
        assert s_all == [x > 0 for x in g] and used == sum(mi for mi, x in zip(m, g) if x > 0)
        _, s_none, used0 = sel.select_shards(g, m, 0)
        assert not any(s_none) and used0 == 0


def _best_subset(g, m, budget):
    best = 0.0
    for r in range(len(g) + 1):
        for sub in itertools.combinations(range(len(g)), r):
            if sum(m[i] for i in sub) <= budget:
                best = max(best, sum(g[i] for i in sub))
    return best


def test_against_brute_force_on_tiny_inputs():
    """Equal footprints: the greedy prefix is the best subset.  Any footprints: it is a prefix of
    the density ranking, respects the budget, and (the fractional-knapsack bound) together with
    the first shard that did not fit it is worth at least the best subset."""
    rng = np.random.default_rng(5)
    for trial in range(200):
        n = int(rng.integers(1, 9))
        g = np.round(rng.normal(0.5, 1.0, n), 3).tolist()
        equal = trial % 2 == 0
        m = [100] * n if equal else rng.integers(1, 400, n).tolist()
        budget = int(rng.integers(0, sum(m) + 1))
        ranking, selected, used = sel.select_shards(g, m, budget)
        chosen = [i for i in ranking if selected[i]]
        assert used == sum(m[i] for i in chosen) <= budget
        pos = [i for i in ranking if g[i] > 0]
        assert ranking[: len(pos)] == pos and chosen == pos[: len(chosen)]  # a prefix of the ranking
        dens = [g[i] / m[i] for i in pos]
        assert all(dens[k] >= dens[k + 1] for k in range(len(dens) - 1))
        got = sum(g[i] for i in chosen)
        best = _best_subset(g, m, budget)
        if equal:
            assert abs(got - best) < 1e-9
        else:
            nxt = g[pos[len(chosen)]] if len(chosen) < len(pos) else 0.0
            assert got + nxt >= best - 1e-9


# ------------------------------------------------------------------ library vs oracle (host function)


@pytest.fixture(scope="module")
def ciera():
    from paper_2609_04609_b200 import ciera as c

    return c


def test_library_selection_matches_oracle(ciera, oracle):
    rng = np.random.default_rng(17)
    for trial in range(60):
        n = int(rng.integers(1, 40))
        world = int(rng.integers(2, 65))
        shards = []
        for _ in range(n):
            shards.append(dict(
                n_values=int(rng.choice([0, 17, 4096, 131072, 1 << 20, 5_000_001])),
                dtype=int(rng.integers(0, 2)), block=int(2 ** rng.integers(0, 13)), q=float(rng.random()),
                world_size=world, alpha=float(rng.random() * 2e-5), beta=float(10 ** rng.uniform(9, 11.5)),
                t_hash=float(rng.random() * 1e-6), t_cmp=float(rng.random() * 2e-5),
                t_decmp=float(rng.random() * 2e-5), overlapped=bool(rng.integers(0, 2))))
        with_sender = bool(trial % 2)
        gains = [oracle.gain(s["n_values"], s["dtype"], s["block"], s["q"], s["world_size"], s["alpha"], s["beta"],
                             None, s["t_hash"], s["t_cmp"], s["t_decmp"], s["overlapped"]) for s in shards]
        fps = [sel.cache_footprint(s["n_values"], world, with_sender) for s in shards]
        budget = int(rng.integers(0, sum(fps) + 2))
        ranking, selected, used = sel.select_shards(gains, fps, budget)
        got = ciera.select_shards(shards, budget, with_sender)
        assert got["gains"] == pytest.approx(gains, rel=1e-12, abs=1e-18)
        assert got["footprints"] == fps
        assert got["ranking"] == ranking and got["selected"] == selected and got["used"] == used


def test_library_selection_rejects_bad_input(ciera):
    with pytest.raises(ciera.CieraError):
        ciera.select_shards([dict(n_values=10, dtype=5, block=64, q=0.1, world_size=4)], 100)
    with pytest.raises(ciera.CieraError):
        ciera.select_shards([dict(n_values=10, dtype=0, block=64, q=1.5, world_size=4)], 100)
    assert ciera.select_shards([], 100)["used"] == 0
