"""Properties of the two device-made work plans of gsd_verify_attn, checked on their plain-Python
model (tests/plan_model.py); the GPU tests compare the tables the planning kernels write with
this model entry by entry."""
import numpy as np
import pytest

from plan_model import balanced_table, per_sequence_table, tiles_of


def random_batch(rng):
    B = int(rng.integers(1, 40))
    Lmax = int(rng.choice([1, 100, 128, 1000, 5000, 40000]))
    lens = rng.integers(-3, Lmax + 5, size=B)          # out-of-range lengths are clamped
    if rng.uniform() < 0.3:
        lens[:] = Lmax
    return lens, Lmax, int(rng.choice([1, 2, 8, 40])), int(rng.integers(1, 5))


@pytest.mark.parametrize("seed", range(5))
def test_balanced_plan_covers_every_tile_once_in_equal_shares(seed):
    rng = np.random.default_rng(seed)
    for _ in range(40):
        lens, Lmax, per_seq, nd = random_batch(rng)
        groups = int(rng.choice([1, 7, 18, 37, 148]))
        t = balanced_table(lens, Lmax, per_seq, nd, groups)
        T = tiles_of(lens, Lmax, nd)
        assert t["total"] == per_seq * sum(T)
        covered = set()
        for g, (first, n) in enumerate(t["runs"]):
            tiles = 0
            partial = 0
            for pair, t0, t1, slot in t["units"][first:first + n]:
                assert 0 <= t0 < t1 <= T[pair // per_seq]
                for k in range(t0, t1):
                    assert (pair, k) not in covered
                    covered.add((pair, k))
                tiles += t1 - t0
                partial += slot >= 0
            assert tiles <= t["share"] and partial <= 2            # a group cuts at most its first and its last pair
            if g + 1 < groups and (g + 1) * t["share"] <= t["total"]:
                assert tiles == t["share"]                          # every share but the last is full
        assert len(covered) == t["total"]
        assert t["slots"] <= 2 * groups
        # the pieces of a cut pair have consecutive slots, in tile order
        for pair, s0, n in t["merge"]:
            pieces = sorted((t0, slot) for p, t0, _, slot in t["units"] if p == pair)
            assert n >= 2 and [s for _, s in pieces] == list(range(s0, s0 + n))


@pytest.mark.parametrize("seed", range(5))
def test_per_sequence_plan_split_counts_and_slot_bound(seed):
    rng = np.random.default_rng(100 + seed)
    for _ in range(200):
        lens, Lmax, per_seq, nd = random_batch(rng)
        wanted = int(rng.choice([2, 16, 296]))
        t = per_sequence_table(lens, Lmax, per_seq, nd, wanted)
        T = tiles_of(lens, Lmax, nd)
        for n, tt in zip(t["nsplit"], T):
            assert 1 <= n <= 32
            assert abs(n - tt / t["target"]) <= 0.5 + 1e-9 or n in (1, 32)      # the rounded ratio, clamped
        assert t["unit_off"][-1] == per_seq * sum(t["nsplit"])
        # what the workspace is sized for: 4/3 of the units aimed at (unless the clamp at 32 binds)
        if max(t["nsplit"]) < 32:
            assert t["slot_off"][-1] <= (4 * wanted + 2) // 3 + 1


def test_uniform_batch_gets_the_same_cut_everywhere():
    t = per_sequence_table([2048] * 4, 2048, 40, 1, 296)
    assert len(set(t["nsplit"])) == 1
    b = balanced_table([4096] * 8, 4096, 8, 2, 8)           # 8 groups, 64 pairs of 34 tiles: whole pairs only
    assert b["slots"] == 0 and all(s == -1 for _, _, _, s in b["units"])
