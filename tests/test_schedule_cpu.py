"""The static tile schedule of the single persistent launch, checked on the CPU: every M-block covered once
by every column tile of every phase, no deadlock for any number of CTA pairs and vector workers, counters
end at their thresholds."""
import numpy as np
import pytest

from paper_2605_23764_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


def _expected_items(counts, d, F, is_bwd):
    mblocks = (counts + 127) // 128
    units = (mblocks + 1) // 2
    # an expert merges its last two units when its M-block count is odd, at least 3, and the last block holds <= 64 rows
    merged = units - ((mblocks % 2 == 1) & (mblocks >= 3) & (counts - (mblocks - 1) * 128 <= 64))
    Ep = len(counts)
    if not is_bwd:
        return int(units.sum()) * ((F + 127) // 128) + int(merged.sum()) * ((d + 255) // 256)
    return (int(units.sum()) * ((F + 255) // 256) + Ep * ((d + 255) // 256) +
            int(merged.sum()) * ((d + 255) // 256) + Ep * ((2 * F + 255) // 256))


@pytest.mark.parametrize("is_bwd", [0, 1])
@pytest.mark.parametrize("workers", [(1, 1), (3, 2), (74, 592), (74, 2368)])
def test_schedule_is_sound(is_bwd, workers):
    rng = np.random.default_rng(7 + is_bwd)
    cases = [
        rng.integers(0, 700, 24),                      # mixed sizes
        np.array([0, 0, 5, 0, 1300, 0, 129, 0]),       # empty experts, one large
        np.array([3000]),                              # a single expert
        np.zeros(6, int),                              # nothing routed at all
        np.full(64, 128),                              # exactly one M-block each
        np.array([300, 257, 320, 577]),                # every expert ends in a merged item
        np.array([384, 321, 640, 385]),                # full last blocks / even counts: nothing merges
    ]
    d, F = 520, 272
    for counts in cases:
        T = max(1, int(counts.sum()) // 2)
        rc, stats = binding.moe_debug_simulate_schedule(counts, T, 2, 0, d, F, is_bwd, *workers)
        assert rc == 0, (counts.tolist(), rc)
        assert stats[0] == _expected_items(counts, d, F, is_bwd)


def test_balanced_units_cover_every_mblock_once():
    """Token-column tiles: the units of an expert (one or two M-blocks each) partition its M-blocks, and a
    lone M-block never comes last when there are three or more (the simulation checks the coverage)."""
    for n in list(range(0, 1200, 7)) + [128, 256, 257, 384, 385, 512, 640, 641]:
        counts = np.array([n, 1, 300])
        for is_bwd in (0, 1):
            rc, stats = binding.moe_debug_simulate_schedule(counts, 64, 2, 1, 384, 48, is_bwd, 5, 7)
            assert rc == 0, (n, rc)


def test_training_config_schedule():
    """Config-4-like counts (256 experts, ~256 rows each) with the launch's real worker counts."""
    rng = np.random.default_rng(4)
    counts = rng.binomial(65536, 1 / 256, 256)
    for is_bwd in (0, 1):
        rc, stats = binding.moe_debug_simulate_schedule(counts, 8192, 8, 0, 7168, 2048, is_bwd, 74, 1184)
        assert rc == 0


def test_skewed_config_schedule():
    """Config-3-like counts: Zipf popularity, empty experts, one expert with thousands of rows."""
    rng = np.random.default_rng(3)
    q = (np.arange(128) + 1.0) ** -1.2
    counts = rng.multinomial(131072, q / q.sum())
    counts[-4:] = 0
    rc, stats = binding.moe_debug_simulate_schedule(counts, 16384, 8, 0, 4096, 1536, 0, 74, 1184)
    assert rc == 0
