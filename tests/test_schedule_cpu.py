"""The static tile schedule of the single persistent launch, checked on the CPU: coverage, producer
tickets before consumer tickets, no deadlock for any worker count, counters end at thresholds."""
import numpy as np
import pytest

from paper_2605_23764_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


def _seg(is_bwd, d, F):
    if not is_bwd:
        return [(F + 127) // 128, (d + 255) // 256, 0, 0]
    return [(F + 255) // 256, (d + 127) // 128, (d + 255) // 256, (2 * F + 127) // 128]


@pytest.mark.parametrize("pair", [0, 1, 2])
@pytest.mark.parametrize("is_bwd", [0, 1])
@pytest.mark.parametrize("workers", [(1, 1), (3, 2), (148, 592)])
@pytest.mark.parametrize("lag", [0, 1, 8])
def test_schedule_is_sound(is_bwd, workers, lag, pair):
    rng = np.random.default_rng(lag * 7 + is_bwd)
    cases = [
        rng.integers(0, 700, 24),                      # mixed sizes
        np.array([0, 0, 5, 0, 1300, 0, 129, 0]),       # empty experts, one large
        np.array([3000]),                              # a single expert
        np.zeros(6, int),                              # nothing routed at all
        np.full(64, 128),                              # exactly one M-block each
    ]
    for counts in cases:
        T = max(1, int(counts.sum()) // 2)
        rc, stats = binding.moe_debug_simulate_schedule(counts, T, 2, is_bwd, _seg(is_bwd, 520, 264), lag, *workers,
                                                        pair=pair)
        assert rc == 0, (counts.tolist(), rc)
        mblocks = (counts + 127) // 128
        M = int(((mblocks + 1) // 2).sum()) if pair else int(mblocks.sum())
        seg = _seg(is_bwd, 520, 264)
        want = M * (seg[0] + (seg[2] if is_bwd else seg[1]))
        if is_bwd:
            want += int((counts > 0).sum()) * (seg[1] + seg[3])
        assert stats[0] == want


def test_balanced_units_cover_every_mblock_once():
    """Token-column tiles: the units of an expert (one or two M-blocks each) partition its M-blocks, and a
    lone M-block never comes last when there are three or more."""
    for n in list(range(0, 1200, 7)) + [128, 256, 257, 384, 385, 512, 640, 641]:
        counts = np.array([n, 1, 300])
        rc, stats = binding.moe_debug_simulate_schedule(counts, 64, 2, 0, [3, 2, 0, 0], 1, 5, 7, pair=2)
        assert rc == 0, (n, rc)


def test_training_config_schedule():
    """Config-4-like counts (256 experts, ~256 rows each) with the launch's real worker counts."""
    rng = np.random.default_rng(4)
    counts = rng.binomial(65536, 1 / 256, 256)
    for is_bwd in (0, 1):
        for pair in (0, 1, 2):
            rc, stats = binding.moe_debug_simulate_schedule(counts, 8192, 8, is_bwd, _seg(is_bwd, 7168, 2048), 8, 148,
                                                            592, pair=pair)
            assert rc == 0
