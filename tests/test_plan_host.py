"""The decode kernels' work decomposition, exercised on the CPU through the functions the kernels run
(pd_plan_ranges, pd_plan_walk): ranges must tile the unit list exactly, respect the caps, and a walk must
visit (sequence, KV head, page) triples in nesting order, skipping empty sequences."""
import numpy as np
import pytest

import paper_2609_35158_b200 as pd


def check_tiling(starts, lens, total):
    assert len(starts) == len(lens)
    if total == 0:
        assert int(lens.sum()) == 0
        return
    assert starts[0] == 0 and np.all(lens > 0)
    assert np.array_equal(starts[1:], (starts + lens)[:-1])  # contiguous, in order, no overlap
    assert int(starts[-1] + lens[-1]) == total


@pytest.mark.parametrize("seed", range(40))
def test_plan_tiles_the_units_exactly(seed):
    rng = np.random.default_rng(seed)
    total = int(rng.choice([0, 1, 5, 17, 300, 4096, 70000, 295112, 1571840, 6400000, int(rng.integers(1, 10 ** 7))]))
    workers = int(rng.choice([1, 8, 296, 1184, 2368]))
    split = int(rng.choice([0, 0, 0, 1, 2, 7, 64, 100000]))
    max_ranges = int(rng.choice([16 * workers, 4 * workers, workers, 37]))
    tail = int(rng.choice([16, 4, 48]))
    levels = int(rng.choice([6, 0, 2]))
    min_pages = int(rng.choice([4, 1]))
    starts, lens = pd.pd_plan_ranges(total, workers, split, max_ranges, min_pages, levels, tail)
    check_tiling(starts, lens, total)
    assert len(starts) <= max(max_ranges, 1)
    if split > 0 and total > 0:
        # one level of equal ranges, at least split pages each (more if the cap forces it), ragged last one
        assert np.all(lens[:-1] == lens[0]) and lens[0] >= min(split, total) and lens[-1] <= lens[0]
        if -(-total // split) <= max_ranges:
            assert lens[0] == min(split, max(total, 1)) or len(lens) == 1


def test_automatic_plan_has_shrinking_levels_and_a_short_tail():
    workers = 1184
    starts, lens = pd.pd_plan_ranges(295112, workers)  # configs[1]: 64 sequences x 8 heads, 2K-16K tokens
    check_tiling(starts, lens, 295112)
    assert len(lens) == 6901 and lens[0] == 125     # what the device reports for this workload
    level_sizes = [int(lens[i * workers]) for i in range(len(lens) // workers)]
    # every level hands each worker one range of half its remaining fair share, then a tail of 16-page ranges
    assert np.all(lens[:workers] == 125)
    assert all(a >= b for a, b in zip(level_sizes, level_sizes[1:]))
    assert lens[-2] == 16 and lens[-1] <= 16
    # few units: a single level; no range shorter than the minimum unless the total is
    s2, l2 = pd.pd_plan_ranges(40, workers)
    check_tiling(s2, l2, 40)
    assert np.all(l2[:-1] >= 4)


def test_walk_visits_triples_in_nesting_order():
    rng = np.random.default_rng(7)
    pages = np.array([3, 0, 5, 1, 0, 0, 7, 2], dtype=np.int32)  # pages per sequence, with empty ones
    cum = np.concatenate([[0], np.cumsum(pages)]).astype(np.int32)
    for Hkv in (1, 2, 8):
        want = [(b, h, p) for b in range(len(pages)) for h in range(Hkv) for p in range(pages[b])]
        total = len(want)
        seq, kvh, page = pd.pd_plan_walk(cum, Hkv, 0, total)
        assert list(zip(seq.tolist(), kvh.tolist(), page.tolist())) == want
        for _ in range(20):  # any start, any length
            a = int(rng.integers(0, total))
            n = int(rng.integers(0, total - a + 1))
            seq, kvh, page = pd.pd_plan_walk(cum, Hkv, a, n)
            assert list(zip(seq.tolist(), kvh.tolist(), page.tolist())) == want[a:a + n]
    with pytest.raises(pd.PdError):
        pd.pd_plan_walk(cum, 2, 0, 2 * int(pages.sum()) + 1)


def test_plan_rejects_bad_parameters():
    for args in ((-1, 8), (10, 0)):
        with pytest.raises(pd.PdError) as e:
            pd.pd_plan_ranges(*args)
        assert e.value.code == pd.PD_ERR_INVALID_ARG
    with pytest.raises(pd.PdError):
        pd.pd_plan_ranges(10, 8, halving_levels=99)


def test_equal_ranges_plan_of_the_fp8_entry_points():
    """halving_levels = 0 is the plan the FP8 kernels take while the fair share is at most 1024 pages: one range
    of ceil(total / workers) units per worker, at most `workers` ranges, tiling the unit list exactly. The figures
    are configs[3]'s (192 496 units, 148 SMs x 16 worker warps): 2 348 ranges of 82 units, the last one 42."""
    import paper_2609_35158_b200 as pd

    total, workers = 192496, 148 * 16
    starts, lens = pd.pd_plan_ranges(total, workers, 0, 16 * workers, 4, 0, 16)
    fair = -(-total // workers)
    assert fair == 82 and len(lens) == 2348 <= workers
    assert all(n == fair for n in lens[:-1]) and lens[-1] == total - fair * (len(lens) - 1) == 42
    assert starts[0] == 0 and all(starts[i + 1] == starts[i] + lens[i] for i in range(len(lens) - 1))
    assert starts[-1] + lens[-1] == total
