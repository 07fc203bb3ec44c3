"""The a-priori cost model behind the work-item order (host code of the library; runs without a GPU) and the
dealing rule of the executors, checked against what they are meant to achieve: with costs known in advance,
heaviest-first order dealt back and forth keeps every CTA's share close to the mean."""
import numpy as np

from paper_1901_06887_b200 import binding as mt


def cost(k_blocks, n_cols, rows):
    return mt.mt_debug_item_cost(k_blocks, n_cols, rows)


def test_cost_is_zero_for_empty_items_and_grows_with_every_dimension():
    assert cost(0, 128, 128) == 0.0 and cost(8, 0, 128) == 0.0 and cost(8, 128, 0) == 0.0
    assert cost(8, 128, 128) < cost(16, 128, 128) < cost(64, 128, 128)          # K
    assert cost(8, 8, 128) < cost(8, 64, 128) < cost(8, 128, 128) < cost(8, 256, 128)   # output columns
    assert cost(8, 128, 1) <= cost(8, 128, 32) < cost(8, 128, 64) < cost(8, 128, 65)    # requests: 1 box, 2 boxes, a full tile
    assert cost(8, 128, 65) == cost(8, 128, 128)                                 # a full tile is fetched whatever its fill


def test_cost_is_linear_in_k_beyond_the_fixed_part():
    c8, c16, c32 = cost(8, 256, 128), cost(16, 256, 128), cost(32, 256, 128)
    assert abs((c32 - c16) - 2 * (c16 - c8)) < 1e-6
    fixed = c8 - 8 * (c16 - c8) / 8
    assert 0 < fixed < c8 / 2


def test_items_cost_the_bytes_they_stream_per_k_block():
    # 256 columns x 64 K of weights plus a full activation tile = 48 KiB per K block: far more SM cycles at an SM's
    # share of the HBM stream than the four instructions need
    per_kb = (cost(9, 256, 128) - cost(8, 256, 128))
    assert abs(per_kb - (256 * 128 + 16384) / 23.0) < 1e-6
    # a transposed item of eight output features moves one 4 KiB activation box and 1 KiB of weights per K block
    per_kb = (cost(9, 8, 32) - cost(8, 8, 32))
    assert abs(per_kb - (8 * 128 + 4096) / 23.0) < 1e-6


def test_back_and_forth_dealing_of_a_sorted_list_is_balanced():
    # the library's dealing rule restated: rounds of `grid` items, odd rounds backwards
    rng = np.random.default_rng(0)
    grid = 148
    # a skewed mix: one tenant with wide layers and many requests among narrow ones with a few
    items = [cost(16, 256, 128)] * 90 + [cost(8, 128, int(r)) for r in rng.integers(1, 64, 1500)]
    items = np.array(sorted(items, reverse=True))

    def imbalance(order, snake):
        per = np.zeros(grid)
        for i, c in enumerate(order):
            k, r = divmod(i, grid)
            per[grid - 1 - r if (snake and k & 1) else r] += c
        return per.max() / per.mean()

    shuffled = items.copy()
    rng.shuffle(shuffled)
    assert imbalance(items, True) <= 1.15      # 90 heavy items over 148 CTAs: the granularity of the first round
    assert imbalance(items, True) <= imbalance(shuffled, False)
    assert imbalance(items, True) <= imbalance(items, False)
