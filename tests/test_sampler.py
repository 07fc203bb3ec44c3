"""The request sampler of the full-size parity tests (host logic, no GPU): it must keep each segment's first and
last row and rows next to tile boundaries over the WHOLE segment, whatever the budget."""
import numpy as np

from gpu_util import sample_positions, stratified_sample


def test_positions_cover_the_whole_segment_within_the_budget():
    rng = np.random.default_rng(0)
    for lo, hi, budget in [(0, 8190, 128), (100, 1140, 16), (5, 6, 4), (5, 7, 4), (0, 8190, 12), (0, 300, 6),
                           (0, 129, 6), (0, 700, 3), (0, 65, 16), (0, 3, 16), (7, 7 + 4096, 2)]:
        p = sample_positions(lo, hi, budget, (128, 256), rng)
        assert len(p) == len(set(p)) == min(max(budget, 2), hi - lo)
        assert all(lo <= q < hi for q in p) and lo in p and hi - 1 in p
        if budget >= 4 and hi - lo > 256:
            last = lo + (hi - lo - 1) // 256 * 256          # first row of the ragged last 256-row tile
            assert last in p and last - 1 in p


def test_all_boundaries_when_the_budget_allows():
    p = set(sample_positions(0, 8190, 128, (128, 256), np.random.default_rng(1)))
    for b in range(128, 8190, 128):
        assert b in p and b - 1 in p


def test_sample_hits_every_tenant_with_requests():
    rng = np.random.default_rng(3)
    ids = rng.integers(0, 9, 5000).astype(np.int32)
    ids[ids == 4] = 5                                        # tenant 4 has no request
    s = stratified_sample(ids, 9, 10)
    assert len(set(s.tolist())) == len(s)
    got = np.bincount(ids[s], minlength=9)
    assert got[4] == 0 and (np.delete(got, 4) == 10).all()
