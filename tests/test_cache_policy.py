"""The weight cache's policy on a made-up clock (host code of the library; no GPU): first-fit placement in a fixed
arena, least-recently-used eviction, blocks of the current tick protected, free ranges merged again."""
import numpy as np
import pytest

from paper_1901_06887_b200 import binding as mt

KB = 1024


@pytest.fixture
def sim():
    h = mt.mt_cache_sim_create(10 * KB)
    yield h
    mt.mt_cache_sim_destroy(h)


def test_hits_misses_and_lru_order(sim):
    acc = lambda i, size, tick: mt.mt_cache_sim_access(sim, i, size, tick)
    assert acc(0, 4 * KB, 1) == (1, 0, [])                 # placed at offset 0
    assert acc(1, 4 * KB, 2) == (1, 4 * KB, [])
    assert acc(0, 4 * KB, 3) == (0, 0, [])                 # hit: refreshes model 0
    r, off, ev = acc(2, 4 * KB, 4)                         # 2 KB free: someone must go, and model 1 is the oldest
    assert (r, ev) == (1, [1]) and off == 4 * KB
    assert acc(1, 4 * KB, 5)[2] == [0]                     # now model 0 (tick 3) is older than model 2 (tick 4)
    st = mt.mt_cache_sim_stats(sim)
    assert (st["tenant_hits"], st["tenant_misses"], st["evictions"]) == (1, 4, 2)
    assert st["bytes_loaded"] == 16 * KB and st["resident_bytes"] == 8 * KB and st["capacity_bytes"] == 10 * KB


def test_blocks_of_the_current_tick_are_never_victims(sim):
    assert mt.mt_cache_sim_access(sim, 0, 4 * KB, 7)[0] == 1
    assert mt.mt_cache_sim_access(sim, 1, 4 * KB, 7)[0] == 1
    r, off, ev = mt.mt_cache_sim_access(sim, 2, 4 * KB, 7)       # the batch of tick 7 does not fit as a whole
    assert (r, off, ev) == (-1, -1, [])
    assert mt.mt_cache_sim_access(sim, 0, 4 * KB, 7)[0] == 0     # and nothing of it was displaced
    assert mt.mt_cache_sim_access(sim, 2, 4 * KB, 8) == (1, 0, [0])   # next tick: ties in age go to the lowest id


def test_a_block_larger_than_the_arena_is_refused_and_sizes_round_to_the_alignment(sim):
    assert mt.mt_cache_sim_access(sim, 0, 11 * KB, 1)[0] == -1
    assert mt.mt_cache_sim_access(sim, 0, 1, 1) == (1, 0, [])
    assert mt.mt_cache_sim_access(sim, 1, 1, 1) == (1, KB, [])         # 1024-byte granules
    assert mt.mt_cache_sim_stats(sim)["resident_bytes"] == 2 * KB


def test_freed_neighbours_merge_so_a_large_block_fits_again(sim):
    for i in range(5):
        assert mt.mt_cache_sim_access(sim, i, 2 * KB, 1 + i)[0] == 1   # five blocks of 2 KB fill the arena
    mt.mt_cache_sim_release(sim, 1)
    mt.mt_cache_sim_release(sim, 3)
    mt.mt_cache_sim_release(sim, 2)                                    # 1, 2, 3 are neighbours: 6 KB in one piece
    r, off, ev = mt.mt_cache_sim_access(sim, 9, 6 * KB, 10)
    assert (r, off, ev) == (1, 2 * KB, [])
    assert mt.mt_cache_sim_stats(sim)["evictions"] == 0                # a withdrawn model is not an eviction


def test_eviction_continues_until_a_contiguous_range_is_free(sim):
    for i in range(5):
        mt.mt_cache_sim_access(sim, i, 2 * KB, 1 + i)
    r, off, ev = mt.mt_cache_sim_access(sim, 7, 5 * KB, 20)            # needs three neighbours gone
    assert r == 1 and ev == [0, 1, 2] and off == 0


def test_against_a_plain_lru_model_on_a_random_trace():
    # equal block sizes: the arena behaves exactly like a textbook LRU list of capacity // size entries
    rng = np.random.default_rng(0)
    size, slots = 3 * KB, 7
    h = mt.mt_cache_sim_create(slots * size)
    lru = []                                   # most recent last
    hits = 0
    for tick, i in enumerate(rng.zipf(1.3, 4000) % 40, start=1):
        r, _, ev = mt.mt_cache_sim_access(h, int(i), size, tick)
        if i in lru:
            assert r == 0 and ev == []
            lru.remove(i)
            hits += 1
        else:
            assert r == 1
            assert ev == ([lru.pop(0)] if len(lru) == slots else [])
        lru.append(i)
    st = mt.mt_cache_sim_stats(h)
    assert st["tenant_hits"] == hits and st["tenant_misses"] == 4000 - hits
    mt.mt_cache_sim_destroy(h)
