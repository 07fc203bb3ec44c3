"""Bit-exact bucketing parity (histogram, exclusive scan, stable scatter, permutation) and the
un-permute round trip, through the C-ABI, against the oracle's stable counting sort."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth
from paper_1901_06887_b200.synth import DENSE, Layer

from gpu_util import check_bucketing, fresh

pytestmark = pytest.mark.gpu


def passthrough_models(T, width=64):
    """T one-layer models that select their input's first 8 features scaled by (id + 1): out = (t+1) * x[:8].
    Exact in bf16/fp32 for small integers, so outputs also prove each row went to its own model and back."""
    models = []
    for t in range(T):
        w = np.zeros((8, width), np.float32)
        w[np.arange(8), np.arange(8)] = float(t % 64 + 1)
        models.append([Layer(DENSE, width, 8, relu=0, weight=synth.f32_to_bf16_bits(w), bias=None)])
    return models


def run_ids(T, ids, registered=None):
    ids = np.asarray(ids, np.int32)
    n = len(ids)
    rng = np.random.default_rng(n + T)
    x = rng.integers(-8, 9, size=(n, 64)).astype(np.float32)
    got = harness.run_batch(ids, synth.f32_to_bf16_bits(x), 8)
    assert mt.mt_get_async_status() == (0, -1)
    check_bucketing(ids, T)
    want = x[:, :8] * ((ids % 64) + 1)[:, None]
    assert np.array_equal(got, want)            # un-permute(bucket(.)) restores arrival order, bit for bit


@pytest.mark.parametrize("T", [1, 4, 37, 1000])
def test_bucketing_distributions(T, small_batch_path):
    fresh(max(64, T))
    harness.register_models(passthrough_models(T))
    rng = np.random.default_rng(T)
    run_ids(T, [0])                                              # n = 1
    run_ids(T, [T - 1] * 33)                                     # all one tenant, n not a multiple of 32
    run_ids(T, rng.integers(0, T, 257))                          # one element past a 256-request block
    run_ids(T, rng.integers(0, T, 5000))                         # many blocks
    run_ids(T, np.arange(3 * T) % T)                             # every tenant, round robin
    run_ids(T, np.repeat(np.arange(T), 2)[::-1].copy())          # descending ids
    if T > 2:
        run_ids(T, rng.choice([0, T - 1], 1000))                 # most tenants empty
    run_ids(T, synth.zipf_ids(3, 4096, T, 0.9))


def test_bucketing_full_size_id_draws():
    for cfg, n, T, s in ((2, 4096, 64, 1.1), (3, 16384, 1000, 0.9), (5, 65536, 8, 0.0), (4, 256, 16, 1.0)):
        fresh(max(64, T))
        harness.register_models(passthrough_models(T))
        run_ids(T, synth.zipf_ids(cfg, n, T, s))


def test_empty_batch_is_a_noop():
    fresh()
    harness.register_models(passthrough_models(2))
    out = torch.zeros((4, 8), device="cuda")
    x = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
    ids = torch.zeros(4, dtype=torch.int32, device="cuda")
    mt.mt_infer(x, ids, 0, out)
    assert mt.mt_get_async_status() == (0, -1)
    assert float(out.abs().sum()) == 0.0


def test_rejected_ids_give_nan_rows_and_a_status(small_batch_path):
    T = 5
    fresh()
    harness.register_models(passthrough_models(T))
    mt.mt_release(3)                                             # id 3 is now dead
    ids = np.array([0, 3, 1, 7, -2, 4, 3, 2, 0], np.int32)       # 3: released, 7: never issued, -2: negative
    x = np.ones((len(ids), 64), np.float32)
    got = harness.run_batch(ids, synth.f32_to_bf16_bits(x), 8)
    st, bad = mt.mt_get_async_status()
    assert st == 2 and bad == 1                                  # MT_ERR_BAD_MODEL_ID, first offending arrival index
    good = np.isin(ids, [0, 1, 2, 4])
    assert np.isnan(got[~good]).all()
    assert np.array_equal(got[good], (ids[good] + 1)[:, None] * np.ones((good.sum(), 8), np.float32))
    counts, offsets, perm, inv = mt.mt_debug_last_bucketing(len(ids))
    assert counts.tolist() == [2, 1, 1, 0, 1] and offsets.tolist() == [0, 2, 3, 4, 4, 5, 9]
    assert perm[:5].tolist() == [0, 8, 2, 7, 5] and sorted(perm[5:].tolist()) == [1, 3, 4, 6]
    assert mt.mt_get_async_status() == (0, -1)                   # reading cleared the sticky status
    # the freed slot is re-issued, lowest first
    assert mt.mt_register_model(passthrough_models(4)[3]) == 3
    run_ids(T, [3, 3, 0])


def test_bounded_device_wait_gives_up_and_context_survives():
    # a wait that nothing satisfies runs into its time limit: status MT_ERR_TIMEOUT, no hang, no trap, and the
    # next batch runs normally
    fresh()
    harness.register_models(passthrough_models(3))
    run_ids(3, [0, 1, 2, 1])
    mt.mt_debug_wait_timeout(20)
    st, bad = mt.mt_get_async_status()
    assert st == 8 and bad == -1                      # MT_ERR_TIMEOUT
    assert mt.mt_get_async_status() == (0, -1)        # cleared by the read
    run_ids(3, [2, 2, 0])
