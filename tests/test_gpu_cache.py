"""Weight residency tier (the paper's Sec. 3.3: weights cached in GPU memory, the rest one PCIe copy away): with a
device cache smaller than the registered models, batches still give the outputs of the all-resident context bit for
bit - a block that comes back is the same bytes - and the oracle's within tolerance; what cannot fit is refused on
the host; a request for an evicted model on the device-id path is reported, never faults."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth

from gpu_util import TOL, fresh

pytestmark = pytest.mark.gpu

WIDTHS = (256, 512, 384, 64)


def block_bytes(widths):
    """Device bytes of one MLP's block as the library lays it out: per layer 128-row x 64-column weight tiles of 16 KiB
    (an even number of row tiles once a layer is 256 wide), then the bias padded to whole tiles; pieces of 1 KiB."""
    total = 0
    for k, n in zip(widths[:-1], widths[1:]):
        tiles = (n + 127) // 128
        if n >= 256 and tiles % 2:
            tiles += 1
        total += tiles * (k // 64) * 16384
        total += (tiles * 128 * 4 + 1023) // 1024 * 1024
    return total


BLOCK = block_bytes(WIDTHS)                                                   # about 0.85 MB


def models_and_batches(T=6, n=700, n_batches=8):
    models = [synth.make_mlp(12, t, WIDTHS) for t in range(T)]
    rng = np.random.default_rng(4)
    batches = []
    for b in range(n_batches):
        live = rng.choice(T, size=3, replace=False)                  # three tenants per batch
        ids = live[rng.integers(0, 3, n)].astype(np.int32)
        x = synth.f32_to_bf16_bits(rng.standard_normal((n, WIDTHS[0])).astype(np.float32))
        batches.append((ids, x))
    return models, batches


def host_run(ids, x, out_elems, stream=None, asynchronous=False):
    n = len(ids)
    h_x = torch.from_numpy(x.view(np.int16)).pin_memory()
    h_ids = torch.from_numpy(ids).pin_memory()
    h_out = torch.full((n, out_elems), float("nan"), dtype=torch.float32).pin_memory()
    (mt.mt_infer_host_async if asynchronous else mt.mt_infer_host)(h_x, h_ids, n, h_out, stream)
    return h_out, (h_x, h_ids)


def test_evict_and_reload_gives_bit_identical_outputs_and_counts_hits():
    models, batches = models_and_batches()
    fresh()
    harness.register_models(models)
    want = [harness.run_batch(ids, x, 64) for ids, x in batches]          # every model resident
    for (ids, x), w in zip(batches[:2], want[:2]):
        assert harness.scaled_error(w, oracle.forward(models, ids, x)).max() <= TOL
    fresh()
    mt.mt_set_cache_bytes(int(3.5 * BLOCK))                                # room for three of the six
    harness.register_models(models)
    st0 = mt.mt_get_cache_stats(reset=True)
    assert st0["capacity_bytes"] > 0 and st0["resident_bytes"] <= st0["capacity_bytes"] and st0["evictions"] >= 3
    for rep in range(2):
        for (ids, x), w in zip(batches, want):
            got, _ = host_run(ids, x, 64)
            assert mt.mt_get_async_status() == (0, -1)
            assert np.array_equal(got.numpy(), w), rep
    st = mt.mt_get_cache_stats()
    assert st["tenant_hits"] + st["tenant_misses"] == 2 * len(batches) * 3
    assert st["tenant_misses"] >= 3 and st["tenant_hits"] >= 1
    assert st["request_hits"] + st["request_misses"] == 2 * sum(len(i) for i, _ in batches)
    assert st["bytes_loaded"] == st["tenant_misses"] * BLOCK
    assert st["resident_bytes"] <= st["capacity_bytes"]
    mt.mt_shutdown()


def test_batches_in_flight_on_two_streams_while_the_cache_thrashes():
    models, batches = models_and_batches(n_batches=10)
    fresh()
    harness.register_models(models)
    want = [harness.run_batch(ids, x, 64) for ids, x in batches]
    fresh()
    mt.mt_set_cache_bytes(int(3.2 * BLOCK))
    harness.register_models(models)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    keep = []
    for rep in range(3):
        outs = []
        for k, (ids, x) in enumerate(batches):                        # no synchronisation between the calls
            o, bufs = host_run(ids, x, 64, streams[k % 2], asynchronous=True)
            outs.append(o)
            keep.append(bufs)
        torch.cuda.synchronize()
        assert mt.mt_get_async_status() == (0, -1)
        for k, o in enumerate(outs):
            assert np.array_equal(o.numpy(), want[k]), (rep, k)
    assert mt.mt_get_cache_stats()["evictions"] > 10
    mt.mt_shutdown()


def test_what_does_not_fit_is_refused_on_the_host():
    models, batches = models_and_batches()
    fresh()
    mt.mt_set_cache_bytes(int(2.2 * BLOCK))                            # two tenants fit, a batch needs three
    harness.register_models(models)                                    # registration itself evicts as it goes
    ids, x = batches[0]
    with pytest.raises(mt.MtError) as e:
        host_run(ids, x, 64)
    assert e.value.code == 5                                           # MT_ERR_OOM, nothing enqueued
    with pytest.raises(mt.MtError) as e:
        mt.mt_prefetch([0, 1, 2])
    assert e.value.code == 5
    two = ids.copy()
    two[two == np.unique(ids)[2]] = np.unique(ids)[0]                  # the same batch on two tenants fits
    got, _ = host_run(two, x, 64)
    assert mt.mt_get_async_status() == (0, -1)
    assert harness.scaled_error(got.numpy(), oracle.forward(models, two, x)).max() <= TOL
    fresh()
    mt.mt_set_cache_bytes(BLOCK // 2)                                  # smaller than one model
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(models[0])
    assert e.value.code == 5
    with pytest.raises(mt.MtError) as e:                               # the cache size is fixed while models are registered
        mt.mt_set_cache_bytes(4 * BLOCK)
        mt.mt_register_model(models[0])
        mt.mt_set_cache_bytes(8 * BLOCK)
    assert e.value.code == 1
    mt.mt_shutdown()


def test_device_id_path_reports_an_evicted_model_and_prefetch_brings_it_back(small_batch_path):
    models, _ = models_and_batches()
    for m in models:                                                   # narrow enough for the one-launch path too
        assert max(l.out_ch for l in m) <= 512
    small = [synth.make_mlp(12, 50 + t, (128, 256, 192, 16)) for t in range(5)]
    block = block_bytes((128, 256, 192, 16))
    fresh()
    mt.mt_set_cache_bytes(int(3.3 * block))
    harness.register_models(small)                                     # tenants 2, 3, 4 are resident afterwards
    rng = np.random.default_rng(6)
    n = 300
    ids = rng.integers(2, 5, n).astype(np.int32)
    ids[17] = 0                                                        # registered, but evicted
    ids[200] = 9                                                       # never issued
    x = synth.f32_to_bf16_bits(rng.standard_normal((n, 128)).astype(np.float32))
    got = harness.run_batch(ids, x, 16)
    st, bad = mt.mt_get_async_status()
    assert st in (10, 2) and bad == 17                                 # MT_ERR_NOT_RESIDENT wins or ties with the unknown id
    assert np.isnan(got[[17, 200]]).all()
    good = np.ones(n, bool); good[[17, 200]] = False
    assert harness.scaled_error(got[good], oracle.forward(small, ids[good], x[good])).max() <= TOL
    ids[200] = 3
    got = harness.run_batch(ids, x, 16)
    assert mt.mt_get_async_status() == (10, 17)
    mt.mt_prefetch([0, 3, 4])                                          # displaces the least recently used tenant
    good[200] = True
    use = np.where(ids == 2, 3, ids).astype(np.int32)                  # tenant 2 was the victim: do not ask for it
    got = harness.run_batch(use, x, 16)
    assert mt.mt_get_async_status() == (0, -1)
    assert harness.scaled_error(got, oracle.forward(small, use, x)).max() <= TOL
    mt.mt_shutdown()
