"""mt_bucket_noalloc - the entry point for callers that may not allocate device memory (allocator callbacks,
serving loops with a frozen memory map) - must give exactly the bucketing that mt_infer computes in its
cudaMalloc'ed workspace.  Two calls in a row on different batches: the second one runs on a scratch array
that still holds the first one's contents.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from paper_1901_06887_b200 import binding as mt, harness, synth
from paper_1901_06887_b200.synth import DENSE, Layer

pytestmark = pytest.mark.gpu


def tiny_models(T):
    w = synth.f32_to_bf16_bits(np.eye(8, 64, dtype=np.float32))
    return [[Layer(DENSE, 64, 8, relu=0, weight=w, bias=None)] for _ in range(T)]


def existing_bucketing(ids):
    x = np.zeros((len(ids), 64), np.uint16)
    harness.run_batch(ids, x, 8)                       # the existing path: mt_infer, workspace from cudaMalloc
    assert mt.mt_get_async_status() == (0, -1)
    return mt.mt_debug_last_bucketing(len(ids))


def test_no_alloc_bucketing_matches_mt_infer_twice_in_a_row():
    T = 300
    mt.mt_shutdown()
    mt.mt_init(0, 512, 0)
    harness.register_models(tiny_models(T))
    batches = [synth.zipf_ids(3, 20000, T, 0.9, salt=7), synth.zipf_ids(3, 777, T, 0.9, salt=8)]
    wanted = [existing_bucketing(ids) for ids in batches]
    # all output buffers exist before the calls; the calls themselves allocate nothing
    n_max = max(len(b) for b in batches)
    counts = torch.empty(T, dtype=torch.int32, device="cuda")
    offsets = torch.empty(T + 1, dtype=torch.int32, device="cuda")
    perm = torch.empty(n_max, dtype=torch.int32, device="cuda")
    inv = torch.empty(n_max, dtype=torch.int32, device="cuda")
    dev_ids = [torch.from_numpy(b).cuda() for b in batches]
    torch.cuda.synchronize()
    for ids, d_ids, (wc, wo, wp, wi) in zip(batches, dev_ids, wanted):
        n = len(ids)
        before = torch.cuda.memory_allocated()
        mt.mt_bucket_noalloc(d_ids, n, T, counts, offsets, perm, inv)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        assert np.array_equal(counts.cpu().numpy(), wc[:T])          # integer work: bit-exact
        assert np.array_equal(offsets.cpu().numpy(), wo[:T + 1])
        assert np.array_equal(perm[:n].cpu().numpy(), wp)
        assert np.array_equal(inv[:n].cpu().numpy(), wi)
    mt.mt_shutdown()


def test_no_alloc_rejects_sizes_beyond_its_fixed_scratch():
    d = torch.zeros(8, dtype=torch.int32, device="cuda")
    for n, T in ((65537, 4), (4, 1025)):
        with pytest.raises(mt.MtError) as e:
            mt.mt_bucket_noalloc(d, n, T, d, d, d, d)
        assert e.value.code == 4                                      # MT_ERR_UNSUPPORTED, nothing was enqueued
    with pytest.raises(mt.MtError) as e:
        mt.mt_bucket_noalloc(d, -1, 4, d, d, d, d)
    assert e.value.code == 1
