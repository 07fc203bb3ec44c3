"""mt_bucket_noalloc - the entry point for callers that may not allocate device memory (allocator callbacks,
serving loops with a frozen memory map) - must give exactly the bucketing that mt_infer computes in its
cudaMalloc'ed workspace, and exactly the oracle's stable counting sort.  Two calls in a row on different batches:
the second one runs on a scratch array that still holds the first one's contents.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
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


class Buffers:
    """The caller's buffers: all of them exist before the calls under test."""
    def __init__(self, n_max, T_max):
        self.counts = torch.empty(T_max, dtype=torch.int32, device="cuda")
        self.offsets = torch.empty(T_max + 1, dtype=torch.int32, device="cuda")
        self.perm = torch.empty(max(n_max, 1), dtype=torch.int32, device="cuda")
        self.inv = torch.empty(max(n_max, 1), dtype=torch.int32, device="cuda")

    def call(self, d_ids, n, T):
        # poison, so that entries the call does not write cannot pass for results
        for t in (self.counts, self.offsets, self.perm, self.inv):
            t.fill_(-7)
        torch.cuda.synchronize()
        mt.mt_bucket_noalloc(d_ids, n, T, self.counts, self.offsets, self.perm, self.inv)
        torch.cuda.synchronize()
        return (self.counts[:T].cpu().numpy(), self.offsets[:T + 1].cpu().numpy(), self.perm[:n].cpu().numpy(),
                self.inv[:n].cpu().numpy())


def oracle_bucketing(ids, T):
    """The oracle's stable counting sort, with ids outside [0, T) sent to an extra last bucket."""
    good = (ids >= 0) & (ids < T)
    oc, oo, op, oi = oracle.bucket(np.where(good, ids, T).astype(np.int32), T + 1)
    return oc[:T], oo[:T + 1], op, oi


def driver_free_bytes():
    return torch.cuda.mem_get_info()[0]                 # the driver's view of the device, not torch's allocator


def test_no_alloc_bucketing_matches_mt_infer_twice_in_a_row():
    T = 300
    mt.mt_shutdown()
    mt.mt_init(0, 512, 0)
    harness.register_models(tiny_models(T))
    batches = [synth.zipf_ids(3, 20000, T, 0.9, salt=7), synth.zipf_ids(3, 777, T, 0.9, salt=8)]
    wanted = [existing_bucketing(ids) for ids in batches]
    buf = Buffers(max(len(b) for b in batches), T)
    dev_ids = [torch.from_numpy(b).cuda() for b in batches]
    buf.call(dev_ids[1], len(batches[1]), T)            # the first call on a device may load the module: not measured
    for ids, d_ids, (wc, wo, wp, wi) in zip(batches, dev_ids, wanted):
        n = len(ids)
        free_before = driver_free_bytes()
        c, o, p, i = buf.call(d_ids, n, T)
        assert driver_free_bytes() == free_before       # no device memory taken or returned by the call
        assert np.array_equal(c, wc[:T])                # integer work: bit-exact
        assert np.array_equal(o, wo[:T + 1])
        assert np.array_equal(p, wp)
        assert np.array_equal(i, wi)
        oc, oo, op, oi = oracle_bucketing(ids, T)       # and the oracle itself
        assert np.array_equal(c, oc) and np.array_equal(o, oo) and np.array_equal(p, op) and np.array_equal(i, oi)
    mt.mt_shutdown()


def test_no_alloc_limits_bad_ids_and_empty_batch_without_a_context():
    mt.mt_shutdown()                                    # no mt_init: the call needs no context
    rng = np.random.default_rng(5)
    T_max, n_max = 1024, 65536
    buf = Buffers(n_max, T_max)
    cases = [
        (rng.integers(0, T_max, n_max).astype(np.int32), T_max),             # the scratch exactly full
        (synth.zipf_ids(3, n_max, T_max, 1.2, salt=3), T_max),               # a few heavy buckets
        (rng.integers(-3, 40, 5000).astype(np.int32), 37),                   # ids below 0 and >= n_models sort last
        (np.full(300, 99, np.int32), 5),                                     # nothing valid at all
        (rng.integers(0, 2, 257).astype(np.int32), 1),                       # one model; id 1 is out of range
        (np.zeros(0, np.int32), 17),                                         # n == 0: counts and offsets all zero
        (rng.integers(0, 9, 1).astype(np.int32), 9),
    ]
    for ids, T in cases:
        n = len(ids)
        d_ids = torch.from_numpy(ids).cuda() if n else torch.zeros(1, dtype=torch.int32, device="cuda")
        c, o, p, i = buf.call(d_ids, n, T)
        oc, oo, op, oi = oracle_bucketing(ids, T) if n else (np.zeros(T, np.int32), np.zeros(T + 1, np.int32),
                                                                  np.zeros(0, np.int32), np.zeros(0, np.int32))
        assert np.array_equal(c, oc) and np.array_equal(o, oo)
        assert np.array_equal(p, op) and np.array_equal(i, oi)
        if n:   # a library routine as a second opinion: stable argsort of the clamped ids
            clamped = np.where((ids >= 0) & (ids < T), ids, T)
            assert np.array_equal(p, np.argsort(clamped, kind="stable").astype(np.int32))


def test_no_alloc_rejects_sizes_beyond_its_fixed_scratch():
    d = torch.zeros(8, dtype=torch.int32, device="cuda")
    for n, T in ((65537, 4), (4, 1025)):
        with pytest.raises(mt.MtError) as e:
            mt.mt_bucket_noalloc(d, n, T, d, d, d, d)
        assert e.value.code == 4                                      # MT_ERR_UNSUPPORTED, nothing was enqueued
    with pytest.raises(mt.MtError) as e:
        mt.mt_bucket_noalloc(d, -1, 4, d, d, d, d)
    assert e.value.code == 1
