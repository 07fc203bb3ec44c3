"""The five workloads at full size, in the launch configuration the bench times, checked on sampled
requests the oracle computes one by one (all outputs of each sampled request), plus properties that hold
at any size: bucketing bit-exact in full, outputs finite, repeat run bitwise identical.  Each case prints
the maximum and the 99.99th percentile of |gpu - oracle| / max(1, |oracle|) over the compared elements
(run with -s to see them); the tolerance is 2e-2."""
import numpy as np
import pytest

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth

from gpu_util import run_and_check, stratified_sample

pytestmark = pytest.mark.gpu


def full(config, per_tenant, max_models=64, more_salts=(), check_sample=None):
    """Registers the workload's models once; checks the default request draw and one further draw of ids and
    inputs per entry of more_salts against the same models."""
    wl = synth.make_workload(config)
    for k, salt in enumerate((0,) + tuple(more_salts)):
        ids, x = (wl.model_ids, wl.inputs) if k == 0 else synth.make_requests(config, wl.models, salt=salt)
        sample = stratified_sample(ids, len(wl.models), per_tenant)
        if check_sample is not None:
            check_sample(ids, len(wl.models), sample)
        stats = {}
        got, err = run_and_check(wl.models, ids, x, sample=sample, max_models=max_models, register=(k == 0), stats=stats)
        again = harness.run_batch(ids, x, wl.out_elems)
        assert np.array_equal(again, got)
        print("config %d, request draw %d: %d sampled requests, %d elements, max scaled error %.3e, 99.99th percentile %.3e"
              % (config, salt, len(sample), stats["elements"], stats["max"], stats["p9999"]))
    mt.mt_shutdown()


def last_pair_tile_is_sampled(ids, n_tenants, sample):
    """Every tenant's last 256-row tile (the ragged one of the CTA-pair executor) and its first one have a sampled
    request, and so does a tile in the middle of the segment."""
    _, offsets, _, inv = oracle.bucket(ids, n_tenants)
    pos = np.sort(inv[sample])
    for t in range(n_tenants):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        mine = pos[(pos >= lo) & (pos < hi)] - lo
        tiles = set((mine // 256).tolist())
        last = (hi - lo - 1) // 256
        assert 0 in tiles and last in tiles and last // 2 in tiles, (t, sorted(tiles), last)
        assert (hi - lo - 1) in mine.tolist()


def test_config2_full():
    full(2, 16, more_salts=(11, 12), check_sample=last_pair_tile_is_sampled)


def test_config3_full():
    full(3, 4, max_models=1024, more_salts=(11, 12))


def test_config4_full(conv_path):
    full(4, 3)


def test_config5_full():
    # at least 1024 requests, at least 128 per tenant: both neighbours of every 128- and 256-row boundary
    def check(ids, n_tenants, sample):
        assert len(sample) >= 1024 and np.bincount(ids[sample], minlength=n_tenants).min() >= 128
        last_pair_tile_is_sampled(ids, n_tenants, sample)
    full(5, 128, check_sample=check)
