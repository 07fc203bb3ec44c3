"""Shared helpers of the GPU parity tests (imported by test files; not a test module)."""
import numpy as np
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness

TOL = 2e-2   # |gpu - oracle| <= TOL * max(1, |oracle|) per output element (bf16 in, fp32 accumulate)


def fresh(max_models=64):
    mt.mt_shutdown()
    mt.mt_init(0, max_models, 0)


def check_bucketing(model_ids, n_tenants):
    counts, offsets, perm, inv = mt.mt_debug_last_bucketing(len(model_ids))
    oc, oo, op, oi = oracle.bucket(model_ids, n_tenants)
    assert np.array_equal(counts[:n_tenants], oc)
    assert np.array_equal(offsets[:n_tenants + 1], oo)
    assert offsets[-1] == len(model_ids)
    assert np.array_equal(perm, op)
    assert np.array_equal(inv, oi)


def run_and_check(models, model_ids, inputs, sample=None, max_models=None, tol=TOL, register=True):
    """Register (optionally), run one batch through the C-ABI, compare with the oracle.
    sample: arrival indices to check against the oracle (None = all).  Returns (gpu_out, max_scaled_err)."""
    if register:
        fresh(max_models or max(64, len(models)))
        ids = harness.register_models(models)
        assert ids == list(range(len(models)))
    got = harness.run_batch(model_ids, inputs, models[0][-1].out_ch)
    st, bad = mt.mt_get_async_status()
    assert (st, bad) == (0, -1)
    check_bucketing(model_ids, len(models))
    assert np.isfinite(got).all()
    if sample is None:
        ref = oracle.forward(models, model_ids, inputs)
        err = harness.scaled_error(got, ref)
    else:
        sample = np.asarray(sample)
        ref = oracle.forward(models, model_ids[sample], inputs[sample])
        err = harness.scaled_error(got[sample], ref)
    assert err.max() <= tol, "max scaled error %.3e (99.99th pct %.3e)" % (err.max(), np.quantile(err, 0.9999))
    return got, float(err.max())


def stratified_sample(model_ids, n_tenants, per_tenant, tile=128, seed=0):
    """Arrival indices covering, per tenant: first and last request of its segment, the neighbours of every
    multiple of `tile` in bucketed order, plus random ones up to per_tenant."""
    rng = np.random.default_rng(seed)
    _, offsets, perm, _ = oracle.bucket(model_ids, n_tenants)
    picked = []
    for t in range(n_tenants):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        pos = {lo, hi - 1}
        for b in range(lo + tile, hi, tile):
            pos.update((b - 1, b))
        pos = sorted(pos)[:max(per_tenant, 2)]
        extra = per_tenant - len(pos)
        if extra > 0 and hi - lo > len(pos):
            pos += rng.choice(np.arange(lo, hi), size=min(extra, hi - lo), replace=False).tolist()
        picked += [int(perm[p]) for p in set(pos)]
    return np.array(sorted(set(picked)), dtype=np.int64)
