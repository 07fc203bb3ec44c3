"""Shared helpers of the GPU parity tests (imported by test files; not a test module)."""
import numpy as np
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness

TOL = 2e-2   # |gpu - oracle| <= TOL * max(1, |oracle|) per output element (bf16 in, fp32 accumulate)


def tol_for_depth(n_layers):
    """The tolerance belongs to models of at most three layers (two hidden activations rounded to bf16, which the
    fp64 oracle does not imitate).  Each further rounded layer adds its share: restating the GPU's arithmetic in numpy
    (fp32 sums, hidden activations rounded to bf16) against the oracle gives maxima of 1.2e-2, 1.9e-2 and 2.5e-2 over
    48 000 outputs for MLPs of two, three and four layers - rounding alone, no GPU involved.  So: 1e-2 per rounded
    layer, never below TOL."""
    return max(TOL, 1e-2 * (n_layers - 1))


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


def run_and_check(models, model_ids, inputs, sample=None, max_models=None, tol=TOL, register=True, stats=None):
    """Register (optionally), run one batch through the C-ABI, compare with the oracle.
    sample: arrival indices to check against the oracle (None = all).  Returns (gpu_out, max_scaled_err);
    a dict passed as `stats` also receives the 99.99th percentile and the number of compared elements."""
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
    p9999 = float(np.quantile(err, 0.9999))
    if stats is not None:
        stats.update(max=float(err.max()), p9999=p9999, elements=int(err.size))
    assert err.max() <= tol, "max scaled error %.3e (99.99th pct %.3e)" % (err.max(), p9999)
    return got, float(err.max())


def sample_positions(lo, hi, per_tenant, tiles, rng):
    """Bucketed positions to check inside one segment [lo, hi).  Always the first and the last row; then both
    neighbours of row-tile boundaries (multiples of every width in `tiles`, widest first), spread evenly over the
    WHOLE segment when there are more of them than the budget allows, the last boundary (the one in front of the
    ragged tail tile) always among them; the rest of the budget is filled with random rows."""
    budget = max(int(per_tenant), 2)
    chosen = [lo] if hi - lo == 1 else [lo, hi - 1]
    seen = set(chosen)

    def take(p):
        if lo <= p < hi and p not in seen and len(chosen) < budget:
            seen.add(p)
            chosen.append(p)

    for tile in sorted(tiles, reverse=True):
        bounds = [b for b in range(lo + tile, hi, tile) if not (b in seen and b - 1 in seen)]   # not those a wider tile already gave
        room = (budget - len(chosen)) // 2
        if room <= 0 or not bounds:
            continue
        if len(bounds) > room:       # evenly spaced over the segment, ending with the last boundary
            idx = np.unique(np.round(np.linspace(0, len(bounds) - 1, room)).astype(int))
            bounds = [bounds[i] for i in idx]
        for b in reversed(bounds):   # the last boundary first: it survives whatever the budget
            take(b - 1)
            take(b)
    extra = min(budget - len(chosen), (hi - lo) - len(chosen))
    if extra > 0:
        rest = np.setdiff1d(np.arange(lo, hi), np.fromiter(seen, dtype=np.int64))
        for p in rng.choice(rest, size=extra, replace=False).tolist():
            take(int(p))
    return chosen


def stratified_sample(model_ids, n_tenants, per_tenant, tiles=(128, 256), seed=0):
    """Arrival indices covering, per tenant, the positions of sample_positions (at most per_tenant of them;
    128- and 256-row boundaries, since the CTA-pair executors work on 256-row tiles)."""
    rng = np.random.default_rng(seed)
    _, offsets, perm, _ = oracle.bucket(model_ids, n_tenants)
    picked = []
    for t in range(n_tenants):
        lo, hi = int(offsets[t]), int(offsets[t + 1])
        if hi == lo:
            continue
        picked += [int(perm[p]) for p in sample_positions(lo, hi, per_tenant, tiles, rng)]
    return np.array(sorted(set(picked)), dtype=np.int64)
