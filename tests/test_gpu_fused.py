"""The one-launch path for small batches of narrow MLPs (bucketing, all layers and the return to arrival order in a
single kernel) and the last layer's direct write to arrival order on the layer-by-layer path: parity with the fp64
oracle element by element, bit-exact bucketing, rejected ids, launch counts.  Everything goes through the C-ABI."""
import numpy as np
import pytest

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth

from gpu_util import TOL, fresh, run_and_check

pytestmark = pytest.mark.gpu


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def launches_of(fn):
    before = mt.mt_debug_launch_count()
    r = fn()
    return r, mt.mt_debug_launch_count() - before


def test_config1_is_one_launch_and_layered_path_agrees(monkeypatch):
    wl = synth.make_workload(1)
    (got, _), k = launches_of(lambda: run_and_check(wl.models, wl.model_ids, wl.inputs))
    assert k == 1
    mt.mt_debug_set_option("fused", 0)
    layered, k = launches_of(lambda: harness.run_batch(wl.model_ids, wl.inputs, 10))
    assert k == 4                                     # bucketing, three layers (the first reads through perm, the last writes through it)
    ref = oracle.forward(wl.models, wl.model_ids, wl.inputs)
    assert harness.scaled_error(layered, ref).max() <= TOL
    assert np.abs(layered - got).max() <= 1e-4        # same products; only the accumulation grouping may differ


@pytest.mark.parametrize("n,T,hidden,out", [(1, 1, (64,), 1), (512, 1, (256, 256), 256), (512, 200, (128, 192), 200),
                                            (300, 37, (256, 64, 256), 10), (129, 2, (192,), 72), (33, 1000, (64,), 8)])
def test_fused_shapes_many_tenants_and_ragged_units(n, T, hidden, out):
    # several 128-row units per tenant, tenants without requests, hidden widths that differ per tenant, outputs that
    # are not a multiple of 8 or 32 wide, more tenants than requests
    rng = np.random.default_rng(n + T)
    widths_of = lambda t: (128,) + tuple(int(rng.choice([64, 128, 192, 256])) if h != 64 else 64 for h in hidden) + (out,)
    models = [synth.make_mlp(7, 1000 * T + t, widths_of(t)) for t in range(T)]
    ids = rng.integers(0, T, n).astype(np.int32)
    if T > 2:
        ids[ids == 1] = 0                             # tenant 1 gets no request
    (_, err), k = launches_of(lambda: run_and_check(models, ids, bits(rng.standard_normal((n, 128))), max_models=max(64, T)))
    assert k == 1


def test_fused_rejected_ids_and_unaligned_output():
    import torch
    T = 6
    rng = np.random.default_rng(3)
    models = [synth.make_mlp(7, t, (64, 128, 12)) for t in range(T)]
    fresh()
    harness.register_models(models)
    mt.mt_release(2)
    ids = rng.integers(-1, T + 1, 200).astype(np.int32)            # -1, T and the released id 2 are rejected
    x = bits(rng.standard_normal((200, 64)))
    good = (ids >= 0) & (ids < T) & (ids != 2)
    # an output buffer that is only 4-byte aligned: the vector stores must not be used
    buf = torch.full((200 * 12 + 1,), float("nan"), dtype=torch.float32, device="cuda")
    out = buf[1:].view(200, 12)
    mt.mt_infer(harness.bf16_bits_to_device(x), torch.from_numpy(ids).cuda(), 200, out)
    st, bad = mt.mt_get_async_status()
    assert st == 2 and bad == int(np.flatnonzero(~good)[0])
    got = out.cpu().numpy()
    assert np.isnan(got[~good]).all()
    ref = oracle.forward(models, ids[good], x[good])
    assert harness.scaled_error(got[good], ref).max() <= TOL
    counts, offsets, perm, inv = mt.mt_debug_last_bucketing(200)
    live_ids = np.where(good, ids, T)
    oc, oo, op, oi = oracle.bucket(live_ids, T + 1)                # rejected requests form a last bucket, arrival order kept
    assert np.array_equal(counts, oc[:T]) and np.array_equal(offsets, oo)
    assert np.array_equal(perm, op) and np.array_equal(inv, oi)


@pytest.mark.parametrize("n", [513, 2000])
def test_layered_last_layer_writes_arrival_order_with_rejected_ids(n):
    # above the fused path's batch limit: the last grouped launch writes through perm and fills the rejected rows
    T = 9
    rng = np.random.default_rng(n)
    models = [synth.make_mlp(7, t, (128, 320, 40)) for t in range(T)]
    fresh()
    harness.register_models(models)
    ids = rng.integers(0, T + 2, n).astype(np.int32)
    x = bits(rng.standard_normal((n, 128)))
    good = ids < T
    (got), k = launches_of(lambda: harness.run_batch(ids, x, 40))
    assert k == 2 + 2                                 # two bucketing passes (rows move in the second), two layers; no un-permute pass
    st, bad = mt.mt_get_async_status()
    assert st == 2 and bad == int(np.flatnonzero(~good)[0])
    assert np.isnan(got[~good]).all() and np.isfinite(got[good]).all()
    ref = oracle.forward(models, ids[good], x[good])
    assert harness.scaled_error(got[good], ref).max() <= TOL


@pytest.mark.parametrize("seed", range(12))
def test_random_families_against_the_oracle(seed):
    # seeded random MLP families and batches: widths from 64 to 640 (inputs of a layer in multiples of 64, outputs
    # arbitrary), 1 to 40 tenants some of which get no request, segment sizes straddling the 64-request
    # (transposed items) and 128-request (row tile) borders, a few rejected ids; small draws take the one-launch
    # path, the others the layer-by-layer path
    rng = np.random.default_rng(1000 + seed)
    T = int(rng.integers(1, 41))
    depth = int(rng.integers(1, 5))
    k_in = 64 * int(rng.integers(1, 6))
    n_out = int(rng.integers(1, 300))
    small = seed % 3 == 0
    hid_choices = [64, 128, 192, 256] if small else [64, 128, 256, 320, 512, 640]
    models = []
    for t in range(T):
        widths = (k_in,) + tuple(int(rng.choice(hid_choices)) for _ in range(depth - 1)) + (n_out,)
        models.append(synth.make_mlp(8, 100 * seed + t, widths))
    sizes = rng.choice([0, 1, 3, 63, 64, 65, 127, 128, 129, 200], size=T)
    if small:
        sizes = np.minimum(sizes, max(1, 500 // T))
    ids = np.repeat(np.arange(T), sizes).astype(np.int32)
    if len(ids) == 0:
        ids = np.zeros(1, np.int32)
    n_bad = int(rng.integers(0, 4))
    ids = np.concatenate([ids, np.full(n_bad, T + 3, np.int32)])
    rng.shuffle(ids)
    n = len(ids)
    x = bits(rng.standard_normal((n, k_in)))
    fresh(max(64, T))
    harness.register_models(models)
    got = harness.run_batch(ids, x, n_out)
    st, bad = mt.mt_get_async_status()
    good = ids < T
    if n_bad:
        assert st == 2 and bad == int(np.flatnonzero(~good)[0])
        assert np.isnan(got[~good]).all()
    else:
        assert (st, bad) == (0, -1)
    counts, offsets, perm, inv = mt.mt_debug_last_bucketing(n)
    oc, oo, op, oi = oracle.bucket(np.where(good, ids, T), T + 1)
    assert np.array_equal(counts, oc[:T]) and np.array_equal(offsets, oo)
    assert np.array_equal(perm, op) and np.array_equal(inv, oi)
    ref = oracle.forward(models, ids[good], x[good])
    assert np.isfinite(got[good]).all()
    assert harness.scaled_error(got[good], ref).max() <= TOL


@pytest.mark.parametrize("case", ["c2_reduced", "c3_reduced", "pair", "ragged_single", "tiny_layered"])
def test_first_layer_reads_rows_through_perm(case, monkeypatch):
    # MT_PERM_GATHER=2: the first dense layer fetches its rows from the caller's buffer through the permutation (four
    # rows per TMA gather) at every batch size - 128-row tiles, transposed small segments, the CTA-pair executor - and
    # no row pass runs; results must equal the row-move path's bit for bit (same operands, same order of products)
    if case == "c2_reduced":
        wl = synth.make_workload(2, n=900, n_tenants=7, widths=(1024, 512, 640, 256))
    elif case == "c3_reduced":
        wl = synth.make_workload(3, n=1500, n_tenants=120)
    elif case == "pair":
        wl = synth.make_workload(5, n=2500, n_tenants=2, widths=(256, 512, 256))
    elif case == "ragged_single":
        wl = synth.make_workload(5, n=385, n_tenants=1, widths=(128, 320, 130))
    else:
        wl = synth.make_workload(1)
        monkeypatch.setenv("MT_FUSED", "0")
    T = len(wl.models)
    monkeypatch.setenv("MT_PERM_GATHER", "2")
    (got, _), k = launches_of(lambda: run_and_check(wl.models, wl.model_ids, wl.inputs, max_models=max(64, T)))
    n_layers = len(wl.models[0])
    assert k == (1 if wl.n <= 512 else 2) + n_layers          # bucketing and the layers, nothing else
    monkeypatch.setenv("MT_PERM_GATHER", "0")
    moved, _ = run_and_check(wl.models, wl.model_ids, wl.inputs, max_models=max(64, T))
    assert np.array_equal(got, moved)


def test_skewed_family_is_scheduled_evenly_and_matches_the_oracle():
    # one tenant with 1024-wide layers and a quarter of the requests among thirty 128-wide ones: its work items cost
    # eight times the others'.  Laid out heaviest first and dealt back and forth, every CTA's modelled share of a layer
    # stays within 1.2x of the mean; the results are the oracle's whatever the order
    rng = np.random.default_rng(77)
    T = 31
    models = [synth.make_mlp(9, 0, (512, 1024, 1024, 64))] + [synth.make_mlp(9, t, (512, 128, 128, 64)) for t in range(1, T)]
    n = 30000                                          # about 4.5 work items per CTA: below that the item size itself bounds the balance
    ids = np.where(rng.random(n) < 0.25, 0, rng.integers(1, T, n)).astype(np.int32)
    x = bits(rng.standard_normal((n, 512)))
    run_and_check(models, ids, x)
    for layer, least_items in ((0, 400), (1, 400)):
        ratio, n_items, n_ctas = mt.mt_debug_schedule_balance(layer)
        assert n_items >= least_items and n_ctas == 148
        assert ratio <= 1.2, (layer, ratio, n_items)


def test_work_item_order_follows_cost_after_release_and_reregistration():
    # ranks are recomputed whenever the set of models changes: release the heavy tenant, run, register it again
    # under the freed id, run again - both batches match the oracle
    rng = np.random.default_rng(78)
    models = [synth.make_mlp(9, 100 + t, (128, 640 if t == 3 else 128, 40)) for t in range(6)]
    fresh()
    harness.register_models(models)
    n = 1500
    x = bits(rng.standard_normal((n, 128)))
    ids = rng.integers(0, 6, n).astype(np.int32)
    run_and_check(models, ids, x, register=False)
    mt.mt_release(3)
    live = ids != 3
    got = harness.run_batch(ids, x, 40)
    assert mt.mt_get_async_status()[0] == 2 and np.isnan(got[~live]).all()
    assert harness.scaled_error(got[live], oracle.forward(models, ids[live], x[live])).max() <= TOL
    assert mt.mt_register_model(models[3]) == 3
    run_and_check(models, ids, x, register=False)


def test_small_conv_batches_are_bucketed_by_the_conv_launch_itself():
    # at most 512 requests on the CTA-pair conv executor, pool + head at the end: no bucketing launch - every CTA of the
    # first conv launch repeats the stable counting sort in shared memory and CTA 0 publishes it for the launches behind
    # it (a second conv launch when there are more than four conv layers, the pool + head launch).  Same bits as with
    # the bucketing launch; rejected ids come back as NaN rows with the status of the smallest offending index.
    for n_conv, n, T, h, w in ((4, 37, 5, 9, 40), (6, 50, 3, 6, 44), (2, 512, 16, 3, 33), (2, 500, 300, 2, 33)):
        wl = synth.make_workload(4, n=n, n_tenants=T, h=h, w=w, n_conv=n_conv)
        ids = wl.model_ids.copy()
        ids[[3, n - 2]] = [T + 4, -1]                               # never issued / negative
        fresh(max_models=max(64, T))
        harness.register_models(wl.models)
        want_launches = (2 if n_conv <= 4 else 3)                   # conv stack(s) + pool-and-head
        got, k = launches_of(lambda: harness.run_batch(ids, wl.inputs, 10))
        assert k == want_launches
        assert mt.mt_get_async_status() == (2, 3)
        good = (ids >= 0) & (ids < T)
        assert np.isnan(got[~good]).all() and np.isfinite(got[good]).all()
        counts, offsets, perm, inv = mt.mt_debug_last_bucketing(n)
        oc, oo, op, oi = oracle.bucket(np.where(good, ids, T).astype(np.int32), T + 1)
        assert np.array_equal(counts[:T], oc[:T]) and np.array_equal(offsets[:T + 1], oo[:T + 1]) and offsets[T + 1] == n
        assert np.array_equal(perm, op) and np.array_equal(inv, oi)
        ref = oracle.forward(wl.models, ids[good], wl.inputs[good])
        assert harness.scaled_error(got[good], ref).max() <= TOL
        mt.mt_debug_set_option("conv_self_bucket", 0)
        try:
            other, k2 = launches_of(lambda: harness.run_batch(ids, wl.inputs, 10))
        finally:
            mt.mt_debug_set_option("conv_self_bucket", 1)
        assert k2 == want_launches + 1 and mt.mt_get_async_status() == (2, 3)
        assert np.array_equal(np.nan_to_num(got, nan=-1.0), np.nan_to_num(other, nan=-1.0))
        # a larger batch on the same context takes the bucketing launch again, then a small one the short way
        big = synth.make_requests(4, wl.models, n=600, salt=7)
        run_and_check(wl.models, big[0], big[1], register=False)
        small = synth.make_requests(4, wl.models, n=11, salt=8)
        _, k3 = launches_of(lambda: run_and_check(wl.models, small[0], small[1], register=False))
        assert k3 == want_launches


def test_conv_context_with_more_id_slots_than_the_conv_launch_sorts_keeps_the_bucketing_launch():
    # the in-launch sort holds its tables for at most 512 id slots: with 513 registered models the batch is bucketed
    # by a launch of its own again, same results against the oracle
    T, h, w = 513, 2, 33
    wl = synth.make_workload(4, n=40, n_tenants=T, h=h, w=w, n_conv=2)
    fresh(max_models=T)
    harness.register_models(wl.models)
    (got, _), k = launches_of(lambda: run_and_check(wl.models, wl.model_ids, wl.inputs, register=False))
    assert k == 3
    mt.mt_release(T - 1)                                           # id slots stay 513: still the bucketing launch
    keep = wl.model_ids != T - 1
    _, k = launches_of(lambda: run_and_check(wl.models, wl.model_ids[keep], wl.inputs[keep], register=False))
    assert k == 3
