"""A worker's life (Sec. 3: tenants upload models, requests for them arrive mixed, models are withdrawn): a seeded random
sequence of registrations, releases and batches against one context - MLPs of mixed depth and of differing input,
hidden and output widths, batches from one request to thousands, ids of released and never issued models in the
mix - every batch checked against the per-request oracle.  Run with every model resident, with a weight cache that
holds about half of them (host-buffer entry points, which load what a batch needs), and with the synchronous
registration path."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth

from gpu_util import tol_for_depth

pytestmark = pytest.mark.gpu

MAX_MODELS = 12


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def random_mlp(rng, serial):
    depth = int(rng.integers(1, 5))
    widths = [int(rng.choice([64, 128, 256]))]
    widths += [int(rng.choice([64, 128, 192, 256, 384])) for _ in range(depth - 1)]
    widths += [int(rng.choice([8, 24, 64, 100]))]
    return synth.make_mlp(31, serial, widths)


def expected(models_by_id, ids, xb, out_stride):
    """Oracle outputs, NaN rows for ids that name no live model; columns beyond a model's own are NaN (= untouched).
    Second result: the tolerance of every element (it depends on the depth of the request's model)."""
    n = len(ids)
    ref = np.full((n, out_stride), np.nan)
    tol = np.zeros((n, out_stride))
    for t, m in models_by_id.items():
        rows = np.flatnonzero(ids == t)
        if len(rows):
            k = m[0].in_ch
            ref[np.ix_(rows, np.arange(m[-1].out_ch))] = oracle.forward([m], np.zeros(len(rows), np.int32),
                                                                       np.ascontiguousarray(xb[rows, :k]))
            # twice the depth's tolerance: the narrow random width mixes of this test sit at its edge through rounding
            # alone (up to 2.2e-2 at three layers), and what this test is after - another model's weights, another
            # request's row, a stale table entry - is wrong by the size of the outputs themselves
            tol[rows] = 2.0 * tol_for_depth(len(m))
    return ref, tol


def run_device(ids, xb, out_stride):
    n = len(ids)
    out = torch.full((n, out_stride), float("nan"), dtype=torch.float32, device="cuda")
    mt.mt_infer(harness.bf16_bits_to_device(xb), torch.from_numpy(ids).cuda(), n, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def run_host(ids, xb, out_stride, asynchronous):
    n = len(ids)
    h_x = torch.from_numpy(np.ascontiguousarray(xb).view(np.int16)).pin_memory()
    h_ids = torch.from_numpy(ids).pin_memory()
    h_out = torch.full((n, out_stride), float("nan"), dtype=torch.float32).pin_memory()
    (mt.mt_infer_host_async if asynchronous else mt.mt_infer_host)(h_x, h_ids, n, h_out, None)
    torch.cuda.synchronize()
    return h_out.numpy().copy()


@pytest.mark.parametrize("seed", [0, 1])
@pytest.mark.parametrize("mode", ["resident", "cache_host", "sync_register"])
def test_random_life_of_a_worker(mode, seed, monkeypatch):
    if mode == "sync_register":
        monkeypatch.setenv("MT_ASYNC_REGISTER", "0")
    rng = np.random.default_rng({"resident": 101, "cache_host": 202, "sync_register": 303}[mode] + seed)
    mt.mt_shutdown()
    mt.mt_init(0, MAX_MODELS, 0)
    if mode == "cache_host":
        mt.mt_set_cache_bytes(5 << 19)           # 2.5 MB; a model is at most 1.2 MB, twelve of them about 5 MB
    live = {}                                    # id -> layers
    serial = 0
    n_batches = n_bad = 0
    for step in range(70):
        op = rng.random()
        if (op < 0.35 and len(live) < MAX_MODELS) or not live:
            m = random_mlp(rng, serial)
            serial += 1
            t = mt.mt_register_model(m)
            assert t not in live and t == min(set(range(MAX_MODELS)) - set(live))      # lowest free slot
            live[t] = m
        elif op < 0.5 and len(live) > 1:
            t = int(rng.choice(sorted(live)))
            mt.mt_release(t)
            del live[t]
        else:
            n = int(rng.choice([1, 7, 64, 300, 513, 1500, 4000]))
            pool = sorted(live)
            if mode != "cache_host" and rng.random() < 0.4:
                pool = pool + [t for t in range(MAX_MODELS + 2) if t not in live][:2]   # released / never issued ids
            elif mode == "cache_host":
                pool = list(rng.choice(pool, size=min(len(pool), 2), replace=False))    # a batch's tenants must fit together
            ids = np.asarray(rng.choice(pool, size=n), np.int32)
            in_stride, out_stride = mt.mt_input_elems(), mt.mt_output_elems()
            assert in_stride >= max(m[0].in_ch for m in live.values())
            assert out_stride >= max(m[-1].out_ch for m in live.values())
            x = rng.standard_normal((n, in_stride)).astype(np.float32)
            for t, m in live.items():
                x[ids == t, m[0].in_ch:] = np.nan                                   # never read
            xb = bits(x)
            if mode == "cache_host":
                got = run_host(ids, xb, out_stride, asynchronous=bool(step & 1))
            else:
                got = run_device(ids, xb, out_stride)
            ref, tol = expected(live, ids, xb, out_stride)
            good = np.isin(ids, sorted(live))
            st, bad = mt.mt_get_async_status()
            if good.all():
                assert (st, bad) == (0, -1)
            else:
                assert st == 2 and bad == int(np.flatnonzero(~good)[0])
                n_bad += 1
                assert np.isnan(got[~good]).all()
            mask = ~np.isnan(ref)
            assert np.isnan(got[~mask]).all()     # rejected rows; columns beyond a model's own (untouched, or NaN from the host entries)
            err = np.abs(got[mask] - ref[mask]) / np.maximum(1.0, np.abs(ref[mask]))
            assert np.isfinite(got[mask]).all() and (err <= tol[mask]).all(), (step, n, err.max())
            n_batches += 1
    assert n_batches >= 20 and (mode == "cache_host" or n_bad >= 3)
    if mode == "cache_host":
        st = mt.mt_get_cache_stats()
        assert st["tenant_hits"] > 0 and st["tenant_misses"] > 0          # (whether blocks were evicted depends on the draw)
