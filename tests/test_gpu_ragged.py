"""Families of mixed depth: MLP tenants with two, three and four layers (and differing hidden widths) share one
context and one batch (the paper's catalogue of models is not uniform: Sec. 3.1 describes models as lists of
standard layers of any length).  A tenant's layer j runs in the family's j-th launch; its last layer - whichever
launch that is - writes the fp32 output in arrival order.  Checked against the per-request oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth

from gpu_util import TOL, fresh, run_and_check

pytestmark = pytest.mark.gpu


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def mixed_models(k_in, n_out, hidden_choices, T, seed, depths=(2, 3, 4, 1)):
    rng = np.random.default_rng(seed)
    models = []
    for t in range(T):
        d = depths[t % len(depths)]
        widths = (k_in,) + tuple(int(rng.choice(hidden_choices)) for _ in range(d - 1)) + (n_out,)
        models.append(synth.make_mlp(11, 1000 * seed + t, widths))
    return models


def test_mixed_depths_small_batch_both_paths(small_batch_path):
    # at most 512 requests, layers at most 256 wide: one fused launch (or, with MT_FUSED=0, the layer-by-layer path)
    models = mixed_models(128, 24, [64, 128, 192, 256], 9, 1)
    assert sorted({len(m) for m in models}) == [1, 2, 3, 4]
    rng = np.random.default_rng(5)
    n = 400
    ids = rng.integers(0, 9, n).astype(np.int32)
    run_and_check(models, ids, bits(rng.standard_normal((n, 128))))


@pytest.mark.parametrize("n,T,hidden", [(3000, 12, [128, 320, 512]), (9000, 5, [256, 512]), (700, 40, [64, 640])])
def test_mixed_depths_layered_path(n, T, hidden):
    # segments from a handful of requests (transposed items) to thousands (full tiles); 128- and 256-column work items
    models = mixed_models(256, 72, hidden, T, 2 + T)
    ids = synth.zipf_ids(3, n, T, 1.0, salt=T)
    rng = np.random.default_rng(n)
    got, _ = run_and_check(models, ids, bits(rng.standard_normal((n, 256))))
    # the order of registration must not matter: deepest model last, so the family grows while models are added
    order = np.argsort([len(m) for m in models], kind="stable")
    remap = np.empty(T, np.int32)
    remap[order] = np.arange(T, dtype=np.int32)
    got2, _ = run_and_check([models[i] for i in order], remap[ids], bits(np.random.default_rng(n).standard_normal((n, 256))))
    assert np.array_equal(got, got2)


def test_mixed_depths_cta_pair_executor_and_rejected_ids():
    # two tenants with thousands of requests each and layers at least 256 wide: the 256 x 256 CTA-pair executor; one
    # tenant stops after two layers, the other after three; two ids are never issued
    m2 = synth.make_mlp(11, 50, (256, 512, 256))
    m3 = synth.make_mlp(11, 51, (256, 512, 256, 256))
    rng = np.random.default_rng(8)
    n = 2600
    ids = rng.integers(0, 2, n).astype(np.int32)
    ids[[7, 2000]] = 5
    x = bits(rng.standard_normal((n, 256)))
    fresh()
    harness.register_models([m2, m3])
    got = harness.run_batch(ids, x, 256)
    assert mt.mt_get_async_status() == (2, 7)
    good = ids < 2
    assert np.isnan(got[~good]).all()
    ref = oracle.forward([m2, m3], ids[good], x[good])
    assert np.isfinite(got[good]).all() and harness.scaled_error(got[good], ref).max() <= TOL


def test_what_a_family_may_mix_and_what_conv_families_keep():
    fresh()
    assert mt.mt_input_elems() == 0 and mt.mt_output_elems() == 0
    assert mt.mt_register_model(synth.make_mlp(11, 0, (64, 128, 10))) == 0
    assert mt.mt_register_model(synth.make_mlp(11, 1, (64, 10))) == 1                  # shallower: accepted
    assert mt.mt_register_model(synth.make_mlp(11, 2, (64, 64, 64, 64, 10))) == 2      # deeper: accepted
    assert (mt.mt_input_elems(), mt.mt_output_elems()) == (64, 10)
    assert mt.mt_register_model(synth.make_mlp(11, 3, (64, 128, 12))) == 3           # a wider output: accepted
    assert (mt.mt_input_elems(), mt.mt_output_elems()) == (64, 12)
    assert mt.mt_register_model(synth.make_mlp(11, 4, (192, 128, 10))) == 4          # a wider input: accepted
    assert (mt.mt_input_elems(), mt.mt_output_elems()) == (192, 12)
    mt.mt_release(4)                                                                 # rows never get shorter
    assert (mt.mt_input_elems(), mt.mt_output_elems()) == (192, 12)
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(synth.make_mlp(11, 5, (100, 128, 10)))                  # not a multiple of 64
    assert e.value.code == 4
    # conv families keep one depth and one input shape
    fresh()
    wl = synth.make_workload(4, n=4, n_tenants=1, h=8, w=8, n_conv=2)
    assert mt.mt_register_model(wl.models[0]) == 0
    deeper = synth.make_workload(4, n=4, n_tenants=1, h=8, w=8, n_conv=3).models[0]
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(deeper)
    assert e.value.code == 3
    larger = synth.make_workload(4, n=4, n_tenants=1, h=16, w=8, n_conv=2).models[0]
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(larger)
    assert e.value.code == 3
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(synth.make_mlp(11, 0, (64 * 8 * 8, 10)))                # an MLP cannot join a conv family
    assert e.value.code == 3


@pytest.mark.parametrize("n", [300, 2500])
def test_tenants_with_different_output_widths(n, small_batch_path):
    # outputs of 10, 64, 200 and 33 columns in one batch: the buffer's rows are as long as the widest output
    # (mt_output_elems), every request gets its own model's columns and the rest of its row is left alone
    outs = [10, 64, 200, 33]
    models = [synth.make_mlp(14, t, (128, 256 if t % 2 else 128, outs[t])) for t in range(4)]
    rng = np.random.default_rng(n)
    ids = rng.integers(0, 4, n).astype(np.int32)
    x = bits(rng.standard_normal((n, 128)))
    fresh()
    harness.register_models(models)
    stride = mt.mt_output_elems()
    assert stride == 200
    out = torch.full((n, stride), -7.0, dtype=torch.float32, device="cuda")
    mt.mt_infer(harness.bf16_bits_to_device(x), torch.from_numpy(ids).cuda(), n, out)
    assert mt.mt_get_async_status() == (0, -1)
    got = out.cpu().numpy()
    for t in range(4):
        rows = np.flatnonzero(ids == t)
        ref = oracle.forward([models[t]], np.zeros(len(rows), np.int32), x[rows])
        assert harness.scaled_error(got[rows, :outs[t]], ref).max() <= TOL
        assert (got[rows, outs[t]:] == -7.0).all()


@pytest.mark.parametrize("n,ins", [(350, [64, 256, 128, 192]), (2500, [128, 512, 64, 320]), (6000, [256, 1024, 64, 576])])
def test_tenants_with_different_input_widths(n, ins, small_batch_path):
    # inputs of four widths in one batch: the buffer's rows are as long as the widest input (mt_input_elems); a request
    # carries its own model's features first, and what follows in its row is never read - the test puts NaN there
    T = len(ins)
    models = [synth.make_mlp(15, t, (ins[t], 256 if t % 2 else 128, 40)) for t in range(T)]
    rng = np.random.default_rng(n)
    ids = synth.zipf_ids(4, n, T, 0.8, salt=n)
    fresh()
    harness.register_models(models)
    stride = mt.mt_input_elems()
    assert stride == max(ins)
    x = rng.standard_normal((n, stride)).astype(np.float32)
    for t in range(T):
        x[ids == t, ins[t]:] = np.nan
    xb = bits(x)
    got = harness.run_batch(ids, xb, 40)
    assert mt.mt_get_async_status() == (0, -1)
    assert np.isfinite(got).all()
    for t in range(T):
        rows = np.flatnonzero(ids == t)
        ref = oracle.forward([models[t]], np.zeros(len(rows), np.int32), np.ascontiguousarray(xb[rows, :ins[t]]))
        assert harness.scaled_error(got[rows], ref).max() <= TOL
    # the same batch through the first layer's TMA gather (rows read through perm) gives the same bits
    mt.mt_debug_set_option("perm_gather", 2)
    try:
        got2 = harness.run_batch(ids, xb, 40)
    finally:
        mt.mt_debug_set_option("perm_gather", 1)
    assert np.array_equal(got, got2)


def test_a_wider_input_registered_between_batches_lengthens_the_rows():
    m0 = synth.make_mlp(16, 0, (128, 256, 16))
    m1 = synth.make_mlp(16, 1, (384, 128, 16))
    rng = np.random.default_rng(3)
    n = 900
    fresh()
    harness.register_models([m0])
    x0 = bits(rng.standard_normal((n, 128)))
    ids0 = np.zeros(n, np.int32)
    first = harness.run_batch(ids0, x0, 16)
    harness.register_models([m1])
    assert mt.mt_input_elems() == 384
    ids = rng.integers(0, 2, n).astype(np.int32)
    x = rng.standard_normal((n, 384)).astype(np.float32)
    x[:, :128] = synth.bf16_bits_to_f32(x0)
    xb = bits(x)
    got = harness.run_batch(ids, xb, 16)
    for t, m, k in ((0, m0, 128), (1, m1, 384)):
        rows = np.flatnonzero(ids == t)
        ref = oracle.forward([m], np.zeros(len(rows), np.int32), np.ascontiguousarray(xb[rows, :k]))
        assert harness.scaled_error(got[rows], ref).max() <= TOL
    rows = np.flatnonzero(ids == 0)
    assert np.array_equal(got[rows], first[rows])      # model 0's requests: same inputs, same bits as before
