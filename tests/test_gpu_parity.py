"""Element-by-element parity of the CUDA path with the fp64 oracle on reduced workloads that still span
several tiles and ragged tails, plus closed forms, edge cases and the properties the paper states
(determinism, no influence between tenants).  Everything goes through the C-ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth
from paper_1901_06887_b200.synth import CONV3X3, DENSE, GLOBAL_AVG_POOL, Layer

from gpu_util import TOL, fresh, run_and_check

pytestmark = pytest.mark.gpu


def bits(a):
    return synth.f32_to_bf16_bits(np.asarray(a, np.float32))


def test_config1_full(small_batch_path):
    wl = synth.make_workload(1)
    run_and_check(wl.models, wl.model_ids, wl.inputs)


def test_identity_and_zero_weights_are_exact_on_the_gpu(small_batch_path):
    rng = np.random.default_rng(0)
    eye = np.eye(256, dtype=np.float32)
    ident = [Layer(DENSE, 256, 256, relu=1, weight=bits(eye), bias=None),
             Layer(DENSE, 256, 256, relu=1, weight=bits(eye), bias=None),
             Layer(DENSE, 256, 10, relu=0, weight=bits(eye[:10]), bias=None)]
    b = [rng.standard_normal(256).astype(np.float32), rng.standard_normal(256).astype(np.float32),
         rng.standard_normal(10).astype(np.float32)]
    zero = [Layer(DENSE, 256, 256, relu=1, weight=bits(np.zeros((256, 256))), bias=b[0]),
            Layer(DENSE, 256, 256, relu=1, weight=bits(np.zeros((256, 256))), bias=b[1]),
            Layer(DENSE, 256, 10, relu=0, weight=bits(np.zeros((10, 256))), bias=b[2])]
    x = bits(rng.standard_normal((300, 256)))
    ids = (np.arange(300) % 2).astype(np.int32)
    got, _ = run_and_check([ident, zero], ids, x)
    xf = synth.bf16_bits_to_f32(x)
    assert np.array_equal(got[ids == 0], np.maximum(xf[ids == 0], 0)[:, :10])   # closed form, bit for bit
    assert np.array_equal(got[ids == 1], np.tile(b[2], (150, 1)))


@pytest.mark.parametrize("n", [1, 2, 127, 128, 129, 385])
def test_ragged_row_tiles_single_tenant(n, small_batch_path):
    rng = np.random.default_rng(n)
    m = synth.make_mlp(1, n, (128, 192, 130))       # He-uniform weights, as in the workloads
    run_and_check([m], np.zeros(n, np.int32), bits(rng.standard_normal((n, 128))))


@pytest.mark.parametrize("K,N", [(64, 1), (64, 10), (64, 128), (128, 129), (320, 257), (1024, 96)])
def test_one_layer_shapes(K, N, small_batch_path):
    rng = np.random.default_rng(K + N)
    models = [synth.make_mlp(1, 10 * K + t, (K, N)) for t in range(3)]
    for t, m in enumerate(models):
        m[0].relu = t % 2
    n = 300
    ids = rng.integers(0, 3, n).astype(np.int32)
    run_and_check(models, ids, bits(rng.standard_normal((n, K))))


def test_config2_reduced():
    wl = synth.make_workload(2, n=900, n_tenants=7, widths=(1024, 512, 640, 256))
    run_and_check(wl.models, wl.model_ids, wl.inputs)


def test_config3_reduced_heterogeneous_widths_and_empty_tenants():
    wl = synth.make_workload(3, n=1500, n_tenants=120)
    assert (np.bincount(wl.model_ids, minlength=120) == 0).any()        # some tenants get no request
    run_and_check(wl.models, wl.model_ids, wl.inputs, max_models=128)


def test_config5_reduced():
    wl = synth.make_workload(5, n=1100, n_tenants=3, widths=(512, 2048, 512))
    run_and_check(wl.models, wl.model_ids, wl.inputs)


@pytest.mark.parametrize("n,tenants,widths", [(2500, 2, (256, 512, 256)), (3100, 3, (128, 768, 10)), (1024, 1, (64, 256, 256))])
def test_cta_pair_executor(n, tenants, widths, monkeypatch):
    # >= 1024 requests per tenant on average and layers >= 256 wide: the 256 x 256 CTA-pair executor runs those
    # layers (ragged last row tiles, tiles whose second half is empty, bf16 and fp32 outputs, the last layer writing
    # arrival order); MT_PAIR=0 sends the same batch to the one-CTA executor, whose result must be equal bit for bit
    # (same products, same accumulation order per output)
    wl = synth.make_workload(5, n=n, n_tenants=tenants, widths=widths)
    got_pair, _ = run_and_check(wl.models, wl.model_ids, wl.inputs)
    monkeypatch.setenv("MT_PAIR", "0")
    got_one, _ = run_and_check(wl.models, wl.model_ids, wl.inputs)
    assert np.array_equal(got_pair, got_one)


def test_cta_pair_executor_rejected_ids_and_unaligned_output():
    wl = synth.make_workload(5, n=2300, n_tenants=2, widths=(128, 256, 260))
    ids = wl.model_ids.copy()
    ids[[5, 900, 2299]] = 7                                   # never issued
    fresh()
    harness.register_models(wl.models)
    buf = torch.full((2300 * 260 + 1,), float("nan"), dtype=torch.float32, device="cuda")
    out = buf[1:].view(2300, 260)                            # 4-byte aligned only
    mt.mt_infer(harness.bf16_bits_to_device(wl.inputs), torch.from_numpy(ids).cuda(), 2300, out)
    assert mt.mt_get_async_status() == (2, 5)
    got = out.cpu().numpy()
    good = ids < 2
    assert np.isnan(got[~good]).all()
    ref = oracle.forward(wl.models, ids[good], wl.inputs[good])
    assert harness.scaled_error(got[good], ref).max() <= TOL


@pytest.mark.parametrize("h,w", [(8, 8), (5, 7), (56, 56), (3, 126), (17, 20)])
def test_config4_reduced_geometries(h, w, conv_path):
    wl = synth.make_workload(4, n=7, n_tenants=3, h=h, w=w, n_conv=2)
    run_and_check(wl.models, wl.model_ids, wl.inputs)


@pytest.mark.parametrize("h,w,n,tenants", [(56, 56, 40, 5), (37, 40, 30, 4), (10, 33, 200, 3)])
def test_conv_many_strips_per_cta(h, w, n, tenants, conv_path):
    # enough images that every CTA walks several strips: tap pairing across strip borders, the ring of TMEM
    # accumulators wrapping around, tenant changes (weight reloads) inside a CTA's range, ragged last strips
    wl = synth.make_workload(4, n=n, n_tenants=tenants, h=h, w=w, n_conv=3)
    run_and_check(wl.models, wl.model_ids, wl.inputs)


@pytest.mark.parametrize("h,w,n,tenants", [(1, 62, 9, 2), (2, 31, 11, 3), (57, 56, 37, 3), (3, 33, 300, 2), (112, 40, 24, 2)])
def test_conv_row_block_ring_edges(h, w, n, tenants, conv_path):
    # padded rows of 64 pixels (the CTA-pair executor's geometry; the one-CTA path runs the same cases): images of one
    # and of an odd number of rows (a last block that is all padding), the widest and the narrowest image of that
    # geometry, tenants with an odd number of images, and CTAs that walk through far more than eight two-row blocks
    # (the shared-memory ring wraps several times, within an image and across images and tenants)
    wl = synth.make_workload(4, n=n, n_tenants=tenants, h=h, w=w, n_conv=2)
    run_and_check(wl.models, wl.model_ids, wl.inputs)


def test_pool_followed_by_head_both_ways(monkeypatch):
    # a global average pool followed by a narrow last dense layer runs as one small launch; MT_POOL_HEAD=0 (and any
    # head wider than 64) takes the pool_finalize + grouped dense path instead: both against the oracle
    wl = synth.make_workload(4, n=23, n_tenants=4, h=12, w=40, n_conv=2)
    got_fused, _ = run_and_check(wl.models, wl.model_ids, wl.inputs)
    monkeypatch.setenv("MT_POOL_HEAD", "0")                    # read by mt_init inside run_and_check
    got_split, _ = run_and_check(wl.models, wl.model_ids, wl.inputs)
    assert np.abs(got_fused - got_split).max() <= 1e-4        # same bf16 pooled values and weights, other summation order
    ids = wl.model_ids.copy(); ids[3] = 9                      # a rejected id on the fused pool + head path
    mt.mt_debug_set_option("pool_head", 1)
    got = harness.run_batch(ids, wl.inputs, 10)
    assert mt.mt_get_async_status() == (2, 3)
    assert np.isnan(got[3]).all() and np.array_equal(np.delete(got, 3, 0), np.delete(got_fused, 3, 0))


@pytest.mark.parametrize("n_out,relu", [(1, 0), (33, 1), (64, 0), (65, 0)])
def test_pool_head_widths(n_out, relu):
    # heads of 1..64 outputs go through the pool + head launch (also with a ReLU on the head), 65 through the
    # pool_finalize + grouped dense path
    rng = np.random.default_rng(n_out)
    H, W = 9, 31
    models = []
    for t in range(3):
        m = synth.make_conv_stack(4, 50 + t, 1, 64, H, W, n_out)
        m[-1].relu = relu
        models.append(m)
    ids = rng.integers(0, 3, 11).astype(np.int32)
    x = bits(rng.standard_normal((11, H * W * 64)))
    run_and_check(models, ids, x)


def test_conv_single_tap_shift_closed_form_on_gpu():
    # tap (ky,kx) with weight 1 on the diagonal: Y = shifted X (zero outside), exact in bf16
    H, W = 6, 9
    rng = np.random.default_rng(5)
    x = rng.integers(0, 5, size=(2, H, W, 64)).astype(np.float32)
    for ky, kx in ((0, 0), (1, 2), (2, 1), (2, 2)):
        wgt = np.zeros((64, 3, 3, 64), np.float32)
        wgt[np.arange(64), ky, kx, np.arange(64)] = 1.0
        head = np.zeros((8, 64), np.float32); head[np.arange(8), np.arange(8)] = 1.0
        m = [Layer(CONV3X3, 64, 64, h=H, w=W, relu=1, weight=bits(wgt), bias=None),
             Layer(GLOBAL_AVG_POOL, 64, 64, h=H, w=W),
             Layer(DENSE, 64, 8, relu=0, weight=bits(head), bias=None)]
        got, _ = run_and_check([m], np.zeros(2, np.int32), bits(x.reshape(2, -1)))
        shifted = np.zeros_like(x)
        ys = slice(max(0, 1 - ky), min(H, H + 1 - ky)); xs = slice(max(0, 1 - kx), min(W, W + 1 - kx))
        ysrc = slice(ys.start + ky - 1, ys.stop + ky - 1); xsrc = slice(xs.start + kx - 1, xs.stop + kx - 1)
        shifted[:, ys, xs, :] = x[:, ysrc, xsrc, :]
        want = shifted.reshape(2, H * W, 64).mean(axis=1)[:, :8]
        assert np.allclose(got, want, rtol=4e-3, atol=0)        # only the pooled mean is rounded to bf16


def test_batch_invariance_and_nan_isolation(small_batch_path):
    wl = synth.make_workload(1, n=48)
    got, _ = run_and_check(wl.models, wl.model_ids, wl.inputs)
    ref = oracle.forward(wl.models, wl.model_ids, wl.inputs)
    # the same request alone, and in another mix / position
    for i in (0, 17, 47):
        alone = harness.run_batch(wl.model_ids[i:i + 1], wl.inputs[i:i + 1], 10)
        assert harness.scaled_error(alone, ref[i:i + 1]).max() <= TOL
        assert np.array_equal(alone[0], got[i])                 # same kernel path here, so also bitwise equal
    order = np.random.default_rng(1).permutation(48)[:31]
    mixed = harness.run_batch(wl.model_ids[order], wl.inputs[order], 10)
    assert np.array_equal(mixed, got[order])
    # NaN weights in another tenant must not leak
    t0 = int(wl.model_ids[0]); other = (t0 + 1) % 4
    mt.mt_release(other)
    poisoned = [Layer(l.kind, l.in_ch, l.out_ch, relu=l.relu, weight=np.full_like(l.weight, 0x7FC0), bias=l.bias)
                for l in wl.models[other]]
    assert mt.mt_register_model(poisoned) == other
    again = harness.run_batch(wl.model_ids, wl.inputs, 10)
    mine = wl.model_ids != other
    assert np.array_equal(again[mine], got[mine])
    assert np.isnan(again[~mine]).all()


def test_repeat_runs_are_bitwise_identical_and_host_entry_matches():
    wl = synth.make_workload(2, n=600, n_tenants=5, widths=(256, 512, 384, 64))
    got, _ = run_and_check(wl.models, wl.model_ids, wl.inputs)
    for _ in range(3):
        assert np.array_equal(harness.run_batch(wl.model_ids, wl.inputs, 64), got)
    x = torch.from_numpy(wl.inputs.view(np.int16)).pin_memory()
    ids = torch.from_numpy(wl.model_ids).pin_memory()
    out = torch.empty((wl.n, 64), dtype=torch.float32).pin_memory()
    mt.mt_infer_host(x, ids, wl.n, out)
    assert np.array_equal(out.numpy(), got)
    # a model re-registered after release gives the same outputs (stateless function of weights and input)
    mt.mt_release(2)
    assert mt.mt_register_model(wl.models[2]) == 2
    assert np.array_equal(harness.run_batch(wl.model_ids, wl.inputs, 64), got)


def test_async_host_entry_on_two_streams_matches_device_entry():
    # five different batches in flight on two alternating streams: every batch's outputs equal mt_infer's, bit for bit
    wl = synth.make_workload(2, n=700, n_tenants=6, widths=(256, 512, 384, 64))
    fresh()
    harness.register_models(wl.models)
    batches = [synth.make_requests(2, wl.models, n=n, salt=50 + k) for k, n in enumerate((700, 300, 700, 650, 1))]
    want = [harness.run_batch(ids, x, 64) for ids, x in batches]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    h_in = [torch.from_numpy(x.view(np.int16)).pin_memory() for _, x in batches]
    h_ids = [torch.from_numpy(ids).pin_memory() for ids, _ in batches]
    h_out = [torch.full((len(ids), 64), float("nan"), dtype=torch.float32).pin_memory() for ids, _ in batches]
    for rep in range(2):
        for k in range(len(batches)):
            mt.mt_infer_host_async(h_in[k], h_ids[k], len(batches[k][0]), h_out[k], streams[k % 2])
        torch.cuda.synchronize()
        assert mt.mt_get_async_status() == (0, -1)
        for k in range(len(batches)):
            assert np.array_equal(h_out[k].numpy(), want[k]), (rep, k)
            h_out[k].fill_(float("nan"))


@pytest.mark.parametrize("family", ["conv", "mlp", "small_mlp"])
def test_different_batches_back_to_back_without_synchronising(family):
    # three different batches enqueued one after the other on one stream, no synchronisation in between (each
    # launch's prologue overlaps its predecessor's tail; workspaces are reused): every batch must match the oracle
    if family == "conv":
        wl = synth.make_workload(4, n=20, n_tenants=4, h=56, w=56, n_conv=2)
        mk = lambda k, n: synth.make_requests(4, wl.models, n=n, salt=70 + k)
        sizes = (20, 9, 20)
    elif family == "mlp":
        wl = synth.make_workload(3, n=900, n_tenants=40)
        mk = lambda k, n: synth.make_requests(3, wl.models, n=n, salt=70 + k)
        sizes = (900, 700, 900)
    else:
        wl = synth.make_workload(1, n=64)
        mk = lambda k, n: synth.make_requests(1, wl.models, n=n, salt=70 + k)
        sizes = (64, 33, 64)
    fresh(max(64, len(wl.models)))
    harness.register_models(wl.models)
    batches = [mk(k, n) for k, n in enumerate(sizes)]
    mt.mt_infer(harness.bf16_bits_to_device(batches[0][1]), torch.from_numpy(batches[0][0]).cuda(), sizes[0],
                torch.empty((sizes[0], wl.out_elems), device="cuda"))      # sizes the workspace
    torch.cuda.synchronize()
    xs = [harness.bf16_bits_to_device(x.reshape(len(i), -1)) for i, x in batches]
    ids = [torch.from_numpy(i).cuda() for i, _ in batches]
    outs = [torch.full((len(i), wl.out_elems), float("nan"), device="cuda") for i, _ in batches]
    for rep in range(3):
        for k in range(3):
            mt.mt_infer(xs[k], ids[k], sizes[k], outs[k])
    torch.cuda.synchronize()
    assert mt.mt_get_async_status() == (0, -1)
    for k, (i, x) in enumerate(batches):
        ref = oracle.forward(wl.models, i, x)
        got = outs[k].cpu().numpy()
        assert np.isfinite(got).all() and harness.scaled_error(got, ref).max() <= TOL, k


def test_growing_batches_and_wider_models_reallocate_correctly(small_batch_path):
    rng = np.random.default_rng(9)
    mk = lambda h: synth.make_mlp(3, h, (128, h, 64))
    fresh()
    models = [mk(128)]
    assert mt.mt_register_model(models[0]) == 0
    for n, add in ((10, None), (300, 256), (50, None), (700, 1024)):
        if add:
            models.append(mk(add))
            assert mt.mt_register_model(models[-1]) == len(models) - 1
        ids = rng.integers(0, len(models), n).astype(np.int32)
        x = bits(rng.standard_normal((n, 128)))
        run_and_check(models, ids, x, register=False)


def test_family_mismatch_is_rejected():
    fresh()
    assert mt.mt_register_model(synth.make_mlp(1, 0, (64, 128, 10))) == 0
    with pytest.raises(mt.MtError) as e:                     # a conv model cannot join an MLP family (widths may differ)
        mt.mt_register_model(synth.make_workload(4, n=4, n_tenants=1, h=8, w=8, n_conv=2).models[0])
    assert e.value.code == 3
    assert mt.mt_register_model(synth.make_mlp(1, 1, (64, 512, 10))) == 1      # hidden width may differ
    with pytest.raises(mt.MtError) as e:
        mt.mt_release(5)
    assert e.value.code == 2


@pytest.mark.parametrize("entry", ["sync", "async"])
def test_host_entries_after_a_wider_family_replaces_a_narrow_one(entry):
    # the host-buffer entry points keep device staging sized for the family's rows: when every model has been released
    # and a family with wider inputs and outputs is registered, a batch of the SAME size must get new staging
    def host_call(models, ids, x, out_elems):
        n = len(ids)
        h_x = torch.from_numpy(x.view(np.int16)).pin_memory()
        h_ids = torch.from_numpy(ids).pin_memory()
        h_out = torch.full((n, out_elems), float("nan"), dtype=torch.float32).pin_memory()
        if entry == "sync":
            mt.mt_infer_host(h_x, h_ids, n, h_out)
        else:
            for _ in range(3):                                   # both staging slots
                mt.mt_infer_host_async(h_x, h_ids, n, h_out)
            torch.cuda.synchronize()
        assert mt.mt_get_async_status() == (0, -1)
        got = h_out.numpy()
        ref = oracle.forward(models, ids, x)
        assert np.isfinite(got).all() and harness.scaled_error(got, ref).max() <= TOL

    rng = np.random.default_rng(21)
    n = 600
    fresh()
    narrow = [synth.make_mlp(2, t, (64, 128, 8)) for t in range(3)]
    ids = harness.register_models(narrow)
    host_call(narrow, rng.integers(0, 3, n).astype(np.int32), bits(rng.standard_normal((n, 64))), 8)
    for i in ids:
        mt.mt_release(i)
    wide = [synth.make_mlp(2, 10 + t, (512, 256, 200)) for t in range(2)]
    assert harness.register_models(wide) == [0, 1]
    host_call(wide, rng.integers(0, 2, n).astype(np.int32), bits(rng.standard_normal((n, 512))), 200)


@pytest.mark.parametrize("mode", ["async", "sync"])
def test_models_registered_while_batches_are_in_flight(mode, monkeypatch):
    # registration does not wait for the device (MT_ASYNC_REGISTER=0: the older path that does): models are added
    # between batches that are still running, the next batch uses them at once, nothing is synchronised in between
    if mode == "sync":
        monkeypatch.setenv("MT_ASYNC_REGISTER", "0")
    models = [synth.make_mlp(13, t, (256, 512, 384, 64)) for t in range(6)]
    rng = np.random.default_rng(31)
    fresh()
    harness.register_models(models[:3])
    n = 900
    batches, outs, keep = [], [], []

    def enqueue(n_live):
        ids = rng.integers(0, n_live, n).astype(np.int32)
        x = bits(rng.standard_normal((n, 256)))
        d_x, d_ids = harness.bf16_bits_to_device(x), torch.from_numpy(ids).cuda()
        out = torch.full((n, 64), float("nan"), dtype=torch.float32, device="cuda")
        mt.mt_infer(d_x, d_ids, n, out)
        batches.append((ids, x)); outs.append(out); keep.append((d_x, d_ids))

    for _ in range(3):
        enqueue(3)
    assert mt.mt_register_model(models[3]) == 3            # while the three batches above are running
    enqueue(4)
    assert harness.register_models(models[4:]) == [4, 5]
    for _ in range(2):
        enqueue(6)
    torch.cuda.synchronize()
    assert mt.mt_get_async_status() == (0, -1)
    for (ids, x), out in zip(batches, outs):
        got = out.cpu().numpy()
        assert np.isfinite(got).all()
        assert harness.scaled_error(got, oracle.forward(models, ids, x)).max() <= TOL


def test_weights_given_as_device_tensors():
    # weights and biases may be device pointers (also unaligned ones): the library reads them on its own stream and the
    # caller may drop them when the call returns
    models = [synth.make_mlp(13, 20 + t, (128, 192, 40)) for t in range(3)]
    fresh()
    for m in models:
        dev_layers = []
        for l in m:
            w = torch.from_numpy(l.weight.view(np.int16).reshape(-1)).cuda()
            pad = torch.empty(w.numel() + 1, dtype=torch.int16, device="cuda")
            pad[1:] = w                                     # 2-byte aligned only
            b = torch.from_numpy(l.bias).cuda()
            dev_layers.append(Layer(l.kind, l.in_ch, l.out_ch, relu=l.relu, weight=pad[1:], bias=b))
        mt.mt_register_model(dev_layers)
        del dev_layers, pad, w, b
        torch.cuda.empty_cache()
    rng = np.random.default_rng(32)
    ids = rng.integers(0, 3, 700).astype(np.int32)
    run_and_check(models, ids, bits(rng.standard_normal((700, 128))), register=False)


@pytest.mark.parametrize("family", ["mlp", "small_mlp", "conv"])
def test_mt_infer_replays_from_a_cuda_graph(family):
    # mt_infer only enqueues work (no allocation, no synchronisation once the workspace exists), so a call can be
    # captured into a CUDA graph - programmatic dependent launches included - and replayed on new inputs in the same
    # buffers: every replay must match the oracle
    if family == "mlp":
        wl = synth.make_workload(3, n=900, n_tenants=40)
        mk = lambda k: synth.make_requests(3, wl.models, n=900, salt=90 + k)
    elif family == "small_mlp":
        wl = synth.make_workload(1, n=64)
        mk = lambda k: synth.make_requests(1, wl.models, n=64, salt=90 + k)
    else:
        wl = synth.make_workload(4, n=12, n_tenants=3, h=56, w=56, n_conv=3)
        mk = lambda k: synth.make_requests(4, wl.models, n=12, salt=90 + k)
    n = wl.n
    fresh(max(64, len(wl.models)))
    harness.register_models(wl.models)
    x = harness.bf16_bits_to_device(wl.inputs.reshape(n, -1)).clone()
    ids = torch.from_numpy(wl.model_ids).cuda()
    out = torch.full((n, wl.out_elems), float("nan"), dtype=torch.float32, device="cuda")
    mt.mt_infer(x, ids, n, out)                       # sizes the workspace, publishes the models' table entries
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph.capture_begin()
        mt.mt_infer(x, ids, n, out, side)
        graph.capture_end()
    torch.cuda.current_stream().wait_stream(side)
    for k in range(3):
        new_ids, new_x = mk(k)
        x.copy_(harness.bf16_bits_to_device(new_x.reshape(n, -1)))
        ids.copy_(torch.from_numpy(new_ids).cuda())
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert mt.mt_get_async_status() == (0, -1)
        got = out.cpu().numpy()
        ref = oracle.forward(wl.models, new_ids, new_x)
        assert np.isfinite(got).all() and harness.scaled_error(got, ref).max() <= TOL, k
