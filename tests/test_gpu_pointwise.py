"""Pointwise (1x1) conv layers inside conv families: the fully-connected layer of the paper's Sec. 1.1 applied at
every pixel, run by the grouped dense executor over the pixels of all requests' images (a tenant's segment is its
images x H x W matrix rows).  3x3 layers around a pair of pointwise ones with a tenant-specific middle width, against
the per-request oracle on every conv path, for batches below and above the single-CTA bucketing limit."""
import numpy as np
import pytest

import oracle
from paper_1901_06887_b200 import binding as mt, harness, synth
from paper_1901_06887_b200.synth import CONV1X1, CONV3X3, DENSE, GLOBAL_AVG_POOL, Layer

from gpu_util import TOL, fresh, run_and_check

pytestmark = pytest.mark.gpu

MID = (128, 256, 64, 192, 320)


def family(T, h, w, n_out=10):
    return [synth.make_pointwise_stack(22, t, MID[t % len(MID)], h, w, n_out) for t in range(T)]


@pytest.mark.parametrize("h,w,n,T", [(12, 40, 23, 4), (7, 20, 31, 5), (57, 56, 9, 3), (2, 33, 700, 6), (5, 100, 12, 2)])
def test_pointwise_layers_between_3x3_layers(h, w, n, T, conv_path):
    # middle widths differ per tenant (the buffer between the two pointwise layers is as wide as the widest); padded
    # rows of 32, 64 and 128 pixels; 700 requests take the two-pass bucketing, whose work items count pixels, not requests
    models = family(T, h, w)
    ids = synth.zipf_ids(22, n, T, 0.8, salt=h * w)
    x = synth.normal_inputs_bf16(22, n, 64 * h * w, salt=n)
    run_and_check(models, ids, x)


def test_pointwise_closed_form_identity_and_rejected_ids():
    # identity pointwise layers (64 -> 64, no bias) between the 3x3 layers change nothing: same bits as the family
    # without them; ids that name no model come back as NaN rows
    H, W, n, T = 6, 40, 19, 3
    rng = np.random.default_rng(3)
    eye = synth.f32_to_bf16_bits(np.eye(64, dtype=np.float32))
    plain, with_pw = [], []
    for t in range(T):
        base = synth.make_conv_stack(22, 50 + t, 2, 64, H, W, 10)
        plain.append(base)
        pw = [Layer(CONV1X1, 64, 64, h=H, w=W, relu=1, weight=eye, bias=None) for _ in range(2)]
        with_pw.append([base[0]] + pw + base[1:])
    ids = rng.integers(0, T, n).astype(np.int32)
    xb = synth.f32_to_bf16_bits(rng.standard_normal((n, H * W * 64)).astype(np.float32))
    want, _ = run_and_check(plain, ids, xb)
    got, _ = run_and_check(with_pw, ids, xb)                  # ReLU of a ReLU output, times one: the same values
    assert np.array_equal(got, want)
    ids[[2, 11]] = [T + 1, -3]
    out = harness.run_batch(ids, xb, 10)
    assert mt.mt_get_async_status() == (2, 2)
    good = (ids >= 0) & (ids < T)
    assert np.isnan(out[~good]).all() and np.array_equal(out[good], want[good])


def test_where_a_pointwise_layer_is_refused():
    H, W = 4, 40
    ok = synth.make_pointwise_stack(22, 0, 128, H, W, 10)
    fresh()
    assert mt.mt_register_model(ok) == 0
    rng = np.random.default_rng(1)
    w = lambda o, c: synth.f32_to_bf16_bits(rng.standard_normal((o, c)).astype(np.float32))
    pw = lambda c, o: Layer(CONV1X1, c, o, h=H, w=W, relu=1, weight=w(o, c), bias=None)
    head = Layer(DENSE, 64, 10, relu=0, weight=w(10, 64), bias=None)
    pool = Layer(GLOBAL_AVG_POOL, 64, 64, h=H, w=W)
    for bad in ([pw(64, 64), ok[0], pool, head],                      # first layer: it would have to read through perm
                [ok[0], pw(64, 64), pool, head],                      # the pool is fused into a conv3x3's epilogue only
                [ok[0], pw(64, 100), pw(100, 64), ok[3], pool, head],  # 100 input channels: not a multiple of 64
                [ok[0], pw(64, 64), head]):                            # a dense layer cannot follow a conv
        with pytest.raises(mt.MtError) as e:
            mt.mt_register_model(bad)
        assert e.value.code == 4, bad
    with pytest.raises(mt.MtError) as e:                               # a family keeps its layer kinds index by index
        mt.mt_register_model(synth.make_conv_stack(22, 1, 4, 64, H, W, 10))
    assert e.value.code == 3
