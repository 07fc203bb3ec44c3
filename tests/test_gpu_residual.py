"""Two-layer residual blocks with an identity shortcut in conv families (the building block of resnet18, the network
the paper's Sec. 1.1 uses as its running example): a conv layer marked `residual` adds the INPUT of the conv layer
before it to its pre-activation.  Tenants of one family may differ in which layers carry the shortcut.  Checked
against the per-request oracle on every conv path, and against closed forms."""
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


def family(T, n_conv, h, w, shortcut_sets, n_out=10, config=21):
    return [synth.make_conv_stack(config, t, n_conv, 64, h, w, n_out, shortcuts=shortcut_sets[t % len(shortcut_sets)])
            for t in range(T)]


@pytest.mark.parametrize("h,w,n,T,n_conv", [(12, 40, 23, 4, 4), (9, 62, 14, 3, 2), (57, 56, 11, 3, 4), (7, 20, 40, 5, 6), (5, 100, 9, 2, 3)])
def test_residual_blocks_against_the_oracle(h, w, n, T, n_conv, conv_path):
    # shortcuts whose source is the caller's buffer (layer 1: read through perm), an activation buffer (layer 3, 5), a
    # shortcut on the layer that feeds the pool (stores nothing) and tenants without any; padded rows of 32, 64 and 128
    # pixels (the last two only on the one-CTA executor); odd image counts per tenant
    sets = [(1, 3, 5), (), (1,), (n_conv - 1,), (2,)]
    models = family(T, n_conv, h, w, [tuple(i for i in s if 1 <= i < n_conv) for s in sets])
    assert any(l.residual for m in models for l in m) and any(not any(l.residual for l in m) for m in models[:2])
    ids = synth.zipf_ids(21, n, T, 0.7, salt=h * w)
    x = synth.normal_inputs_bf16(21, n, 64 * h * w, salt=n)
    run_and_check(models, ids, x)


def test_zero_weight_block_returns_the_block_input_plus_bias(conv_path):
    # conv1's weights are zero: a2 = relu(b1 + a0) whatever conv0 does - the shortcut reads the BLOCK'S input, in
    # arrival order (several tenants, so bucketing permutes the images), before the activation.  Then the pool's mean
    # and an identity head return it channel by channel.
    H, W, T, n = 6, 40, 3, 17
    rng = np.random.default_rng(4)
    head = np.zeros((8, 64), np.float32); head[np.arange(8), np.arange(8)] = 1.0
    models, b1s = [], []
    for t in range(T):
        b1 = rng.standard_normal(64).astype(np.float32)
        b1s.append(b1)
        models.append([
            Layer(CONV3X3, 64, 64, h=H, w=W, relu=1, weight=bits(rng.standard_normal((64, 3, 3, 64)) * 0.05), bias=None),
            Layer(CONV3X3, 64, 64, h=H, w=W, relu=1, weight=bits(np.zeros((64, 3, 3, 64))), bias=b1, residual=1),
            Layer(GLOBAL_AVG_POOL, 64, 64, h=H, w=W),
            Layer(DENSE, 64, 8, relu=0, weight=bits(head), bias=None)])
    ids = rng.integers(0, T, n).astype(np.int32)
    xb = bits(rng.standard_normal((n, H * W * 64)))
    got, _ = run_and_check(models, ids, xb)
    a0 = synth.bf16_bits_to_f32(xb).astype(np.float64).reshape(n, H * W, 64)
    for i in range(n):
        want = np.maximum(a0[i] + b1s[ids[i]].astype(np.float64), 0.0).mean(axis=0)[:8]
        assert np.allclose(got[i], want, rtol=5e-3, atol=1e-3)   # the pooled mean is rounded to bf16 for the head


def test_flag_is_per_tenant_and_where_it_is_refused():
    H, W = 8, 40
    plain = synth.make_conv_stack(21, 0, 2, 64, H, W, 10)
    block = synth.make_conv_stack(21, 0, 2, 64, H, W, 10, shortcuts=(1,))     # same weights, with the shortcut
    rng = np.random.default_rng(6)
    n = 10
    xb = bits(rng.standard_normal((n, H * W * 64)))
    ids = (np.arange(n) % 2).astype(np.int32)
    got, _ = run_and_check([plain, block], ids, xb)
    ref_plain = oracle.forward([plain], np.zeros(n, np.int32), xb)
    assert harness.scaled_error(got[ids == 0], ref_plain[ids == 0]).max() <= TOL
    assert np.abs(got[ids == 1] - ref_plain[ids == 1]).max() > 0.05          # the shortcut changes the answer
    # refused: on the family's first layer, on a dense layer
    fresh()
    first = synth.make_conv_stack(21, 1, 2, 64, H, W, 10)
    first[0].residual = 1
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(first)
    assert e.value.code == 4
    mlp = synth.make_mlp(21, 2, (64, 64, 10))
    mlp[1].residual = 1
    with pytest.raises(mt.MtError) as e:
        mt.mt_register_model(mlp)
    assert e.value.code == 4


def test_models_with_shortcuts_come_and_go(conv_path):
    # the executors pick their shortcut form only while a live model has one on that layer: register a plain family,
    # add a model with shortcuts, release it again, bring another in on a different layer - every batch against the oracle
    H, W = 10, 44
    plain = [synth.make_conv_stack(21, t, 3, 64, H, W, 10) for t in range(2)]
    late = synth.make_conv_stack(21, 7, 3, 64, H, W, 10, shortcuts=(2,))
    early = synth.make_conv_stack(21, 8, 3, 64, H, W, 10, shortcuts=(1,))
    rng = np.random.default_rng(9)

    def batch(models_by_id, n=13):
        ids = np.asarray(rng.choice(sorted(models_by_id), size=n), np.int32)
        xb = bits(rng.standard_normal((n, H * W * 64)))
        got = harness.run_batch(ids, xb, 10)
        assert mt.mt_get_async_status() == (0, -1)
        for t, m in models_by_id.items():
            rows = np.flatnonzero(ids == t)
            if len(rows):
                ref = oracle.forward([m], np.zeros(len(rows), np.int32), xb[rows])
                assert harness.scaled_error(got[rows], ref).max() <= TOL

    fresh()
    live = {mt.mt_register_model(m): m for m in plain}
    batch(live)
    t_late = mt.mt_register_model(late)
    live[t_late] = late
    batch(live)
    mt.mt_release(t_late)
    del live[t_late]
    batch(live)
    t_early = mt.mt_register_model(early)
    assert t_early == t_late                      # the slot is reused, with other flags
    live[t_early] = early
    batch(live)
    live[mt.mt_register_model(late)] = late
    batch(live, n=31)


def test_shortcut_from_a_caller_buffer_that_is_only_16_byte_aligned(conv_path):
    # layer 1's shortcut reads the caller's input buffer; mt_infer asks for 16-byte alignment only, and the 32-byte
    # loads of the CTA-pair executor's shortcut path need more: it must fall back to 16-byte loads, same results
    H, W, n = 8, 40, 9
    models = [synth.make_conv_stack(21, t, 2, 64, H, W, 10, shortcuts=(1,)) for t in range(2)]
    rng = np.random.default_rng(12)
    ids = rng.integers(0, 2, n).astype(np.int32)
    xb = bits(rng.standard_normal((n, H * W * 64)))
    fresh()
    harness.register_models(models)
    want = harness.run_batch(ids, xb, 10)
    flat = torch.zeros(xb.size + 8, dtype=torch.int16, device="cuda")
    shifted = flat[8:]                                           # 16 bytes past a 256-byte boundary
    assert shifted.data_ptr() % 32 == 16
    shifted.copy_(torch.from_numpy(xb.view(np.int16).reshape(-1)).cuda())
    out = torch.full((n, 10), float("nan"), dtype=torch.float32, device="cuda")
    mt.mt_infer(shifted, torch.from_numpy(ids).cuda(), n, out)
    assert mt.mt_get_async_status() == (0, -1)
    assert np.array_equal(out.cpu().numpy(), want)
    ref = oracle.forward(models, ids, xb)
    assert harness.scaled_error(want, ref).max() <= TOL
