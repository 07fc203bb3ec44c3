"""Pins for the fp64 oracle: closed forms, brute force and library routines that do not go through
the oracle's own formulas.  A dropped term, wrong sign/index or transposed operand in the oracle
fails at least one of these.  CPU only."""
import numpy as np
import pytest
import torch
from scipy.signal import correlate2d

from paper_1901_06887_b200 import synth
from paper_1901_06887_b200.synth import CONV3X3, DENSE, GLOBAL_AVG_POOL, Layer


def bits(x):
    """Values exactly representable in bf16 -> bit patterns (asserts exactness)."""
    b = synth.f32_to_bf16_bits(np.asarray(x, np.float32))
    assert np.array_equal(synth.bf16_bits_to_f32(b), np.asarray(x, np.float32))
    return b


def rand_bits(rng, shape, scale=1.0):
    return synth.f32_to_bf16_bits((rng.standard_normal(shape) * scale).astype(np.float32))


def f64(b):
    return synth.bf16_bits_to_f32(b).astype(np.float64)


# ----------------------------------------------------------------- bf16 decode / generator rounding
def test_bf16_decode_and_rne_against_torch():
    rng = np.random.default_rng(0)
    x = rng.standard_normal(4096).astype(np.float32) * 37.0
    x[:6] = [1.0, 1.00390625, 1.01171875, -1.00390625, 3.0e-39, 65504.0]  # ties to even both ways, subnormal
    b = synth.f32_to_bf16_bits(x)
    tb = torch.from_numpy(x).to(torch.bfloat16)
    assert np.array_equal(b.view(np.int16), tb.view(torch.int16).numpy())
    assert np.array_equal(synth.bf16_bits_to_f32(b), tb.to(torch.float32).numpy())


def test_oracle_reads_bf16_bits_exactly(oracle_mod):
    # 1-layer identity model returns the decoded input: pins the oracle's own bf16 decode.
    rng = np.random.default_rng(1)
    xb = rand_bits(rng, (64,), 5.0)
    layer = Layer(DENSE, 64, 64, relu=0, weight=bits(np.eye(64)), bias=None)
    out = oracle_mod.forward_one([layer], xb)
    want = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(out, want)


# ----------------------------------------------------------------- dense
def test_dense_identity_chain_closed_form(oracle_mod):
    # W = first rows of I, b = 0, ReLU between layers, none at the end: out = max(x,0)[:10]
    rng = np.random.default_rng(2)
    xb = rand_bits(rng, (256,))
    eye = np.eye(256, dtype=np.float32)
    model = [Layer(DENSE, 256, 256, relu=1, weight=bits(eye), bias=np.zeros(256, np.float32)),
             Layer(DENSE, 256, 256, relu=1, weight=bits(eye), bias=np.zeros(256, np.float32)),
             Layer(DENSE, 256, 10, relu=0, weight=bits(eye[:10]), bias=np.zeros(10, np.float32))]
    out = oracle_mod.forward_one(model, xb)
    assert np.array_equal(out, np.maximum(f64(xb), 0.0)[:10])


def test_dense_zero_weights_closed_form(oracle_mod):
    # zero weights: hidden = ReLU(b_l); out = b_last exactly (no ReLU on the output layer)
    rng = np.random.default_rng(3)
    b1 = rng.standard_normal(32).astype(np.float32)
    b2 = rng.standard_normal(10).astype(np.float32)
    model = [Layer(DENSE, 16, 32, relu=1, weight=bits(np.zeros((32, 16))), bias=b1),
             Layer(DENSE, 32, 10, relu=0, weight=bits(np.zeros((10, 32))), bias=b2)]
    out = oracle_mod.forward_one(model, rand_bits(rng, (16,)))
    assert np.array_equal(out, b2.astype(np.float64))
    assert (b1 < 0).any() and (out < 0).any()                   # ReLU really skipped on the output
    # second layer sums ReLU(b1): W2 = ones -> out = sum(max(b1,0)) + b2
    model[1] = Layer(DENSE, 32, 10, relu=0, weight=bits(np.ones((10, 32))), bias=b2)
    out = oracle_mod.forward_one(model, rand_bits(rng, (16,)))
    want = np.maximum(b1.astype(np.float64), 0).sum() + b2.astype(np.float64)
    assert np.allclose(out, want, rtol=0, atol=1e-12)


def test_dense_one_hot_selects_weight_column(oracle_mod):
    rng = np.random.default_rng(4)
    K, N = 24, 7
    wb = rand_bits(rng, (N, K)); b = rng.standard_normal(N).astype(np.float32)
    for k in (0, 5, K - 1):
        x = np.zeros(K, np.float32); x[k] = 2.0
        out = oracle_mod.forward_one([Layer(DENSE, K, N, relu=0, weight=wb, bias=b)], bits(x))
        assert np.allclose(out, 2.0 * f64(wb)[:, k] + b, rtol=0, atol=1e-14)


def naive_matmul_abT(A, B):
    """C = A . B^T by three nested loops over the whole batch (i, j, k ascending)."""
    M, K = A.shape; N = B.shape[0]
    C = [[0.0] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            s = 0.0
            for k in range(K):
                s += float(A[i, k]) * float(B[j, k])
            C[i][j] = s
    return np.array(C, np.float64)


def test_single_tenant_vs_triple_loop_and_numpy(oracle_mod):
    rng = np.random.default_rng(5)
    n, K, N = 9, 40, 13     # non-square on purpose: a transposed operand cannot pass
    xb = rand_bits(rng, (n, K)); wb = rand_bits(rng, (N, K))
    model = [Layer(DENSE, K, N, relu=0, weight=wb, bias=np.zeros(N, np.float32))]
    out = oracle_mod.forward([model], np.zeros(n, np.int32), xb)
    ref = naive_matmul_abT(f64(xb), f64(wb))
    assert np.allclose(out, ref, rtol=1e-12, atol=1e-12)
    assert np.allclose(out, f64(xb) @ f64(wb).T, rtol=1e-10, atol=1e-10)


def test_mlp_vs_numpy_float64(oracle_mod):
    rng = np.random.default_rng(6)
    widths = (48, 80, 33, 10)
    model = []
    for li in range(3):
        model.append(Layer(DENSE, widths[li], widths[li + 1], relu=int(li < 2),
                           weight=rand_bits(rng, (widths[li + 1], widths[li]), 0.3),
                           bias=rng.standard_normal(widths[li + 1]).astype(np.float32)))
    xb = rand_bits(rng, (5, 48))
    out = oracle_mod.forward([model], np.zeros(5, np.int32), xb)
    a = f64(xb)
    for l in model:
        a = a @ f64(l.weight).T + l.bias.astype(np.float64)
        if l.relu:
            a = np.maximum(a, 0.0)
    assert np.allclose(out, a, rtol=1e-10, atol=1e-10)
    assert (out < 0).any()


# ----------------------------------------------------------------- conv
def conv_layer(w_f32, bias, h, w, relu):
    o, _, _, c = w_f32.shape
    return Layer(CONV3X3, c, o, h=h, w=w, relu=relu, weight=synth.f32_to_bf16_bits(w_f32.astype(np.float32)),
                 bias=None if bias is None else bias.astype(np.float32))


def brute_conv(x, w, b):
    """Independent route: materialise a zero-padded copy, then loop 7 deep."""
    H, W, C = x.shape; O = w.shape[0]
    xp = np.zeros((H + 2, W + 2, C), np.float64)
    xp[1:H + 1, 1:W + 1, :] = x
    y = np.zeros((H, W, O), np.float64)
    for yy in range(H):
        for xx in range(W):
            for o in range(O):
                s = float(b[o])
                for ky in range(3):
                    for kx in range(3):
                        for c in range(C):
                            s += w[o, ky, kx, c] * xp[yy + ky, xx + kx, c]
                y[yy, xx, o] = s
    return y


def test_conv_centre_tap_identity(oracle_mod):
    rng = np.random.default_rng(7)
    H, W, C = 5, 6, 4
    w = np.zeros((C, 3, 3, C)); w[np.arange(C), 1, 1, np.arange(C)] = 1.0
    xb = rand_bits(rng, (H * W * C,))
    out = oracle_mod.forward_one([conv_layer(w, None, H, W, 1)], xb)
    assert np.array_equal(out, np.maximum(f64(xb), 0.0))


@pytest.mark.parametrize("ky,kx", [(a, b) for a in range(3) for b in range(3)])
def test_conv_single_tap_is_a_shift(oracle_mod, ky, kx):
    # one tap (ky,kx) on channel 1 -> output channel 0: Y[y,x,0] = X[y+ky-1, x+kx-1, 1], zero outside
    rng = np.random.default_rng(8)
    H, W, C, O = 4, 5, 3, 2       # H != W, C != O: swapped axes cannot pass
    w = np.zeros((O, 3, 3, C)); w[0, ky, kx, 1] = 1.0
    xb = rand_bits(rng, (H, W, C))
    out = oracle_mod.forward_one([conv_layer(w, None, H, W, 0)], xb.reshape(-1)).reshape(H, W, O)
    x = f64(xb)
    want = np.zeros((H, W))
    for y in range(H):
        for xx in range(W):
            ys, xs = y + ky - 1, xx + kx - 1
            if 0 <= ys < H and 0 <= xs < W:
                want[y, xx] = x[ys, xs, 1]
    assert np.array_equal(out[:, :, 0], want)
    assert np.array_equal(out[:, :, 1], np.zeros((H, W)))


def test_conv_all_ones_counts_padding(oracle_mod):
    H, W, c = 4, 6, 3.0
    w = np.ones((1, 3, 3, 1))
    out = oracle_mod.forward_one([conv_layer(w, None, H, W, 0)], bits(np.full(H * W, c))).reshape(H, W)
    want = np.full((H, W), 9 * c); want[0, :] = want[-1, :] = want[:, 0] = want[:, -1] = 6 * c
    want[0, 0] = want[0, -1] = want[-1, 0] = want[-1, -1] = 4 * c
    assert np.array_equal(out, want)


@pytest.mark.parametrize("H,W,C,O", [(5, 5, 2, 3), (1, 1, 3, 2), (2, 3, 1, 1), (3, 2, 4, 5)])
def test_conv_vs_brute_force_and_scipy(oracle_mod, H, W, C, O):
    rng = np.random.default_rng(9)
    wb = rand_bits(rng, (O, 3, 3, C), 0.5); b = rng.standard_normal(O).astype(np.float32)
    xb = rand_bits(rng, (H, W, C))
    layer = Layer(CONV3X3, C, O, h=H, w=W, relu=0, weight=wb, bias=b)
    out = oracle_mod.forward_one([layer], xb.reshape(-1)).reshape(H, W, O)
    assert np.allclose(out, brute_conv(f64(xb), f64(wb), b), rtol=1e-12, atol=1e-12)
    x, w = f64(xb), f64(wb)
    lib = np.zeros((H, W, O))
    for o in range(O):
        lib[:, :, o] = b[o] + sum(correlate2d(x[:, :, c], w[o, :, :, c], mode="same", boundary="fill", fillvalue=0.0)
                                  for c in range(C))
    assert np.allclose(out, lib, rtol=1e-10, atol=1e-10)


def test_conv_via_im2col_and_triple_loop(oracle_mod):
    rng = np.random.default_rng(10)
    H, W, C, O = 3, 4, 2, 3
    wb = rand_bits(rng, (O, 3, 3, C)); xb = rand_bits(rng, (H, W, C))
    out = oracle_mod.forward_one([Layer(CONV3X3, C, O, h=H, w=W, relu=0, weight=wb, bias=None)], xb.reshape(-1))
    x = f64(xb)
    cols = np.zeros((H * W, 9 * C))
    for y in range(H):
        for xx in range(W):
            for ky in range(3):
                for kx in range(3):
                    ys, xs = y + ky - 1, xx + kx - 1
                    if 0 <= ys < H and 0 <= xs < W:
                        cols[y * W + xx, (ky * 3 + kx) * C:(ky * 3 + kx + 1) * C] = x[ys, xs]
    ref = naive_matmul_abT(cols, f64(wb).reshape(O, 9 * C))
    assert np.allclose(out.reshape(H * W, O), ref, rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------- pointwise conv
def test_conv1x1_is_the_dense_layer_at_every_pixel_and_the_centre_tap_of_a_3x3(oracle_mod):
    rng = np.random.default_rng(31)
    H, W, C, O = 3, 5, 4, 6            # H != W, C != O
    wb = rand_bits(rng, (O, C), 0.5); b = rng.standard_normal(O).astype(np.float32)
    xb = rand_bits(rng, (H * W, C))
    pw = Layer(synth.CONV1X1, C, O, h=H, w=W, relu=1, weight=wb, bias=b)
    out = oracle_mod.forward_one([pw], xb.reshape(-1)).reshape(H * W, O)
    # (a) the dense layer, one pixel at a time
    dense = Layer(DENSE, C, O, relu=1, weight=wb, bias=b)
    for p in range(H * W):
        assert np.array_equal(out[p], oracle_mod.forward_one([dense], xb[p]))
    # (b) numpy in float64
    assert np.allclose(out, np.maximum(f64(xb) @ f64(wb).T + b, 0.0), rtol=1e-12, atol=1e-12)
    # (c) a 3x3 conv whose only non-zero tap is the centre one
    w3 = np.zeros((O, 3, 3, C), np.float32); w3[:, 1, 1, :] = synth.bf16_bits_to_f32(wb).reshape(O, C)
    c3 = Layer(CONV3X3, C, O, h=H, w=W, relu=1, weight=synth.f32_to_bf16_bits(w3), bias=b)
    assert np.array_equal(out.reshape(-1), oracle_mod.forward_one([c3], xb.reshape(-1)))
    # and inside a chain: 3x3 -> 1x1 -> 1x1 -> pool -> dense against numpy
    l0 = Layer(CONV3X3, C, C, h=H, w=W, relu=1, weight=rand_bits(rng, (C, 3, 3, C), 0.5), bias=None)
    l2 = Layer(synth.CONV1X1, O, 2, h=H, w=W, relu=0, weight=rand_bits(rng, (2, O)), bias=None)
    head = Layer(DENSE, 2, 3, relu=0, weight=rand_bits(rng, (3, 2)), bias=rng.standard_normal(3).astype(np.float32))
    full = oracle_mod.forward_one([l0, pw, l2, Layer(GLOBAL_AVG_POOL, 2, 2, h=H, w=W), head], xb.reshape(-1))
    a = np.maximum(brute_conv(f64(xb).reshape(H, W, C), f64(l0.weight), np.zeros(C)), 0.0).reshape(H * W, C)
    a = np.maximum(a @ f64(wb).T + b, 0.0) @ f64(l2.weight).T
    assert np.allclose(full, f64(head.weight) @ a.mean(axis=0) + head.bias, rtol=1e-10, atol=1e-10)


# ----------------------------------------------------------------- identity shortcut (two-layer residual block)
def test_shortcut_with_zero_weights_is_a_closed_form_of_the_block_input(oracle_mod):
    # block: a1 = relu(conv0(a0)); a2 = relu(conv1(a1) + b1 + a0).  With conv1's weights zero, a2 = relu(b1 + a0): it
    # depends on the BLOCK'S input alone.  A shortcut that is dropped gives relu(b1); one taken from a1 gives
    # relu(b1 + a1); one added after the activation gives relu(b1) + a0 (a0 has negative values, so that differs too).
    rng = np.random.default_rng(21)
    H, W, C = 4, 5, 3
    b1 = np.array([0.25, -0.5, 1.0], np.float32)
    l0 = Layer(CONV3X3, C, C, h=H, w=W, relu=1, weight=rand_bits(rng, (C, 3, 3, C)), bias=rng.standard_normal(C).astype(np.float32))
    l1 = Layer(CONV3X3, C, C, h=H, w=W, relu=1, weight=bits(np.zeros((C, 3, 3, C))), bias=b1, residual=1)
    xb = rand_bits(rng, (H * W * C,))
    a0 = f64(xb).reshape(H, W, C)
    out = oracle_mod.forward_one([l0, l1], xb).reshape(H, W, C)
    want = np.maximum(a0 + b1.astype(np.float64), 0.0)
    assert np.array_equal(out, want)
    assert (a0 < 0).any() and not np.array_equal(want, np.maximum(b1.astype(np.float64), 0.0) + 0 * a0)
    # without the activation the sum itself comes out
    l1n = Layer(CONV3X3, C, C, h=H, w=W, relu=0, weight=l1.weight, bias=b1, residual=1)
    assert np.array_equal(oracle_mod.forward_one([l0, l1n], xb).reshape(H, W, C), a0 + b1.astype(np.float64))
    # and a layer without the flag ignores the block's input
    l1p = Layer(CONV3X3, C, C, h=H, w=W, relu=1, weight=l1.weight, bias=b1, residual=0)
    assert np.array_equal(oracle_mod.forward_one([l0, l1p], xb).reshape(H, W, C),
                          np.broadcast_to(np.maximum(b1.astype(np.float64), 0.0), (H, W, C)))


def test_shortcut_blocks_vs_scipy(oracle_mod):
    # two blocks in a row, then pool and head; the second block's input is the first block's output
    rng = np.random.default_rng(22)
    H, W, C = 5, 4, 2
    convs = [Layer(CONV3X3, C, C, h=H, w=W, relu=1, weight=rand_bits(rng, (C, 3, 3, C), 0.5),
                   bias=rng.standard_normal(C).astype(np.float32), residual=int(i in (1, 3))) for i in range(4)]
    head = Layer(DENSE, C, 3, relu=0, weight=rand_bits(rng, (3, C)), bias=rng.standard_normal(3).astype(np.float32))
    xb = rand_bits(rng, (H * W * C,))

    def lib_conv(x, l):
        w = f64(l.weight)
        y = np.zeros((H, W, C))
        for o in range(C):
            y[:, :, o] = l.bias[o] + sum(correlate2d(x[:, :, c], w[o, :, :, c], mode="same", boundary="fill", fillvalue=0.0)
                                         for c in range(C))
        return y

    a0 = f64(xb).reshape(H, W, C)
    a1 = np.maximum(lib_conv(a0, convs[0]), 0.0)
    a2 = np.maximum(lib_conv(a1, convs[1]) + a0, 0.0)
    a3 = np.maximum(lib_conv(a2, convs[2]), 0.0)
    a4 = np.maximum(lib_conv(a3, convs[3]) + a2, 0.0)
    out = oracle_mod.forward_one(convs, xb).reshape(H, W, C)
    assert np.allclose(out, a4, rtol=1e-10, atol=1e-10)
    assert not np.allclose(out, np.maximum(lib_conv(a3, convs[3]) + a3, 0.0), atol=1e-3)    # the wrong tensor is far off
    full = oracle_mod.forward_one(convs + [Layer(GLOBAL_AVG_POOL, C, C, h=H, w=W), head], xb)
    assert np.allclose(full, f64(head.weight) @ a4.reshape(H * W, C).mean(axis=0) + head.bias, rtol=1e-10, atol=1e-10)


def test_shortcut_needs_two_conv_layers_of_one_shape(oracle_mod):
    rng = np.random.default_rng(23)
    conv = lambda c, o, res: Layer(CONV3X3, c, o, h=3, w=3, relu=1, weight=rand_bits(rng, (o, 3, 3, c)), bias=None, residual=res)
    xb = rand_bits(rng, (3 * 3 * 2,))
    with pytest.raises(Exception):
        oracle_mod.forward_one([conv(2, 2, 1)], xb)                      # nothing before it
    with pytest.raises(Exception):
        oracle_mod.forward_one([conv(2, 4, 0), conv(4, 4, 1)], xb)       # the block's input has another shape


def test_conv_relu_and_stack_with_pool_and_head(oracle_mod):
    rng = np.random.default_rng(11)
    H, W, C = 4, 3, 2
    layers = [Layer(CONV3X3, C, C, h=H, w=W, relu=1, weight=rand_bits(rng, (C, 3, 3, C)),
                    bias=rng.standard_normal(C).astype(np.float32)) for _ in range(2)]
    layers.append(Layer(GLOBAL_AVG_POOL, C, C, h=H, w=W))
    layers.append(Layer(DENSE, C, 3, relu=0, weight=rand_bits(rng, (3, C)), bias=rng.standard_normal(3).astype(np.float32)))
    xb = rand_bits(rng, (H * W * C,))
    out = oracle_mod.forward_one(layers, xb)
    a = f64(xb).reshape(H, W, C)
    for l in layers[:2]:
        a = np.maximum(brute_conv(a, f64(l.weight), l.bias), 0.0)
    g = a.reshape(H * W, C).mean(axis=0)
    want = f64(layers[3].weight) @ g + layers[3].bias
    assert np.allclose(out, want, rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------- pooling
def test_gap_constant_and_1x1(oracle_mod):
    C = 5
    vals = np.arange(1, C + 1, dtype=np.float32)
    img = np.tile(vals, (3 * 4, 1))
    out = oracle_mod.forward_one([Layer(GLOBAL_AVG_POOL, C, C, h=3, w=4)], bits(img.reshape(-1)))
    assert np.array_equal(out, vals.astype(np.float64))
    out = oracle_mod.forward_one([Layer(GLOBAL_AVG_POOL, C, C, h=1, w=1)], bits(vals))
    assert np.array_equal(out, vals.astype(np.float64))
    # a ramp over positions: mean of 0..11 = 5.5 in channel 0, channel 1 stays 2
    ramp = np.stack([np.arange(12, dtype=np.float32), np.full(12, 2, np.float32)], axis=1)
    out = oracle_mod.forward_one([Layer(GLOBAL_AVG_POOL, 2, 2, h=3, w=4)], bits(ramp.reshape(-1)))
    assert np.array_equal(out, np.array([5.5, 2.0]))


# ----------------------------------------------------------------- bucketing
def brute_bucket(ids, T):
    counts = [sum(1 for v in ids if v == t) for t in range(T)]
    perm = [i for t in range(T) for i, v in enumerate(ids) if v == t]
    offsets = [0]
    for c in counts:
        offsets.append(offsets[-1] + c)
    inv = [0] * len(ids)
    for j, i in enumerate(perm):
        inv[i] = j
    return counts, offsets, perm, inv


@pytest.mark.parametrize("n,T,seed", [(0, 3, 0), (1, 1, 1), (7, 1, 2), (33, 4, 3), (100, 7, 4), (257, 50, 5), (64, 200, 6)])
def test_bucket_vs_brute_force_and_argsort(oracle_mod, n, T, seed):
    rng = np.random.default_rng(seed)
    ids = rng.integers(0, T, n).astype(np.int32)
    counts, offsets, perm, inv = oracle_mod.bucket(ids, T)
    bc, bo, bp, bi = brute_bucket(ids.tolist(), T)
    assert counts.tolist() == bc and offsets.tolist() == bo and perm.tolist() == bp and inv.tolist() == bi
    assert np.array_equal(perm, np.argsort(ids, kind="stable"))
    assert np.array_equal(counts, np.bincount(ids, minlength=T))


def test_bucket_invariants_on_zipf_draws(oracle_mod):
    for cfg, n, T in ((2, 4096, 64), (3, 16384, 1000), (5, 65536, 8)):
        ids = synth.zipf_ids(cfg, n, T, {2: 1.1, 3: 0.9, 5: 0.0}[cfg])
        counts, offsets, perm, inv = oracle_mod.bucket(ids, T)
        assert offsets[0] == 0 and offsets[-1] == n and (np.diff(offsets) == counts).all()
        assert np.array_equal(np.sort(perm), np.arange(n))
        assert (np.diff(ids[perm]) >= 0).all()
        same = ids[perm][1:] == ids[perm][:-1]
        assert (np.diff(perm)[same] > 0).all()                  # stable inside each segment
        assert np.array_equal(inv[perm], np.arange(n))
        assert np.array_equal(perm, np.argsort(ids, kind="stable"))


def test_bucket_rejects_bad_id(oracle_mod):
    with pytest.raises(ValueError):
        oracle_mod.bucket(np.array([0, 3], np.int32), 3)
    with pytest.raises(ValueError):
        oracle_mod.bucket(np.array([-1], np.int32), 3)


# ----------------------------------------------------------------- whole pass
def test_batch_invariance_and_tenant_isolation(oracle_mod):
    wl = synth.make_workload(1, n=40)
    full = oracle_mod.forward(wl.models, wl.model_ids, wl.inputs)
    assert full.shape == (40, 10)
    for i in (0, 7, 39):                                        # alone == in the mix, bit for bit
        alone = oracle_mod.forward_one(wl.models[wl.model_ids[i]], wl.inputs[i])
        assert np.array_equal(alone, full[i])
    order = np.random.default_rng(0).permutation(40)            # another position / another mix
    shuffled = oracle_mod.forward(wl.models, wl.model_ids[order], wl.inputs[order])
    assert np.array_equal(shuffled, full[order])
    # poisoning another tenant's weights does not change this tenant's outputs
    t0 = int(wl.model_ids[0])
    other = (t0 + 1) % len(wl.models)
    models = [list(m) for m in wl.models]
    bad = wl.models[other][0]
    models[other][0] = Layer(bad.kind, bad.in_ch, bad.out_ch, relu=bad.relu,
                             weight=np.full_like(bad.weight, 0x7FC0), bias=bad.bias)   # bf16 NaN
    poisoned = oracle_mod.forward(models, wl.model_ids, wl.inputs)
    mine = wl.model_ids == t0
    assert np.array_equal(poisoned[mine], full[mine])
    assert np.isnan(poisoned[wl.model_ids == other]).all()
    # each request really uses its own tenant's weights: the same input under two tenants differs
    a = oracle_mod.forward_one(wl.models[0], wl.inputs[0]); b = oracle_mod.forward_one(wl.models[1], wl.inputs[0])
    assert not np.allclose(a, b)


def test_threads_do_not_change_results(oracle_mod):
    wl = synth.make_workload(1)
    a = oracle_mod.forward(wl.models, wl.model_ids, wl.inputs, n_threads=1)
    b = oracle_mod.forward(wl.models, wl.model_ids, wl.inputs, n_threads=4)
    assert np.array_equal(a, b)


def test_conv_workload_reduced_vs_numpy(oracle_mod):
    wl = synth.make_workload(4, n=6, n_tenants=3, h=6, w=5, ch=8, n_conv=2)
    out = oracle_mod.forward(wl.models, wl.model_ids, wl.inputs)
    for i in range(wl.n):
        m = wl.models[wl.model_ids[i]]
        a = f64(wl.inputs[i]).reshape(6, 5, 8)
        for l in m[:2]:
            a = np.maximum(brute_conv(a, f64(l.weight), l.bias), 0.0)
        g = a.reshape(30, 8).mean(axis=0)
        want = f64(m[3].weight) @ g + m[3].bias
        assert np.allclose(out[i], want, rtol=1e-11, atol=1e-12)
