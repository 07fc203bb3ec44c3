"""The C-ABI library loads without a GPU and exports every symbol include/mt.h declares; host-side
validation paths that never touch the device behave as documented.  CPU only (no compute calls)."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1901_06887_b200 import binding as mt, build, synth
from paper_1901_06887_b200.synth import CONV3X3, DENSE, GLOBAL_AVG_POOL, Layer

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_lib()
    return mt.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mt_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert "mt_register_model" in names and "mt_infer" in names and "mt_release" in names
    for name in names:
        assert hasattr(lib, name), name
        assert hasattr(mt, name), "binding lacks " + name
    assert sorted(mt.EXPORTS) == names


def test_status_strings(lib):
    assert mt.mt_status_string(0) == "ok"
    assert len({mt.mt_status_string(c) for c in range(10)}) == 10
    assert mt.mt_status_string(1234) == "unknown status"


def w_bits(shape):
    return np.zeros(shape, np.uint16)


def reg_code(layers):
    try:
        mt.mt_register_model(layers)
    except mt.MtError as e:
        return e.code
    return 0


def test_register_validation_happens_on_the_host(lib):
    # every case below is rejected before any device call, so it is safe without a GPU
    d = lambda k, n, **kw: Layer(DENSE, k, n, weight=w_bits((n, k)), bias=None, **kw)
    assert reg_code([]) == 1                                              # no layers
    assert reg_code([d(64, 8)] * 9) == 4                                  # too many layers
    assert reg_code([Layer(7, 64, 8, weight=w_bits((8, 64)))]) == 1       # unknown kind
    assert reg_code([Layer(DENSE, 64, 8, weight=None)]) == 1              # missing weights
    assert reg_code([d(0, 8)]) == 1                                       # non-positive dim
    assert reg_code([d(100, 8)]) == 4                                     # K not a multiple of 64
    assert reg_code([d(64, 128), d(64, 8)]) == 3                          # chain mismatch
    conv = Layer(CONV3X3, 64, 64, h=8, w=8, relu=1, weight=w_bits((64, 3, 3, 64)))
    pool = Layer(GLOBAL_AVG_POOL, 64, 64, h=8, w=8)
    assert reg_code([conv, d(64, 8)]) == 4                                # dense directly after conv
    assert reg_code([pool, d(64, 8)]) == 4                                # pool first
    assert reg_code([conv, pool]) == 4                                    # last layer must be dense
    assert reg_code([Layer(CONV3X3, 32, 32, h=8, w=8, weight=w_bits((32, 3, 3, 32))), pool, d(32, 8)]) == 4
    assert reg_code([conv, Layer(GLOBAL_AVG_POOL, 64, 64, h=4, w=8), d(64, 8)]) == 3


def test_calls_before_init_fail_cleanly(lib):
    mt.mt_shutdown()
    for fn, args in ((lib.mt_release, (0,)), (lib.mt_infer, (None, None, 4, None, None)),
                     (lib.mt_infer_host, (None, None, 4, None, None)), (lib.mt_infer_host_async, (None, None, 4, None, None)),
                     (lib.mt_get_async_status, (None, None, None)), (lib.mt_debug_wait_timeout, (20, None))):
        assert fn(*args) == 9                                             # MT_ERR_NOT_INIT
    assert mt.mt_debug_launch_count() >= 0                                # a plain counter: no device needed
    assert lib.mt_debug_launch_count(None) == 1                           # MT_ERR_INVALID_ARG


def test_synth_workloads_match_their_descriptions():
    wl = synth.make_workload(1)
    assert wl.n == 64 and len(wl.models) == 4 and wl.in_elems == 256 and wl.out_elems == 10
    assert [l.relu for l in wl.models[0]] == [1, 1, 0]
    w = synth.bf16_bits_to_f32(wl.models[0][0].weight)
    bound = np.sqrt(6.0 / 256)
    assert np.abs(w).max() <= bound * 1.01 and np.abs(w).max() > bound * 0.95 and abs(w.mean()) < 0.01
    assert abs(wl.models[0][0].bias.std() - 0.01) < 0.003
    x = synth.bf16_bits_to_f32(wl.inputs)
    assert abs(x.std() - 1.0) < 0.02
    # same seed -> same draw; another salt -> another draw
    assert np.array_equal(synth.make_workload(1).inputs, wl.inputs)
    assert not np.array_equal(synth.make_workload(1, salt=1).model_ids, wl.model_ids)
    # Zipf: the most popular tenant of config 2 gets about 1 / H_64(1.1) of the requests
    ids = synth.zipf_ids(2, 4096, 64, 1.1)
    top = np.bincount(ids, minlength=64).max() / 4096
    p1 = 1.0 / np.sum(np.arange(1, 65) ** -1.1)
    assert abs(top - p1) < 0.03
    # heterogeneous widths of config 3 come from the stated set
    ms = synth.make_models(3, n_tenants=12)
    assert {m[0].out_ch for m in ms} | {m[1].out_ch for m in ms} <= {128, 256, 512, 1024}
    assert all(m[0].in_ch == 512 and m[2].out_ch == 64 and m[1].in_ch == m[0].out_ch for m in ms)
    # closed-form work counts (Sec. 3.2: flops per layer known a priori)
    assert synth.workload_flops(wl.models, wl.model_ids) == 64 * 2 * (256 * 256 * 2 + 256 * 10)
    c4 = synth.make_models(4, n_tenants=1)
    assert sum(synth.layer_flops(l) for l in c4[0]) == 4 * 2 * 9 * 64 * 64 * 56 * 56 + 2 * 64 * 10
