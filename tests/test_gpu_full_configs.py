"""The five workloads at full size, in the launch configuration the bench times, checked on sampled
requests the oracle computes one by one (all outputs of each sampled request), plus properties that hold
at any size: bucketing bit-exact in full, outputs finite, repeat run bitwise identical."""
import numpy as np
import pytest

from paper_1901_06887_b200 import binding as mt, harness, synth

from gpu_util import run_and_check, stratified_sample

pytestmark = pytest.mark.gpu


def full(config, per_tenant, max_models=64):
    wl = synth.make_workload(config)
    sample = stratified_sample(wl.model_ids, len(wl.models), per_tenant)
    got, err = run_and_check(wl.models, wl.model_ids, wl.inputs, sample=sample, max_models=max_models)
    again = harness.run_batch(wl.model_ids, wl.inputs, wl.out_elems)
    assert np.array_equal(again, got)
    print("config %d: %d sampled requests, max scaled error %.3e" % (config, len(sample), err))
    mt.mt_shutdown()


def test_config2_full():
    full(2, 6)


def test_config3_full():
    full(3, 4, max_models=1024)


def test_config4_full(conv_path):
    full(4, 3)


def test_config5_full():
    full(5, 12)
