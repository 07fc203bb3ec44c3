import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(scope="session")
def oracle_mod():
    import oracle
    oracle.build()
    return oracle


@pytest.fixture(params=["fused", "layered"])
def small_batch_path(request, monkeypatch):
    """Batches of at most 512 requests against narrow dense models run as one fused launch; MT_FUSED=0 sends the
    same batch down the layer-by-layer path.  Tests that take this fixture run once on each."""
    if request.param == "layered":
        monkeypatch.setenv("MT_FUSED", "0")
    return request.param


@pytest.fixture(params=["pair", "pair_layerwise", "pair_bucketing_launch", "single"])
def conv_path(request, monkeypatch):
    """Conv layers whose padded row length is 64 pixels run on CTA pairs (two images of a tenant per cluster), consecutive
    conv layers as ONE launch with grid-wide barriers in between, and batches of at most 512 requests are bucketed by
    that launch itself; MT_CONV_STACK=0 gives every conv layer a launch of its own, MT_CONV_SELF_BUCKET=0 keeps the
    bucketing launch and MT_CONV_PAIR=0 sends the layers to the one-CTA executor.  Tests that take this fixture run once
    on each."""
    if request.param == "single":
        monkeypatch.setenv("MT_CONV_PAIR", "0")
    elif request.param == "pair_layerwise":
        monkeypatch.setenv("MT_CONV_STACK", "0")
    elif request.param == "pair_bucketing_launch":
        monkeypatch.setenv("MT_CONV_SELF_BUCKET", "0")
    return request.param
