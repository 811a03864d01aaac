import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        have = torch.cuda.is_available()
    except Exception:
        have = False
    if have:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for it in items:
        if "gpu" in it.keywords:
            it.add_marker(skip)


@pytest.fixture(scope="session")
def oracle_mod():
    import oracle
    oracle.build()
    return oracle


@pytest.fixture
def tune():
    """tune(key=value, ...) forces launch-shape choices of the library through grass_set_tuning (None restores
    the automatic choice); everything is back on automatic after the test."""
    import paper_2505_18976_b200 as G
    touched = set()

    def set_(**kw):
        for k, v in kw.items():
            G.grass_set_tuning(k, v)
            touched.add(k)
    yield set_
    for k in touched:
        G.grass_set_tuning(k, None)


@pytest.fixture(params=["streaming", "cluster"])
def fg_path(request):
    """Runs a FactGraSS test once on the streaming kernel and once with the cluster kernel forced wherever the
    layers fit it (calls that do not fit fall back to the streaming kernel by themselves)."""
    import paper_2505_18976_b200 as G
    G.grass_set_tuning("factgrass_path", 0 if request.param == "streaming" else 1)
    yield request.param
    G.grass_set_tuning("factgrass_path", None)
