import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (runs the sm_100a library)")


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if not has_gpu:
        skip = pytest.mark.skip(reason="no CUDA device")
        for it in items:
            if "gpu" in it.keywords:
                it.add_marker(skip)


@pytest.fixture(scope="session")
def rec0():
    import pcr_synth
    return pcr_synth.make_record(0)


@pytest.fixture(scope="session")
def rec1_small():
    import pcr_synth
    return pcr_synth.make_record(1, n_images=12)


@pytest.fixture(scope="session")
def rec2_small():
    import pcr_synth
    return pcr_synth.make_record(2, n_images=6)


@pytest.fixture(scope="session")
def rec3_small():
    import pcr_synth
    return pcr_synth.make_record(3, n_images=3)
