import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200); run with -m gpu")


@pytest.fixture(autouse=True, scope="session")
def _prefill_arrangement():
    """MPFA_TEST_ARRANGEMENT=1 runs the whole GPU suite on the two-query-tile arrangement of the prefill kernel
    (the default arrangement needs nothing; a few tests select arrangement 1 themselves)."""
    a = os.environ.get("MPFA_TEST_ARRANGEMENT")
    if a is not None:
        from paper_2609_33135_b200 import binding
        binding.mpfa_set_prefill_arrangement(int(a))
    yield


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:  # pragma: no cover
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)
