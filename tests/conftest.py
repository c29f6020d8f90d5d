import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a B200 (runs the CUDA library)")


def pytest_collection_modifyitems(config, items):
    """GPU tests are skipped, not failed, where no CUDA device is present."""
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


FWD_SHORT_LEN_DEFAULT = -1        # the library chooses by head layout


@pytest.fixture(params=["cta_pair_forward", "short_sequence_forward"])
def both_forward_kernels(request):
    """Runs a GPU test once with every pair on the CTA-pair forward kernel and once with every pair on the
    short-sequence forward kernel (the library routes by length; the small parity cases would otherwise only
    ever see one of the two)."""
    import paper_2609_34318_b200 as P
    P.hydra_set_fwd_short_len(0 if request.param == "cta_pair_forward" else 1 << 20)
    yield request.param
    P.hydra_set_fwd_short_len(FWD_SHORT_LEN_DEFAULT)
