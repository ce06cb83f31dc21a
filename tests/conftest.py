import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--parity-report", action="store", default=None,
                     help="write the parity figures the GPU tests measured (flip fractions, raw and tie-aware "
                          "cross-covariance errors, objective errors, Procrustes gaps) to this JSON file")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200)")


def pytest_sessionfinish(session, exitstatus):
    path = session.config.getoption("--parity-report")
    if not path:
        return
    import json
    from tests import parity_util
    with open(path, "w") as f:
        json.dump(parity_util.REPORT, f, indent=1)


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if has_gpu:
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


@pytest.fixture(autouse=True)
def workspace_guard_bands(request):
    """Stand-in for a memory checker: every calibration context a GPU test creates gets guard bands behind its
    workspace regions; after the test every context still alive is checked, and so was every context closed during
    the test.  A kernel that writes past its region fails the test that ran it."""
    if "gpu" not in request.keywords:
        yield
        return
    from paper_2605_10793_b200 import binding
    binding.DEBUG_CANARIES = True
    del binding.CANARY_FAILURES[:]
    yield
    import gc
    gc.collect()
    damaged = list(binding.CANARY_FAILURES)
    for ctx in list(binding._live_contexts or ()):
        if getattr(ctx, "h", None):
            bad = ctx.check_canaries()
            if bad:
                damaged.append((ctx.d, ctx.batch, ctx.mode, bad))
    binding.DEBUG_CANARIES = False
    assert not damaged, f"workspace guard bands overwritten (d, batch, mode, bands): {damaged}"
