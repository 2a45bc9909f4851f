import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")
    config.addinivalue_line("markers", "fullp: compares EVERY coordinate of a full-size workload with the oracle "
                                       "(minutes of CPU time each); runs only when asked for with -m fullp")
    # The oracle front end loads whatever SLOWMO_ORACLE_LIB names; only the mutation tests, which
    # check that planted mistakes are noticed, may use that. A stray variable would silently swap
    # the checker under every other test.
    if os.environ.get("SLOWMO_ORACLE_LIB") and os.environ.get("SLOWMO_ORACLE_MUTATION_RUN") != "1":
        raise pytest.UsageError("SLOWMO_ORACLE_LIB is set: the tests would check against a substitute oracle; "
                                "unset it (only tests/test_oracle_mutations.py sets it, for its own subprocesses)")


def pytest_collection_modifyitems(config, items):
    mutation_run = os.environ.get("SLOWMO_ORACLE_MUTATION_RUN") == "1"
    wants_fullp = "fullp" in (config.getoption("-m") or "")
    for item in items:
        if mutation_run and "gpu" in item.keywords:
            item.add_marker(pytest.mark.skip(reason="a substitute oracle never checks the GPU"))
        if "fullp" in item.keywords and not wants_fullp:
            item.add_marker(pytest.mark.skip(reason="full-coverage run: select with -m fullp"))
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
