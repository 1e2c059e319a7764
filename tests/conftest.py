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


# ---- measured error ratios of the full-size parity tests, written where a GPU run's artefacts go ----
_ERRORS = {}


def record_error(name, err_over_tensor_rms, err_over_row_rms):
    """max |err| / RMS(reference tensor) and the worst row's max |err| / RMS(that row), for the record."""
    _ERRORS[name] = {"max_err_over_tensor_rms": err_over_tensor_rms, "max_err_over_row_rms": err_over_row_rms}


def pytest_sessionfinish(session, exitstatus):
    if not _ERRORS:
        return
    import json
    out = os.environ.get("DASH_TEST_RECORD_DIR", os.path.join(ROOT, "test_records"))      # where the session's record goes
    try:
        os.makedirs(out, exist_ok=True)
        with open(os.path.join(out, "parity_errors.json"), "w") as f:
            json.dump(_ERRORS, f, indent=1, sort_keys=True)
    except OSError:
        pass
