import os
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent
# tests/test_oracle_mutations.py runs the pins against a (mutated) copy of oracle/ placed elsewhere
_ORACLE_ROOT = os.environ.get("QNN_TEST_ORACLE_ROOT")
if _ORACLE_ROOT:
    sys.path[:] = [p for p in sys.path if p not in ("", _ORACLE_ROOT, str(ROOT))]
    sys.path.insert(0, _ORACLE_ROOT)          # ahead of the working directory, which holds the real oracle/
    sys.path.insert(1, str(ROOT))
elif str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


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


@pytest.fixture(scope="session")
def golden_dir():
    return ROOT / "tests" / "golden"
