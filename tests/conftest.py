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


@pytest.fixture(scope="session", autouse=True)
def built_libraries():
    """Build the CUDA library and the C oracle once per session if they are missing or stale (a no-op when the
    digest of the sources matches the library on disk).  A failing build is reported by the tests that need it."""
    if os.environ.get("QNN_TEST_ORACLE_ROOT"):
        return                                     # pins running against a mutated oracle copy: nothing else needed
    try:
        from paper_2106_09886_b200 import build
        build.build()
    except Exception as exc:                       # e.g. no nvcc on this machine but a library already present
        print(f"[conftest] libqnn build skipped/failed: {exc}", file=sys.stderr)
    try:
        import oracle
        oracle.build()
    except Exception as exc:
        print(f"[conftest] oracle build failed: {exc}", file=sys.stderr)
