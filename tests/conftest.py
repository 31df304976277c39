import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on the B200 box)")


@pytest.fixture(scope="session")
def golden_dir():
    return os.path.join(ROOT, "tests", "golden")


@pytest.fixture(autouse=True, scope="session")
def _selection_kernel_choice():
    """DEFT_SINGLE_PASS=1 / 0 runs the whole GPU suite with the single-pass selection kernel forced on / off,
    DEFT_RING=0 with that kernel reading with plain loads instead of through its ring of bulk copies
    (results must not depend on either choice; the default picks the kernel by call size)."""
    import os
    if os.environ.get("DEFT_SINGLE_PASS") in ("0", "1") or os.environ.get("DEFT_RING") == "0":
        from paper_2307_03500_b200 import build as deft_build
        deft_build.build()
        from paper_2307_03500_b200 import deft
        if os.environ.get("DEFT_SINGLE_PASS") in ("0", "1"):
            deft.deft_debug_select_kernel(os.environ["DEFT_SINGLE_PASS"] == "1")
        if os.environ.get("DEFT_RING") == "0":
            deft.deft_debug_select_ring(False)
    yield
