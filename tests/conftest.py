import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


# machine constants used by the planner tests: integers, frozen (sustained bf16 peak, HBM copy
# bandwidth, pinned host-to-device and device-to-host bandwidth at 256 MiB measured on the machine's B200)
MACHINE = dict(peak_flops=1362800000000000, hbm_Bps=6541100000000, h2d_Bps=55570000000, d2h_Bps=56900000000)


@pytest.fixture(scope="session")
def machine():
    return dict(MACHINE)
