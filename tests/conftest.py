import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (B200) and the built CUDA library")
    # the C-ABI library and the oracle are built in-tree when missing or stale (nvcc / gcc, no GPU needed)
    from paper_2402_03293_b200 import _build
    from oracle import flora_oracle
    _build.build()
    flora_oracle.build()
