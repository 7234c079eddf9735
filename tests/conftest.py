import glob
import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_addoption(parser):
    parser.addoption("--full-lengths", action="store_true", default=False,
                     help="run the largest workload's oracle comparison over its whole generation length")


@pytest.fixture
def full_lengths(request):
    return request.config.getoption("--full-lengths")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")
    # native pieces that need no GPU to build: input generator, CPU checker, CUDA library (cross-compiled)
    from paper_2505_18164_b200 import build
    build.build_inputs()
    from oracle import mdi_oracle
    mdi_oracle.build()
    if glob.glob(os.path.join(ROOT, 'paper_2505_18164_b200', 'csrc', '*.cu')):
        build.build_mdi()


def pytest_collection_modifyitems(config, items):
    try:
        import torch
        has_gpu = torch.cuda.is_available()
    except Exception:
        has_gpu = False
    if not has_gpu:
        skip = pytest.mark.skip(reason="no CUDA device")
        for it in items:
            if "gpu" in it.keywords:
                it.add_marker(skip)
