import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200)")


def pytest_collection_modifyitems(config, items):
    import torch

    if torch.cuda.is_available():
        return
    skip = pytest.mark.skip(reason="no CUDA device")
    for item in items:
        if "gpu" in item.keywords:
            item.add_marker(skip)


# The decode entry points pick one of two kernels by problem size (a cluster per (sequence, KV head) for small
# batches, the split kernel otherwise). The decode parity modules run once with the library's own choice and
# once with every call kept on the split kernel, so that small test shapes cover both.
_DECODE_MODULES = {"test_gpu_decode", "test_gpu_decode_append", "test_gpu_paged", "test_gpu_random_shapes",
                   "test_gpu_cuda_graph", "test_gpu_rope_append", "test_gpu_fp8"}


def pytest_generate_tests(metafunc):
    if metafunc.module.__name__.split(".")[-1] in _DECODE_MODULES:
        if "decode_kernel_choice" not in metafunc.fixturenames:
            metafunc.fixturenames.append("decode_kernel_choice")
        metafunc.parametrize("decode_kernel_choice", ["auto", "split"], indirect=True)


@pytest.fixture
def decode_kernel_choice(request):
    mode = getattr(request, "param", "auto")
    old = os.environ.get("L4L_DECODE_CLUSTER")
    if mode == "split":
        os.environ["L4L_DECODE_CLUSTER"] = "0"
    else:
        os.environ.pop("L4L_DECODE_CLUSTER", None)
    yield mode
    if old is None:
        os.environ.pop("L4L_DECODE_CLUSTER", None)
    else:
        os.environ["L4L_DECODE_CLUSTER"] = old
