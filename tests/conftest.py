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
# (the static-scratch test pins its shapes to the split kernel itself and asserts that choice)


def pytest_generate_tests(metafunc):
    if metafunc.module.__name__.split(".")[-1] in _DECODE_MODULES:
        if "decode_kernel_choice" not in metafunc.fixturenames:
            metafunc.fixturenames.append("decode_kernel_choice")
        metafunc.parametrize("decode_kernel_choice", ["auto", "split"], indirect=True)


@pytest.fixture
def decode_kernel_choice(request):
    from paper_2608_21836_b200 import binding as l4l

    mode = getattr(request, "param", "auto")
    with l4l.decode_override(cluster=0 if mode == "split" else -1):
        yield mode
