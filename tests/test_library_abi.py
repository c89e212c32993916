"""CPU-side checks of the boundary: the library builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before anything could be launched."""
import ctypes
import os
import re

import pytest

from paper_2608_21836_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "l4l.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(l4l_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_are_all_exported(lib):
    names = declared_symbols()
    assert set(binding.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/l4l.h but not exported"


def test_status_strings_and_version(lib):
    assert binding.version().count(".") == 1
    seen = {binding.status_string(s) for s in range(6)}
    assert len(seen) == 6 and "ok" in seen


def test_workspace_bytes_and_shape_guards(lib):
    wb = binding.l4l_workspace_bytes
    assert wb(binding.L4L_OP_PREFILL, 4, 32, 8, 128, 8192) >= 256
    d = wb(binding.L4L_OP_DECODE, 32, 32, 8, 128, 4096)
    assert d >= 256 + 32 * 32 * 129 * 4
    assert wb(binding.L4L_OP_DECODE, 32, 32, 8, 96, 4096) == 0      # head_dim not supported
    assert wb(binding.L4L_OP_DECODE, 32, 30, 8, 128, 4096) == 0     # Hq % Hkv != 0
    assert wb(binding.L4L_OP_DECODE, 1, 32, 1, 128, 4096) == 0      # group of 32 > 16
    assert wb(7, 1, 8, 8, 128, 16) == 0


def test_host_validation_returns_codes_without_a_gpu(lib):
    T4, KV = binding.Tensor4, binding.KVCache
    null4 = T4(None, 0, 0, 0)
    nullkv = KV(None, None, 0, 0, 0, 0)
    fake = 0x1000  # an aligned non-null address that is never dereferenced on these paths
    ok4 = T4(fake, 1024, 512, 128)
    okkv = KV(fake, fake, 1 << 20, 1 << 17, 128, 1024)
    # unsupported head_dim / grouping
    assert lib.l4l_attn_decode(fake, fake, okkv, fake, 16, 1, 8, 8, 96, 1.0, None, fake, 1 << 20, None) == binding.L4L_ERR_UNSUPPORTED
    assert lib.l4l_attn_decode(fake, fake, okkv, fake, 16, 1, 6, 4, 128, 1.0, None, fake, 1 << 20, None) == binding.L4L_ERR_UNSUPPORTED
    assert lib.l4l_attn_prefill(ok4, ok4, ok4, ok4, nullkv, fake, 16, 1, 8, 8, 80, 1.0, None, fake, 256, None) == binding.L4L_ERR_UNSUPPORTED
    # null / misaligned pointers, bad strides
    assert lib.l4l_attn_decode(None, fake, okkv, fake, 16, 1, 8, 8, 128, 1.0, None, fake, 1 << 20, None) == binding.L4L_ERR_INVALID_ARG
    assert lib.l4l_attn_decode(fake + 2, fake, okkv, fake, 16, 1, 8, 8, 128, 1.0, None, fake, 1 << 20, None) == binding.L4L_ERR_INVALID_ARG
    assert lib.l4l_attn_decode(fake, fake, nullkv, fake, 16, 1, 8, 8, 128, 1.0, None, fake, 1 << 20, None) == binding.L4L_ERR_INVALID_ARG
    assert lib.l4l_attn_decode(fake, fake, okkv, fake, 4096, 1, 8, 8, 128, 1.0, None, fake, 1 << 20, None) == binding.L4L_ERR_INVALID_ARG  # max_kv_len > cache.max_len
    bad_stride = T4(fake, 1024, 516, 128)
    assert lib.l4l_attn_prefill(bad_stride, ok4, ok4, ok4, nullkv, fake, 16, 1, 8, 8, 128, 1.0, None, fake, 256, None) == binding.L4L_ERR_INVALID_ARG
    assert lib.l4l_attn_prefill(null4, ok4, ok4, ok4, nullkv, fake, 16, 1, 8, 8, 128, 1.0, None, fake, 256, None) == binding.L4L_ERR_INVALID_ARG
    assert lib.l4l_kv_append(nullkv, ok4, ok4, fake, None, 1, 1, 8, 128, None) == binding.L4L_ERR_INVALID_ARG
    assert lib.l4l_kv_append(okkv, ok4, ok4, None, None, 1, 1, 8, 128, None) == binding.L4L_ERR_INVALID_ARG
    # workspace missing / too small
    assert lib.l4l_attn_decode(fake, fake, okkv, fake, 16, 1, 8, 8, 128, 1.0, None, None, 0, None) == binding.L4L_ERR_WORKSPACE
    assert lib.l4l_attn_decode(fake, fake, okkv, fake, 1024, 4, 8, 8, 128, 1.0, None, fake, 300, None) == binding.L4L_ERR_WORKSPACE
    assert lib.l4l_attn_prefill(ok4, ok4, ok4, ok4, nullkv, fake, 16, 1, 8, 8, 128, 1.0, None, fake, 100, None) == binding.L4L_ERR_WORKSPACE
    assert lib.l4l_workspace_init(None, 0, None) == binding.L4L_ERR_WORKSPACE
    # empty problems are fine and launch nothing
    assert lib.l4l_attn_decode(fake, fake, okkv, fake, 16, 0, 8, 8, 128, 1.0, None, fake, 256, None) == binding.L4L_OK
    assert lib.l4l_kv_append(okkv, ok4, ok4, fake, None, 0, 1, 8, 128, None) == binding.L4L_OK


def test_missing_library_is_an_error_not_a_fallback(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(FileNotFoundError):
        binding.load()
