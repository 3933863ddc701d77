"""The C-ABI library loads without a GPU and exports every declared symbol."""
import os
import re

import pytest

from paper_2410_09615_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "slim.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(slim_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert "slim_pack" in names and "slim_linear_fwd" in names and len(names) >= 10
    for n in names:
        assert hasattr(lib, n), f"{n} not exported"
        assert n in binding.SIGNATURES, f"{n} has no Python signature"
    assert sorted(binding.SIGNATURES) == names


def test_error_strings_and_version(lib):
    assert binding.strerror(binding.SLIM_OK) == "ok"
    texts = {binding.strerror(c) for c in range(9)}
    assert len(texts) == 9 and all(texts)
    assert b"sm_100a" in lib.slim_version()


def test_workspace_bytes_host_logic(lib):
    f = binding.slim_workspace_bytes
    assert f(0, 512, 512, 64) == 0            # b < 1
    assert f(8, 500, 512, 64) == 0            # d_out % 16
    assert f(8, 512, 520, 64) == 0            # d_in % 64
    assert f(8, 512, 512, 60) == 0            # r % 16
    small = f(8, 512, 512, 64)
    assert small >= binding.WORKSPACE_SYNC_BYTES + 8 * 64 * 4 and small % 256 == 0
    assert f(16, 4096, 4096, 416) > small
    # grows with the token count (the adapter intermediate is b x r fp32)
    assert f(2048, 4096, 4096, 416) >= 2048 * 416 * 4


def test_host_side_argument_checks_need_no_device(lib):
    # null pointers and bad shapes are rejected before any CUDA call
    assert lib.slim_pack(None, None, 16, 64, None, None, None, None) == binding.SLIM_ERR_INVALID_ARG
    assert lib.slim_unpack(None, None, 16, 64, None, None, None) == binding.SLIM_ERR_INVALID_ARG
    assert lib.slim_linear_fwd(None, 1, None, None, 1.0, None, None, 0, 16, 64, None, None, 0, None,
                               None) == binding.SLIM_ERR_INVALID_ARG
    assert lib.slim_workspace_reset(None, 0, None) == binding.SLIM_ERR_WORKSPACE
    one = 16  # a fake, aligned, never dereferenced address: shape errors come first
    assert lib.slim_pack(one, one, 16, 60, one, one, None, None) == binding.SLIM_ERR_UNSUPPORTED_SHAPE
    assert lib.slim_pack(one, one, 10, 64, one, one, None, None) == binding.SLIM_ERR_UNSUPPORTED_SHAPE
    assert lib.slim_pack(one + 4, one, 16, 64, one, one, None, None) == binding.SLIM_ERR_INVALID_ARG


def test_tiled_entry_points_host_logic(lib):
    assert binding.slim_tiled_bytes(4096, 4096) == 4096 * 4096 * 3 // 8
    assert binding.slim_tiled_bytes(48, 256) == 64 * 256 * 3 // 8      # whole groups of 64 rows
    assert binding.slim_tiled_bytes(4096, 4096, 2) == 0           # unknown layout
    assert binding.slim_tiled_bytes(4100, 4096) == 0 and binding.slim_tiled_bytes(4096, 4160) == 0
    one = 16
    assert lib.slim_repack_tiled(None, None, 16, 256, 1, None, None) == binding.SLIM_ERR_INVALID_ARG
    assert lib.slim_repack_tiled(one, one, 16, 320, 1, one, None) == binding.SLIM_ERR_UNSUPPORTED_SHAPE
    assert lib.slim_linear_fwd_tiled(None, 1, None, 1, 1.0, None, None, 0, 16, 256, None, None, 0, None,
                                     None) == binding.SLIM_ERR_INVALID_ARG
    # a scale that is not finite is an argument error, before any device work
    for bad in (float("nan"), float("inf"), -float("inf")):
        assert lib.slim_linear_fwd(one, 1, one, one, bad, None, None, 0, 16, 64, one, one, 1 << 20, None,
                                   None) == binding.SLIM_ERR_INVALID_ARG
        assert lib.slim_linear_fwd_tiled(one, 1, one, 1, bad, None, None, 0, 16, 256, one, one, 1 << 20, None,
                                         None) == binding.SLIM_ERR_INVALID_ARG


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libslim.so")
    with pytest.raises(binding.SlimError):
        binding.lib()


def test_header_enums_match_the_binding():
    """Every SLIM_ERR_* / SLIM_KERNEL_* value of the header has the same value in the binding."""
    import re
    text = open(os.path.join(ROOT, "include", "slim.h")).read()
    pairs = re.findall(r"\b(SLIM_(?:ERR|KERNEL)_[A-Z_]+|SLIM_OK)\s*=\s*(\d+)", text)
    assert len(pairs) >= 12
    for name, value in pairs:
        py = name if name.startswith("SLIM_ERR") or name == "SLIM_OK" else name.replace("SLIM_", "")
        assert hasattr(binding, py), f"{name} missing from the binding"
        assert getattr(binding, py) == int(value), name
