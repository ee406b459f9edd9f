"""The C-ABI library: it builds, loads, exports every declared symbol, and rejects bad
arguments on the host before anything is launched (no GPU needed for any of this)."""
import ctypes
import os
import re

import pytest

from paper_2607_20457_b200 import _build, binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "pulsar.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(pulsar_[a-z0-9_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    raw = ctypes.CDLL(binding.library_path())
    for name in declared:
        assert getattr(raw, name) is not None


def test_status_strings_and_version(lib):
    assert lib.pulsar_abi_version() == 1
    for code, name in binding.STATUS_NAMES.items():
        assert lib.pulsar_status_string(code) == name.encode()
    assert lib.pulsar_status_string(99) == b"PULSAR_ERR_UNKNOWN"


def test_workspace_sizes(lib):
    # selection: B presence bitmaps of ceil(V/32) words + a uint16 df table + a uint16 level per
    # chunk, each 256-byte rounded
    words = (128256 + 31) // 32
    exp = -(-16 * words * 4 // 256) * 256 + -(-128256 * 2 // 256) * 256 + 16 * 256 * 2
    assert binding.maxidf_select_workspace_bytes(131072, 128256, 8192, 32, 16, 64) == exp
    # phase 1: gathered prefix K and V + the work counter
    assert binding.phase1_workspace_bytes(131072, 32, 8, 128, 8192, 7744) == 2 * 7744 * 8 * 128 * 2 + 256
    # phase 2: fp32 partials for the chosen number of parts
    assert binding.phase2_workspace_bytes(512, 16, 8192, 32, 8, 128, 4) == 4 * 512 * 32 * 129 * 4 + 256   # + work counter
    assert binding.phase2_workspace_bytes(512, 16, 8192, 32, 8, 128, 1) == 256
    # a sequence that ends inside a block: ceil(100/64) = 2 blocks of ceil(64/8) = 8 chunk slots
    assert binding.maxidf_select_workspace_bytes(100, 128, 64, 8, 1, 0) == 3 * 256
    # shapes the kernels do not cover give 0
    assert binding.maxidf_select_workspace_bytes(128, 128, 64, 8, 9, 0) == 0
    assert lib.pulsar_chunk_select_workspace_bytes(100, 128, 64, 8, 1, 0, 2) == 3 * 256   # the other scores too
    assert binding.phase1_workspace_bytes(4096, 4, 1, 96, 1024, 0) == 0


def test_host_validation_launches_nothing(lib):
    null = None
    one = ctypes.c_void_p(256)          # never dereferenced: validation fails first
    # selection: k above chunks per block, sink above the block, more blocks than the 16-bit levels cover
    assert lib.pulsar_maxidf_select(one, 128, 128, 64, 8, 9, 0, one, one, one, null, null, one, 1 << 20, null, null) == 2
    assert lib.pulsar_maxidf_select(one, 128, 128, 64, 8, 1, 65, one, one, one, null, null, one, 1 << 20, null, null) == 2
    assert lib.pulsar_maxidf_select(one, 65534, 128, 1, 1, 1, 0, one, one, one, null, null, one, 1 << 30, null, null) == 2
    # NULL data pointer, misaligned pointer, workspace too small
    assert lib.pulsar_maxidf_select(null, 128, 128, 64, 8, 1, 0, one, one, one, null, null, one, 1 << 20, null, null) == 1
    assert lib.pulsar_maxidf_select(ctypes.c_void_p(260), 128, 128, 64, 8, 1, 0, one, one, one, null, null, one, 1 << 20, null, null) == 3
    assert lib.pulsar_maxidf_select(one, 128, 128, 64, 8, 1, 0, one, one, one, null, null, one, 16, null, null) == 4
    # phase 1: head dim, GQA ratio
    args = lambda d, Hq, Hkv: (one, one, one, 4096, Hq, Hkv, d, 1024, one, one, 64, 0.0, one, null, null, null, one, 1 << 30, null, null)
    assert lib.pulsar_phase1_attn(*args(96, 4, 1)) == 2
    assert lib.pulsar_phase1_attn(*args(64, 5, 2)) == 2
    # phase 2: partial outputs need an explicit split count; a split count that would leave a part
    # empty is rejected (32 key tiles cannot be cut into 31 non-empty runs of whole tiles)
    assert lib.pulsar_phase2_attn(one, 8, one, one, 4, 1024, 4, 1, 64, 0.0, 0, one, null, one, one, one, 1 << 30, null, null) == 1
    assert lib.pulsar_phase2_attn(one, 8, one, one, 4, 1024, 4, 1, 64, 0.0, 31, one, null, null, null, one, 1 << 30, null, null) == 2
    # merge: d must be a multiple of 4
    assert lib.pulsar_lse_merge(one, one, 2, 8, 6, one, null, null) == 2


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(_build, "LIB", str(tmp_path / "absent.so"))
    with pytest.raises(FileNotFoundError):
        binding.load_library()
