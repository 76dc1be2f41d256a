"""The C-ABI library loads without a GPU and exports what the header declares;
host-side argument checks answer before any device work."""
import ctypes
import os
import re

import paper_1908_07782_b200 as combo
from paper_1908_07782_b200 import build as cuda_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "combo_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(combo_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    cuda_build.build()
    lib = ctypes.CDLL(cuda_build.LIB)
    names = declared_symbols()
    assert {"combo_select_peers", "combo_segment_aggregate", "combo_segment_aggregate_bf16",
            "combo_segment_aggregate_sgd", "combo_round_host"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_status_strings_and_version():
    lib = combo.load()
    assert combo.combo_version() >= 100
    seen = {lib.combo_status_string(i).decode() for i in range(7)}
    assert len(seen) == 7 and "ok" in seen
    assert lib.combo_status_string(77).decode() == "unknown status"


def test_host_side_argument_checks_need_no_device():
    lib = combo.load()
    # invalid sizes are rejected before any CUDA call
    assert lib.combo_select_peers(1, 0, 0, 1, 0, None) == 1
    assert lib.combo_select_peers(1, 0, 4, 2, 4, None) == 1
    assert lib.combo_select_peers(1, 0, 4, 2, 0, None) == 0          # R = 0: nothing to do
    buf = ctypes.create_string_buffer(64)
    a = ctypes.addressof(buf)
    a += (-a) % 16
    assert lib.combo_segment_aggregate(a, a, None, None, 1, 4, 1, 0, None) == 2       # alias
    assert lib.combo_segment_aggregate(a + 4, a + 32, None, None, 1, 4, 1, 0, None) == 1  # misaligned
    assert lib.combo_segment_aggregate(a, a + 32, None, None, 2, 4, 1, 1, None) == 1  # idx missing


def test_launch_column_limit_keeps_copy_coordinates_in_int32():
    # the staged kernels pass column numbers to the copy engine as signed 32-bit values: the
    # widest range one launch takes, plus the widest box (256 columns), must stay below 2^31,
    # and shards must start on 16-byte boundaries for both element sizes
    lim = combo.combo_max_launch_columns()
    assert lim + 256 < 2 ** 31 and lim % 64 == 0 and lim >= 2 ** 28
    # a 2^31-column row (8 GB in binary32) is therefore cut into several launches
    assert -(-(2 ** 31) // lim) >= 2
    combo.combo_set_launch_columns(100_000)      # rounded down to a multiple of 64; no device needed
    combo.combo_set_launch_columns(0)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_1908_07782_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    try:
        binding.load()
    except RuntimeError as e:
        assert "no fallback" in str(e)
    else:
        raise AssertionError("a missing library must raise")
