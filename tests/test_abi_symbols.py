"""The C-ABI library builds, loads without a GPU and exports every symbol the header declares."""
import ctypes as C
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2607_11211_b200 import build
    return C.CDLL(str(build.build()))


def declared_functions():
    names = set()
    for header in sorted((ROOT / "include").glob("*.h")):
        text = re.sub(r"/\*.*?\*/", "", header.read_text(), flags=re.S)
        names |= set(re.findall(r"\b(fasttps_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"fasttps_attn_decode", "fasttps_mlp_decode", "fasttps_layer_decode", "fasttps_model_decode",
            "fasttps_create", "fasttps_destroy", "fasttps_baseline_attn", "fasttps_baseline_mlp"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_host_side_argument_checks_need_no_gpu(lib):
    lib.fasttps_strerror.restype = C.c_char_p
    assert lib.fasttps_strerror(0) == b"ok"
    assert b"invalid" in lib.fasttps_strerror(-1)
    assert lib.fasttps_create(None, None) == -1
    assert lib.fasttps_destroy(None) == -1
    assert lib.fasttps_attn_decode(None, None, None, None, None, None, None, None, None, 1, None) == -1
    assert lib.fasttps_mlp_decode(None, None, None, None, None, 1, None) == -1
    lib.fasttps_packed_bytes.restype = C.c_size_t
    assert lib.fasttps_packed_bytes(None, 0) == 0


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    from paper_2607_11211_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", tmp_path / "nope.so")
    with pytest.raises(binding.FasttpsError):
        binding.load_library()
