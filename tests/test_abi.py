"""The C-ABI library builds for sm_100a, loads without a GPU and exports every declared symbol;
host-only entry points (workspace sizing, argument checks) behave as the header states."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2512_07993_b200 import build, binding
    build.build()
    return binding


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(skipkv_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(binding):
    lib = binding.lib()
    names = declared_symbols()
    assert {"skipkv_score", "skipkv_select", "skipkv_compact", "skipkv_decode_attn", "skipkv_steer"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(binding.SYMBOLS) <= set(names)


def test_workspace_bytes_and_shape_checks(binding):
    B = binding
    ok = B.make_shape(10, 32, 8, 128, 32, 4096, 700, 32768, None, None)
    n = B.skipkv_workspace_bytes(ok)
    assert n % 256 == 0 and 1 << 20 < n < 1 << 30
    bigger = B.make_shape(16, 40, 8, 128, 64, 5120, 5000, 65536, None, None)
    assert B.skipkv_workspace_bytes(bigger) > n
    for bad, code in [
        (B.make_shape(10, 32, 8, 64, 32, 4096, 700, 32768, None, None), -2),     # head_dim != 128
        (B.make_shape(10, 30, 8, 128, 32, 4096, 700, 32768, None, None), -2),    # Hq % Hk != 0
        (B.make_shape(10, 128, 8, 128, 32, 4096, 700, 32768, None, None), -2),   # group 16 > 8
        (B.make_shape(10, 32, 8, 128, 256, 4096, 700, 32768, None, None), -2),   # group*window > 512
        (B.make_shape(0, 32, 8, 128, 32, 4096, 700, 32768, None, None), -1),     # batch 0
        (B.make_shape(10, 32, 8, 128, 32, 4096, 700, 0, None, None), -1),        # max_cap 0
        (B.make_shape(10, 32, 8, 128, 32, 4100, 700, 32768, None, None), -2),    # d_model % 8 != 0
    ]:
        with pytest.raises(B.SkipKVError) as e:
            B.skipkv_workspace_bytes(bad)
        assert e.value.code == code


def test_null_arguments_are_rejected_before_any_launch(binding):
    lib = binding.lib()
    shape = binding.make_shape(1, 4, 1, 128, 8, 256, 16, 128, None, None)
    # slab_off / cap are null: every compute entry point must refuse without touching CUDA
    null = C.c_void_p(None)
    p = binding.make_params(budget=8)
    assert lib.skipkv_score(C.byref(shape), C.byref(p), null, null, null, null, null, null, null, null, null, null,
                            null, null) == -1
    assert lib.skipkv_select(C.byref(shape), C.byref(p), null, null, null, null, null, null, null, null, null) == -1
    assert lib.skipkv_compact(C.byref(shape), null, null, null, null, null, null, null, null, null, null) == -1
    assert lib.skipkv_decode_attn(C.byref(shape), null, null, null, null, null, null, null, null, null, null,
                                  null) == -1
    assert lib.skipkv_steer(C.c_int32(1), C.c_int32(256), null, null, null, null, null) == -1
    assert lib.skipkv_steer(C.c_int32(1), C.c_int32(250), C.c_void_p(16), C.c_void_p(16), C.c_void_p(16),
                            C.c_void_p(16), null) == -2


def test_binding_fails_loudly_without_library(binding, monkeypatch):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", "/nonexistent/libskipkv.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.lib()
