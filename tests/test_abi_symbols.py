"""The C-ABI library loads without a GPU and exports every function that
include/dgc.h declares; host-only entry points behave; device entry points
fail loudly (no CPU fallback)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_1712_01887_b200 import build
    build.build()
    from paper_1712_01887_b200 import binding
    return binding


def _declared():
    text = open(os.path.join(ROOT, "include", "dgc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dgc_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = _declared()
    assert "dgc_compress" in names and "dgc_decode_accumulate" in names and len(names) >= 15
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(B.EXPORTED)


def test_host_only_calls(B):
    assert [B.warmup_sparsity(i) for i in range(5)] == [0.75, 0.9375, 0.984375, 0.996, 0.999]
    with pytest.raises(B.DgcError):
        B.warmup_sparsity(5)
    # per worker: 11 tile boundaries + 1024 input-check words
    assert B.decode_workspace_bytes(8, 4096 * 10) == 8 * (11 + 1024) * 4
    assert B.decode_workspace_bytes(0, 10) < 0 and B.decode_workspace_bytes(65, 10) < 0
    assert isinstance(B.launch_count(), int)


def test_no_cpu_fallback(B):
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for the box without a GPU")
    with pytest.raises(B.DgcError) as e:
        B.State([1000], 1, 0.9, 0.0, 0.999)
    assert e.value.code == B.ECUDA


def test_struct_layout_matches_header(B):
    # dgc_config: 2 x int32, pointer, 2 x float, 2 x double, uint64, 5 x int32 (+ 4 bytes of
    # tail padding to the 8-byte alignment) = 72 bytes
    assert ctypes.sizeof(B.Config) == 72
    assert B.Config.nesterov.offset == 56 and B.Config.clip_scope.offset == 64
    assert B.Config.tensor_numel.offset == 8 and B.Config.sparsity.offset == 24
    assert B.Config.seed.offset == 40 and B.Config.device.offset == 48
    assert ctypes.sizeof(B.Status) == 40
