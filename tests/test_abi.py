"""The C-ABI library builds for sm_100a, loads without a GPU and exports what include/ppow.h declares.
Host-only entry points (sizes, strings) are exercised; nothing here launches a kernel."""
import ctypes
import os
import re

import pytest

from paper_2605_14978_b200 import binding as B
from paper_2605_14978_b200 import build as build_mod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build_mod.build()
    return B.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "ppow.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ppow_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert set(names) == set(B.EXPORTS)
    for n in names:
        assert hasattr(lib, n), n


def test_struct_layouts_match_header():
    assert ctypes.sizeof(B.ppow_params) == 9 * 4
    assert ctypes.sizeof(B.ppow_outputs) == 18 * ctypes.sizeof(ctypes.c_void_p)
    text = open(os.path.join(ROOT, "include", "ppow.h")).read()
    body = re.search(r"typedef struct \{(.*?)\} ppow_outputs;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    order = re.findall(r"\*\s*([a-z_]+)\s*;", body)
    assert order == [n for n, _ in B.ppow_outputs._fields_]


def test_host_only_entry_points(lib):
    assert B.ppow_version() >= 100
    assert B.ppow_status_string(B.PPOW_OK) == "ok"
    for st in range(0, 7):
        assert isinstance(B.ppow_status_string(st), str) and B.ppow_status_string(st)
    p = B.make_params(2048, 8, 128256, B.PPOW_BF16, B.PPOW_STOCHASTIC, 0.04)
    need = B.ppow_score_workspace_bytes(p)
    assert need >= 256 + 2048 * 8 * 32 and need % 16 == 0
    assert B.ppow_score_workspace_bytes(B.make_params(4, 8, 128256, B.PPOW_BF16, 0, 0.04)) >= 256 + 32 * 32
    assert B.ppow_score_workspace_bytes(B.make_params(4, 0, 10, B.PPOW_BF16, 0, 0.04)) == 0     # invalid K
    assert B.ppow_score_workspace_bytes(B.make_params(4, 40, 10, B.PPOW_BF16, 0, 0.04)) == 0    # K > 32
    assert B.ppow_score_workspace_bytes(B.make_params(4, 4, 10, 7, 0, 0.04)) == 0               # bad dtype
    assert B.ppow_select_workspace_bytes(0) == 0
    assert B.ppow_select_workspace_bytes(8192) > 0
    assert B.ppow_select_workspace_bytes(100000) >= 131072 * 8


def test_score_workspace_grows_with_the_number_of_windows(lib):
    # the host-buffer entry point scores chunks of different sizes out of one workspace sized for the largest:
    # a shorter chunk must never need more
    for K, V, dt in ((8, 32000, B.PPOW_BF16), (8, 128256, B.PPOW_BF16), (10, 151936, B.PPOW_F16), (4, 1000, B.PPOW_F32),
                     (12, 152064, B.PPOW_F32), (1, 5000, B.PPOW_BF16), (32, 777, B.PPOW_BF16)):
        last = 0
        for N in list(range(1, 400)) + list(range(400, 9000, 37)):
            need = B.ppow_score_workspace_bytes(B.make_params(N, K, V, dt, B.PPOW_GREEDY, 0.05))
            assert need >= last and need >= 256 + 64 * N * K and need <= 256 + 64 * 32 * N * K, (N, K, V)
            last = need


def test_binding_refuses_cpu_tensors(lib):
    import torch
    x = torch.zeros((1, 1, 8), dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        B._dev_ptr(x, torch.bfloat16, "draft_logits")


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libppow.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        B.load_library()
