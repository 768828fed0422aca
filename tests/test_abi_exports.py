"""The C-ABI library without a GPU: it loads, exports every function that
include/alexnet.h declares, the Python binding names the same set, and the
host-only entry points (sizes, argument checks) behave as the header states."""
import ctypes
import os
import re

import pytest

from paper_1412_2302_b200 import alexnet as A
from paper_1412_2302_b200 import build as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "alexnet.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(alexnet_[a-z0-9_]+)\s*\(", src)))


@pytest.fixture(scope="module")
def lib():
    B.build()
    return A.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "alexnet_create" in names and "alexnet_train_step" in names and len(names) >= 19
    for n in names:
        assert getattr(lib, n) is not None, n
    assert sorted(A.EXPORTS) == names


def test_binding_enums_match_header():
    src = open(os.path.join(ROOT, "include", "alexnet.h")).read()
    tensors = re.findall(r"ALEXNET_T_([A-Z0-9]+)", src.split("ALEXNET_T_CROPFLIP = 0", 1)[1].split("ALEXNET_T_COUNT")[0])
    assert ["CROPFLIP"] + tensors == A.TENSORS
    ops = re.findall(r"ALEXNET_OP_([A-Z0-9_]+)", src.split("ALEXNET_OP_CONV1_FWD = 0", 1)[1].split("ALEXNET_OP_COUNT")[0])
    assert ["CONV1_FWD"] + ops == A.OPS


def test_host_only_entry_points(lib):
    assert lib.alexnet_param_count() == 60965224
    cfg = A.Config(128, 1, 1, 0.01, 0.9, 5e-4, 5, 1e-4, 0.75, 2.0, 0.5, 0.0, 0)
    one = lib.alexnet_workspace_bytes(ctypes.byref(cfg))
    cfg2 = A.Config(128, 2, 1, 0.01, 0.9, 5e-4, 5, 1e-4, 0.75, 2.0, 0.5, 0.0, 0)
    two = lib.alexnet_workspace_bytes(ctypes.byref(cfg2))
    # parameters, momentum, gradients (fp32) and the bf16 copy: at least 14 bytes per parameter and replica
    assert one > 14 * 60965224 and two > one + 14 * 60965224 and one % 1024 == 0
    assert two < 8 * 2**30                                   # two batch-128 replicas stay far below one GPU's HBM
    for bad in (A.Config(0, 1, 1, 0.01, 0.9, 5e-4, 5, 1e-4, 0.75, 2.0, 0.5, 0.0, 0),       # batch
                A.Config(8, 3, 1, 0.01, 0.9, 5e-4, 5, 1e-4, 0.75, 2.0, 0.5, 0.0, 0),       # replicas
                A.Config(8, 1, 1, 0.01, 0.9, 5e-4, 3, 1e-4, 0.75, 2.0, 0.5, 0.0, 0),       # LRN size
                A.Config(8, 1, 1, 0.01, 0.9, 5e-4, 5, 1e-4, 0.75, 2.0, 1.0, 0.0, 0)):      # dropout p
        assert lib.alexnet_workspace_bytes(ctypes.byref(bad)) == 0
    assert lib.alexnet_workspace_bytes(None) == 0
    h = ctypes.c_void_p()
    assert lib.alexnet_create(None, None, 0, None, None, None, ctypes.byref(h)) == A.ERR_ARG and not h.value
    assert lib.alexnet_create(ctypes.byref(cfg), None, 0, None, None, None, None) == A.ERR_ARG
    for fn in (lib.alexnet_destroy, lib.alexnet_sync, lib.alexnet_replica_average):
        assert fn(None) == A.ERR_ARG
    assert lib.alexnet_train_step(None, 0, None) == A.ERR_ARG
    assert lib.alexnet_last_error(None) == b"null handle"
    assert lib.alexnet_launch_count(None) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(A, "_lib", None)
    monkeypatch.setattr(B, "LIB", str(tmp_path / "nothing.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        A.load_library()
