"""The C-ABI library loads without a GPU and exports every symbol include/tppo.h declares; host-only
entry points (version, status names, workspace sizes) behave; argument errors are reported before
any launch."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_15050_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tppo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tppo_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"tppo_egae", "tppo_select_tokens", "tppo_policy_loss_fwd_bwd", "tppo_value_loss",
            "tppo_lmhead_logprob_fwd_bwd", "tppo_advance_batch", "tppo_workspace_bytes", "tppo_version",
            "tppo_status_string"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_host_only_calls(lib):
    lib.tppo_status_string.restype = ctypes.c_char_p
    assert lib.tppo_version() >= 200
    assert lib.tppo_status_string(0) == b"ok"
    assert b"workspace" in lib.tppo_status_string(2)
    lib.tppo_workspace_bytes.restype = ctypes.c_size_t
    lib.tppo_workspace_bytes.argtypes = [ctypes.c_int, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, ctypes.c_int32]
    for op in range(4):
        small = lib.tppo_workspace_bytes(op, 1000, 4, 1000, 1000)
        big = lib.tppo_workspace_bytes(op, 20_000_000, 4096, 20_000_000, 152064)
        assert small > 0 and small % 256 == 0 and big >= small
    assert lib.tppo_workspace_bytes(99, 10, 1, 10, 10) == 0
    assert lib.tppo_workspace_bytes(0, -1, 1, 10, 10) == 0


def test_argument_errors_are_reported_before_any_launch(lib):
    """Null pointers / bad sizes return a status code on a machine without a GPU too."""
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    lib.tppo_egae.argtypes = [vp, vp, vp, vp, vp, vp, i32, i64, f32, f32, vp, vp, vp, vp, sz, vp]
    assert lib.tppo_egae(None, None, None, None, None, None, 1, 10, 1.0, 0.95, None, None, None, None, 0, None) == 1
    assert lib.tppo_egae(None, None, None, None, None, None, -1, 10, 1.0, 0.95, None, None, None, None, 0, None) == 1
    buf = (ctypes.c_char * 4096)()
    p = ctypes.cast(buf, vp)
    assert lib.tppo_egae(p, p, p, p, p, None, 1, 10, 1.5, 0.95, p, None, p, None, 0, None) == 1   # gamma > 1
    assert lib.tppo_egae(p, p, p, p, p, None, 1, 10, 1.0, 0.95, p, None, p, None, 0, None) == 2   # no workspace
    lib.tppo_select_tokens.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, vp, i32, i64, vp, vp, vp, vp, sz, vp]
    assert lib.tppo_select_tokens(p, p, p, p, p, -1, None, None, None, 1, 10, p, p, p, p, 4096, None) == 1
    assert lib.tppo_select_tokens(p, p, p, p, p, 0, None, None, None, 1, 10, p, p, p, None, 0, None) == 2
    lib.tppo_value_loss.argtypes = [vp, vp, vp, i64, vp, vp, i64, f32, f32, f32, vp, vp, vp, vp, sz, vp]
    assert lib.tppo_value_loss(p, p, p, 10, None, None, 20, 0.5, 0.6, 0.0, p, None, p, p, 4096, None) == 1
    lib.tppo_policy_loss_fwd_bwd.argtypes = [vp, i32, i64, i32, i64, vp, vp, vp, i64, vp, vp, vp, i64, f32, f32,
                                             f32, vp, vp, vp, vp, vp, i32, i32, vp, sz, vp]
    args = [p, 0, 4, 64, 64, p, None, None, 4, None, p, p, 4, 0.2, 0.2, 0.0, None, None, p, p, None, 0, 0, None, 0, None]
    assert lib.tppo_policy_loss_fwd_bwd(*args) == 2
    args[1] = 7
    assert lib.tppo_policy_loss_fwd_bwd(*args) == 1
    args[1], args[4] = 0, 32
    assert lib.tppo_policy_loss_fwd_bwd(*args) == 1        # ld < V


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    """The product path has no CPU fallback: a missing library is an import error."""
    import importlib
    import sys
    import paper_2506_15050_b200 as pkg
    src = open(os.path.join(os.path.dirname(pkg.__file__), "binding.py")).read()
    mod_dir = tmp_path / "fakepkg"
    mod_dir.mkdir()
    (mod_dir / "__init__.py").write_text("")
    (mod_dir / "binding.py").write_text(src)
    sys.path.insert(0, str(tmp_path))
    try:
        with pytest.raises(ImportError):
            importlib.import_module("fakepkg.binding")
    finally:
        sys.path.remove(str(tmp_path))
        sys.modules.pop("fakepkg", None)
        sys.modules.pop("fakepkg.binding", None)
