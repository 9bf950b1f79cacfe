"""The C-ABI library loads without a GPU and exports every function pass.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "pass.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pass_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    from paper_2311_13581_b200.build import build_library
    lib = ctypes.CDLL(build_library())
    names = declared_functions()
    assert len(names) >= 15 and "pass_step" in names and "pass_forward_tokens" in names
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_names():
    from paper_2311_13581_b200.binding import EXPORTS
    assert sorted(EXPORTS) == declared_functions()


def test_host_side_argument_checks_need_no_gpu():
    from paper_2311_13581_b200 import binding
    lib = binding.load_library()
    cfg = binding._Config(2, 256, 4, 64, 688, 1024, 8, 1, 128, 0, 1e-6, 1e4)
    assert lib.pass_kv_bytes(ctypes.byref(cfg)) == 2 * 1 * 128 * 256 * 4
    assert lib.pass_workspace_bytes(ctypes.byref(cfg)) > 0
    bad = binding._Config(2, 256, 4, 60, 688, 1024, 8, 1, 128, 0, 1e-6, 1e4)     # d_head 60
    assert lib.pass_kv_bytes(ctypes.byref(bad)) == 0
    h = ctypes.c_void_p()
    assert lib.pass_create(ctypes.byref(bad), None, None, 0, None, 0, None, ctypes.byref(h)) == -1
    assert lib.pass_strerror(-2).decode().startswith("capacity")
    assert lib.pass_step(None, 1, 0.0, None, None, None) == -1


def test_no_cpu_fallback_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    import synthetic_inputs as si
    import paper_2311_13581_b200 as pb
    with pytest.raises(RuntimeError):
        pb.PassContext(si.SHAPES["tiny"], {}, 1, 64)
