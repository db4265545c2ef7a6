"""The C-ABI library loads, exports every symbol the header declares, answers
its host-only queries and rejects bad arguments before touching a device.
CPU only: no compute call succeeds here."""
import ctypes
import os
import re

import pytest

import __graft_entry__  # noqa: F401  (builds the library if needed)
from paper_2205_14756_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000  # 16-byte aligned, never dereferenced on the host


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "msla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(msla_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    lib = ctypes.CDLL(binding.LIB_PATH)
    names = declared_symbols()
    assert "msla_linattn_relu" in names and "msla_forward" in names and len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in msla.h but not exported"
        assert n in binding.EXPORTS, f"{n} has no Python binding"


def test_version_and_strings():
    lib = binding.lib()
    assert binding.msla_version() >= 100
    assert lib.msla_status_string(0) == b"ok"
    for s in range(1, 7):
        assert len(lib.msla_status_string(s)) > 0


def test_core_workspace_query():
    assert binding.msla_linattn_relu_workspace_bytes(8, 16, 4096, 32) > 8 * 16 * 32 * 33 * 4
    assert binding.msla_linattn_relu_workspace_bytes(1, 1, 1, 16) > 0
    for bad in [(0, 1, 1, 32), (1, 0, 1, 32), (1, 1, 0, 32), (1, 1, 1, 0), (1, 1, 8, 24), (1, 1, 8, 64)]:
        assert binding.msla_linattn_relu_workspace_bytes(*bad) == 0


def test_core_split_depends_on_shape_only():
    a = binding.msla_linattn_relu_workspace_bytes(1, 16, 262144, 32)
    assert a == binding.msla_linattn_relu_workspace_bytes(1, 16, 262144, 32)
    # more tokens per head -> more chunks -> more scratch, until the cap
    assert binding.msla_linattn_relu_workspace_bytes(1, 1, 1 << 20, 32) >= binding.msla_linattn_relu_workspace_bytes(1, 1, 1024, 32)


def _core(*args):
    return binding.lib().msla_linattn_relu(*args)


def test_core_rejects_bad_arguments_on_the_host():
    lib = binding.lib()
    assert _core(None, FAKE, FAKE, FAKE, 1, 1, 8, 32, 1e-15, None) == 1
    assert b"null" in lib.msla_last_error()
    assert _core(FAKE, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 0, 32, 1e-15, None) == 1
    assert _core(FAKE, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 8, 24, 1e-15, None) == 2
    assert _core(FAKE + 2, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 8, 32, 1e-15, None) == 3
    # out aliases q
    assert _core(FAKE, FAKE + 4096, FAKE + 8192, FAKE, 1, 1, 8, 32, 1e-15, None) == 1
    assert _core(FAKE, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 8, 32, -1.0, None) == 1
    # workspace variant: too small
    assert lib.msla_linattn_relu_ws(1, FAKE, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 8, 32, 1e-15,
                                    FAKE + 65536, 16, None) == 4
    assert lib.msla_linattn_relu_ws(7, FAKE, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 8, 32, 1e-15,
                                    FAKE + 65536, 1 << 20, None) == 1


def test_forward_descriptor_validation():
    ok = binding.make_desc(1, 64, 16, 16, 4, 16, 64, binding.MSLA_F32)
    need = binding.msla_forward_workspace_bytes(ok)
    # at least the multi-scale buffer (6C') and the attention output (2C')
    assert need >= 256 * (6 * 64 + 2 * 64) * 4
    for field, value in [("n_scales", 4), ("n_scales", 1), ("agg_kernel", 7), ("agg_kernel", 4), ("d", 20), ("heads", 0), ("struct_size", 8), ("C", 60)]:
        bad = binding.make_desc(1, 64, 16, 16, 4, 16, 64, binding.MSLA_F32)
        setattr(bad, field, value)
        assert binding.msla_forward_workspace_bytes(bad) == 0, field
    lib = binding.lib()
    w = binding.msla_weights()
    w.w_qkv = w.w_dw = w.w_pw = w.w_proj = FAKE
    # no workspace -> MSLA_ERR_WORKSPACE, before any device access
    assert lib.msla_forward(ctypes.byref(ok), FAKE, ctypes.byref(w), FAKE + (1 << 20), None) == 4
    bad = binding.make_desc(1, 64, 16, 16, 4, 16, 64, binding.MSLA_F32)
    bad.n_scales = 1
    assert lib.msla_forward(ctypes.byref(bad), FAKE, ctypes.byref(w), FAKE + (1 << 20), None) == 2


def test_compute_call_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    st = _core(FAKE, FAKE + 4096, FAKE + 8192, FAKE + 12288, 1, 1, 8, 32, 1e-15, None)
    assert st in (5, 6)            # MSLA_ERR_ARCH or MSLA_ERR_CUDA, never MSLA_OK
    assert len(binding.lib().msla_last_error()) > 0
