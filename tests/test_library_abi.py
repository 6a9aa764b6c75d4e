"""CPU-only checks of the compiled library: it builds, loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2512_06547_b200 as a3po
from paper_2512_06547_b200 import build as a3po_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    a3po_build.build()
    return a3po.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "a3po.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(a3po_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_functions()
    assert "a3po_token_logprobs_fwd" in names and "a3po_loss_bwd" in names and len(names) >= 12
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(a3po.exported_symbols())


def test_version_and_strings(lib):
    assert a3po.a3po_version() >= 1000
    assert lib.a3po_status_string(0) == b"ok"
    assert b"workspace" in lib.a3po_status_string(-3)
    assert lib.a3po_status_string(12345) == b"unknown a3po status"


def test_workspace_sizes_are_monotone():
    small = a3po.a3po_loss_workspace_bytes(1 << 10)
    big = a3po.a3po_loss_workspace_bytes(1 << 20)
    assert 0 < small < big and big - small >= 4 * ((1 << 20) - (1 << 10))
    for dt in (a3po.A3PO_F32, a3po.A3PO_BF16):
        fwd = a3po.a3po_token_logprobs_workspace_bytes(4096, 1536, 151936, dt, 0)
        bwd = a3po.a3po_token_logprobs_workspace_bytes(4096, 1536, 151936, dt, 1)
        mn = a3po.a3po_token_logprobs_min_workspace_bytes(4096, 1536, 151936, dt, 1)
        assert 0 < fwd and 0 < mn <= bwd
    assert a3po.a3po_token_logprobs_workspace_bytes(-1, 64, 100, 0, 0) == 0
    assert a3po.a3po_train_step_workspace_bytes(512, 64, 1000, 0) >= a3po.a3po_loss_workspace_bytes(512)
    assert a3po.a3po_train_step_stage_bytes(512, 64, 0) >= 512 * 64 * 4


def test_host_side_argument_errors(lib):
    """None of these reaches a device: the argument check comes first."""
    one = ctypes.c_void_p(256)  # fake, aligned, never dereferenced
    inval, unsup, wsp = -1, -2, -3
    # loss: NULL output, negative N, negative eps, missing workspace
    assert lib.a3po_loss_fwd(one, one, one, 0, None, 0, 1, one, one, 8, 0.2, None, None, one, 1 << 20, None) == inval
    assert lib.a3po_loss_fwd(one, one, one, 0, None, 0, 1, one, one, -1, 0.2, one, None, one, 1 << 20, None) == inval
    assert lib.a3po_loss_fwd(one, one, one, 0, None, 0, 1, one, one, 8, -0.1, one, None, one, 1 << 20, None) == inval
    assert lib.a3po_loss_fwd(one, one, one, 0, None, 0, 1, one, one, 8, 0.2, one, None, None, 0, None) == wsp
    assert lib.a3po_loss_fwd(one, one, one, 0, None, 0, 1, one, one, 8, 0.2, one, None, one, 16, None) == wsp
    assert lib.a3po_loss_fwd(one, one, one, 1, None, 0, 1, one, one, 8, 0.2, one, None, one, 1 << 20, None) == inval
    # LM head: bad dims, bad dtype, misaligned operand
    assert lib.a3po_token_logprobs_fwd(one, one, one, None, 8, 0, 100, 0, 1.0, one, one, None, one, 1 << 20, None, None) == inval
    assert lib.a3po_token_logprobs_fwd(one, one, one, None, 8, 64, 100, 7, 1.0, one, one, None, one, 1 << 20, None, None) == unsup
    assert lib.a3po_token_logprobs_fwd(ctypes.c_void_p(260), one, one, None, 8, 64, 100, 0, 1.0, one, one, None, one, 1 << 20, None, None) == unsup
    assert lib.a3po_token_logprobs_fwd(one, one, one, None, 8, 64, 100, 0, 0.0, one, one, None, one, 1 << 20, None, None) == inval
    assert lib.a3po_token_logprobs_bwd(one, one, one, one, one, 8, 64, 100, 0, 1.0, one, None, 0, one, 1 << 20, None, None) in (inval, -5)


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        a3po.load_library(str(tmp_path / "absent.so"))
