"""The C-ABI library loads and exports every symbol the header declares; host-only entry
points behave (no kernel is launched here)."""
import ctypes
import glob
import os
import re

from conftest import ROOT


def _declared_symbols():
    names = set()
    for h in glob.glob(os.path.join(ROOT, "include", "*.h")):
        src = open(h).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        names |= set(re.findall(r"\b(bs_[a-z0-9_]+)\s*\(", src))
    return names


def test_every_declared_symbol_is_exported_and_bound(lib):
    declared = _declared_symbols()
    assert {"bs_softmax_verify", "bs_residual_sample", "bs_bandit_select", "bs_bandit_update"} <= declared
    so = ctypes.CDLL(lib.LIB_PATH)
    for name in declared:
        assert hasattr(so, name), f"{name} declared in include/ but not exported"
        assert name in lib.SIGNATURES, f"{name} has no Python binding"
    assert set(lib.SIGNATURES) <= declared


def test_host_only_entry_points(lib):
    assert lib._lib.bs_status_string(0) == b"ok"
    assert b"workspace" in lib._lib.bs_status_string(lib.BS_ERR_WORKSPACE)
    n = lib.bs_workspace_bytes(64, 8, 128256)
    assert n > 0 and n % 256 == 0
    assert lib.bs_workspace_bytes(64, 8, 128256) <= lib.bs_workspace_bytes(128, 8, 128256)
    assert lib.bs_workspace_bytes(0, 8, 1000) == 0
    assert lib.bs_workspace_bytes(4, lib.BS_MAX_GAMMA + 1, 1000) == 0
    assert lib.bs_workspace_bytes(lib.BS_MAX_BATCH + 1, 4, 1000) == 0
    assert lib.bs_bandit_state_bytes(lib.BS_UCB, 256, 4) >= 256 + 256 * 4 * 16
    assert lib.bs_bandit_state_bytes(lib.BS_EXP3, 1, lib.BS_MAX_ARMS + 1) == 0
    assert lib.bs_bandit_state_bytes(7, 1, 2) == 0


def test_argument_checks_reject_before_any_launch(lib):
    # NULL pointers and bad sizes are refused on the host: safe without a GPU
    f = lib._lib.bs_softmax_verify
    assert f(None, None, 0, None, None, None, 1.0, 4, 2, 100, None, None, None, None, 0, None) == lib.BS_ERR_INVALID_ARG
    assert f(None, None, 0, None, None, None, 1.0, 0, 2, 100, None, None, None, None, 0, None) == lib.BS_ERR_INVALID_ARG
    assert f(None, None, 0, None, None, None, 1.0, 4, 40, 100, None, None, None, None, 0, None) == lib.BS_ERR_UNSUPPORTED
    g = lib._lib.bs_residual_sample
    assert g(None, None, 0, None, None, None, None, 1.0, 4, 2, 100, None, None, None, 0, None) == lib.BS_ERR_INVALID_ARG
    assert lib._lib.bs_bandit_select(None, 0, 0, 4, 2, None, None, None, None, None, None) == lib.BS_ERR_INVALID_ARG
    assert lib._lib.bs_bandit_update(None, 0, 0, 4, 2, None, None, None, None) == lib.BS_ERR_INVALID_ARG
    assert lib._lib.bs_workspace_init(None, 0, None) == lib.BS_ERR_INVALID_ARG
