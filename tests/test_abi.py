"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2603_06619_b200 import build, nat

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "nat.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(nat_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    build.build()
    lib = ctypes.CDLL(nat.LIB_PATH)
    names = _declared()
    assert set(nat.SYMBOLS) <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    assert nat.load().nat_version() >= 1


def test_host_side_validation_needs_no_gpu():
    lib = nat.load()
    assert lib.nat_status_string(0) == b"ok"
    # invalid selection parameters are refused before any device work
    bad = nat.select_params("urs", p=0.0)
    assert lib.nat_select(ctypes.byref(bad), 2, 1, 0, 1, 1, None, None) == -1
    assert b"0 < p <= 1" in lib.nat_last_error()
    assert lib.nat_grpo_adv(1, 0, None, 1e-6, None, None) == -1
    assert lib.nat_compact_workspace_bytes(0) == 256
    assert lib.nat_compact_workspace_bytes(4096 * 3 + 1) >= 5 * 4
    p = nat.loss_params(4096, 151936, nat.NAT_BF16, 128)
    need = lib.nat_policy_loss_workspace_bytes(ctypes.byref(p), 200000)
    # bounded scratch: far below the 200000 x 151936 logits a naive path would store
    assert 0 < need < 200000 * 151936 * 2 // 10
    assert lib.nat_policy_loss_workspace_bytes(ctypes.byref(p), -1) == 0


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(nat, "_lib", None)
    monkeypatch.setattr(nat, "LIB_PATH", str(tmp_path / "absent.so"))
    with pytest.raises(nat.NatError):
        nat.load()
