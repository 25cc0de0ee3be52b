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
    assert lib.nat_select(ctypes.byref(bad), 2, 4096, 0, 4096, 4096, None, None) == -1
    assert b"0 < p <= 1" in lib.nat_last_error()
    assert lib.nat_grpo_adv(1, 0, None, 1e-6, None, None) == -1
    assert lib.nat_compact_workspace_bytes(0) == 256
    assert lib.nat_compact_workspace_bytes(4096 * 3 + 1) >= 5 * 4
    p = nat.loss_params(4096, 151936, nat.NAT_BF16, 128)
    need = lib.nat_policy_loss_workspace_bytes(ctypes.byref(p), 200000)
    # bounded scratch: far below the 200000 x 151936 logits a naive path would store
    assert 0 < need < 200000 * 151936 * 2 // 10
    assert lib.nat_policy_loss_workspace_bytes(ctypes.byref(p), -1) == 0
    # the float32 path covers d <= 1024 only: no workspace size, and the call is refused
    big = nat.loss_params(2048, 512, nat.NAT_F32, 8)
    assert lib.nat_policy_loss_workspace_bytes(ctypes.byref(big), 100) == 0
    ok = nat.loss_params(1024, 512, nat.NAT_F32, 8)
    assert lib.nat_policy_loss_workspace_bytes(ctypes.byref(ok), 100) > 0
    args = [ctypes.byref(big)] + [4096] * 10 + [100] + [4096] * 4 + [1 << 20, None]
    assert lib.nat_policy_loss_fwd(*args) == -2
    assert b"d <= 1024" in lib.nat_last_error()


def test_misaligned_buffers_are_refused_before_any_launch():
    """mask, pi, surv and q are read and written with 16-byte accesses; a pointer off that
    boundary must come back as an error, never as a misaligned-address fault."""
    lib = nat.load()
    sp = nat.select_params("urs", p=0.5)
    a16, odd = 4096, 4096 + 4          # fake device addresses: nothing is dereferenced
    assert lib.nat_select(ctypes.byref(sp), 2, a16, 64, odd, a16, None, None) == -1
    assert b"16-byte aligned" in lib.nat_last_error()
    assert lib.nat_select(ctypes.byref(sp), 2, a16, 64, a16, odd, None, None) == -1
    bad = nat.select_params("urs", p=0.5, resp_base=-1)
    assert lib.nat_select(ctypes.byref(bad), 2, a16, 64, a16, a16, None, None) == -1
    assert b"resp_base" in lib.nat_last_error()
    assert lib.nat_compact(2, a16, 64, odd, a16, a16, a16, a16, 64, a16, 1 << 20, None) == -1
    assert b"16-byte aligned" in lib.nat_last_error()
    assert lib.nat_compact_static(2, a16, 64, odd, a16, a16, a16, a16, 64, None) == -1
    assert lib.nat_select_survival(2, a16, 64, odd, 0, 0, 0, a16, a16, None) == -1
    need = lib.nat_select_cutlaw_workspace_bytes(2, 64)
    assert need >= 2 * 8 + 3 * 8 and need % 256 == 0
    assert lib.nat_select_cutlaw(2, a16, 64, odd, 0, 0, 0, a16, a16, a16, a16, need, None) == -1
    assert lib.nat_select_cutlaw(2, a16, 64, a16, 0, 0, 0, a16, a16, a16, a16, need - 1, None) == -3
    assert lib.nat_select_cutlaw(2, a16, 64, a16, 0, 0, -1, a16, a16, a16, a16, need, None) == -1
    assert lib.nat_compact_prefix(2, a16, 64, None, a16, a16, a16, a16, 64, None) == -1
    assert lib.nat_poll_status(None, None, None) == -1


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(nat, "_lib", None)
    monkeypatch.setattr(nat, "LIB_PATH", str(tmp_path / "absent.so"))
    with pytest.raises(nat.NatError):
        nat.load()
