"""The C-ABI library builds, loads without a GPU and exports every symbol include/trl.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2510_17891_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def _declared():
    src = open(os.path.join(ROOT, "include", "trl.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(trl_[a-z_]+)\s*\(", src)))


def test_header_declares_the_four_calls():
    names = _declared()
    for n in ("trl_token_logprobs", "trl_hrd_advantages", "trl_pg_loss_fwd", "trl_pg_loss_bwd"):
        assert n in names


def test_every_declared_symbol_is_exported(lib):
    for n in _declared():
        assert hasattr(lib, n), n


def test_binding_covers_every_declared_symbol():
    import paper_2510_17891_b200 as trl
    assert set(_declared()) <= set(trl.exported_symbols())
    for n in _declared():
        assert hasattr(trl, n)


def test_host_only_calls(lib):
    import paper_2510_17891_b200 as trl
    assert trl.trl_status_string(0) == "ok"
    assert "workspace" in trl.trl_status_string(4)
    # workspace sizes: monotone in the shape, min <= recommended, 0 for nonsense
    a = trl.trl_workspace_bytes(trl.TRL_CALL_PG_LOSS_BWD, 64, 2048, 4096, 151936, trl.TRL_BF16)
    b = trl.trl_workspace_bytes_min(trl.TRL_CALL_PG_LOSS_BWD, 64, 2048, 4096, 151936, trl.TRL_BF16)
    assert 0 < b <= a < 64 * 2 ** 30
    assert trl.trl_workspace_bytes(trl.TRL_CALL_TOKEN_LOGPROBS, 0, 5, 5, 5, trl.TRL_BF16) == 0
    assert trl.trl_workspace_bytes(99, 1, 1, 8, 8, trl.TRL_BF16) == 0
    # null pointers are rejected on the host before anything is launched
    rc = lib.trl_hrd_advantages(None, None, None, None, 1, 1, 1, 0, None, None, None, None, None, None, None, None, None)
    assert rc == 1


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2510_17891_b200.binding as binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "lib_path", lambda: "/nonexistent/libtrl.so")
    with pytest.raises(binding.TrlError):
        binding.load_library()
