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


def test_misaligned_pointers_are_rejected_on_the_host_before_any_launch():
    """Every tensor the kernels touch with 16-byte accesses or TMA must be 16-byte aligned.  The
    pointers below are never dereferenced: a misaligned one must make the call return
    TRL_ERR_INVALID_ARG from its host-side checks, and the same call with aligned pointers but a
    zero-byte workspace must get past those checks and stop at TRL_ERR_WORKSPACE_TOO_SMALL."""
    import ctypes as C
    import paper_2510_17891_b200 as trl
    from paper_2510_17891_b200.binding import PgConfig
    lib = trl.load_library()
    base = 0x7f0000000000
    A = lambda k: C.c_void_p(base + 0x100000 * k)            # distinct, 256-byte aligned
    cfg = PgConfig(0.2, 0.2, 0.1, 0, 0)
    B, T, H, V, P, G = 4, 64, 64, 512, 2, 2
    INVALID, TOO_SMALL = 1, 4

    def logprobs(off=(), ws_bytes=0):
        a = [A(k) if k not in off else C.c_void_p(base + 0x100000 * k + 4) for k in range(8)]
        return lib.trl_token_logprobs(a[0], a[1], a[2], a[3], B, T, H, V, trl.TRL_BF16, a[4], a[5], a[6], ws_bytes, None, None)

    assert logprobs() == TOO_SMALL
    for k in (0, 1, 2, 4, 5):                                 # hidden, W, ids, logp, lse
        assert logprobs(off=(k,)) == INVALID, k
    assert logprobs(off=(6,), ws_bytes=1 << 40) == INVALID    # workspace

    def loss_fwd(off=(), ws_bytes=0):
        a = [A(k) if k not in off else C.c_void_p(base + 0x100000 * k + 4) for k in range(10)]
        return lib.trl_pg_loss_fwd(a[0], a[1], a[2], a[3], a[4], P, G, T, cfg, a[5], a[6], a[7], a[8], ws_bytes, None, None)

    assert loss_fwd() == TOO_SMALL
    for k in (0, 1, 2, 3, 6):                                 # logp, old_logp, adv, seg, g
        assert loss_fwd(off=(k,)) == INVALID, k
    assert loss_fwd(off=(8,), ws_bytes=1 << 30) == INVALID    # workspace (was unchecked before)

    def loss_bwd(off=(), ws_bytes=0):
        a = [A(k) if k not in off else C.c_void_p(base + 0x100000 * k + 4) for k in range(10)]
        return lib.trl_pg_loss_bwd(a[0], a[1], a[2], a[3], a[4], a[5], B, T, H, V, trl.TRL_BF16, a[6], a[7], a[8], ws_bytes, None, None)

    assert loss_bwd() == TOO_SMALL
    for k in (0, 1, 2, 4, 5, 6, 7):                           # hidden, W, ids, lse, g, dHidden, dW
        assert loss_bwd(off=(k,)) == INVALID, k

    def fused(off=(), ws_bytes=0):
        a = [A(k) if k not in off else C.c_void_p(base + 0x100000 * k + 4) for k in range(17)]
        return lib.trl_pg_step_fused(a[0], a[1], a[2], a[3], a[4], a[5], a[6], a[7], P, G, T, H, V, trl.TRL_BF16, cfg,
                                     a[8], a[9], a[10], a[11], a[12], a[13], a[14], a[15], ws_bytes, None, None)

    assert fused() == TOO_SMALL
    for k in (0, 1, 2, 4, 5, 6, 7, 8, 9, 11, 13, 14):         # every [B*T] and matrix argument
        assert fused(off=(k,)) == INVALID, k

    def hrd(off=()):
        a = [A(k) if k not in off else C.c_void_p(base + 0x100000 * k + 4) for k in range(11)]
        return lib.trl_hrd_advantages(a[0], a[1], a[2], a[3], P, G, T, 0, a[4], a[5], a[6], a[7], a[8], a[9], a[10], None, None)

    for k in (6, 7, 10):                                      # seg, adv (16 bytes), n_valid (8 bytes)
        assert hrd(off=(k,)) == INVALID, k

    def static(off=()):
        a = [A(k) if k not in off else C.c_void_p(base + 0x100000 * k + 4) for k in range(8)]
        return lib.trl_pg_loss_fwd_static(a[0], a[1], a[2], a[3], a[4], P, G, T, cfg, a[5], a[6], a[7], None, None)

    for k in (0, 1, 2, 3, 6):
        assert static(off=(k,)) == INVALID, k


def test_config_string_names_the_tuning_settings_and_follows_the_environment(lib):
    """Host-only: the settings string lists the library's own choices, and the environment knobs
    (read once per process, hence child processes) replace them."""
    import subprocess
    import sys
    code = "import paper_2510_17891_b200 as t; print(t.trl_config_string())"

    def run(**env):
        r = subprocess.run([sys.executable, "-c", code], cwd=ROOT, env=dict(os.environ, **env), capture_output=True, text=True)
        assert r.returncode == 0, r.stderr
        return dict(kv.split("=") for kv in r.stdout.split())

    base = run()
    assert base["cta_group_fwd"] == "1" and base["cta_group_bwd"] == "1"
    assert {k: int(v) for k, v in base.items() if k.startswith("raster_band")} == {
        "raster_band_lse": 32, "raster_band_e": 32, "raster_band_dh": 8, "raster_band_dw": 8}
    tuned = run(TRL_CTA_GROUP="2", TRL_RASTER_BAND_LSE="48", TRL_RASTER_BAND_DW="16", TRL_RASTER_BAND_DH="nonsense")
    assert tuned["cta_group_fwd"] == "2" and tuned["raster_band_lse"] == "48" and tuned["raster_band_dw"] == "16"
    assert tuned["raster_band_dh"] == "8" and tuned["raster_band_e"] == "32"


def test_bounds_checked_build_compiles_and_exports_the_same_symbols():
    from paper_2510_17891_b200 import build
    dbg = ctypes.CDLL(build.build(debug=True))
    for n in _declared():
        assert hasattr(dbg, n), n
    dbg.trl_status_string.restype = ctypes.c_char_p
    assert b"debug build" in dbg.trl_status_string(11)
