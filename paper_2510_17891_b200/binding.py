"""ctypes binding of libtrl.so: argument marshalling only."""
import ctypes
import os

import torch

TRL_F32, TRL_BF16 = 0, 1
TRL_CALL_TOKEN_LOGPROBS, TRL_CALL_PG_LOSS_FWD, TRL_CALL_PG_LOSS_BWD, TRL_CALL_PG_STEP_FUSED = 0, 1, 2, 3
_STATUS_BITS = {7: "index out of range (token id / len / bnd)", 8: "pipeline wait timed out",
                9: "lse_hint out of range", 10: "more valid rows than rows_bound",
                11: "store index outside its buffer (bounds-checked debug build)"}

_PKG = os.path.dirname(os.path.abspath(__file__))
_lib = None


class TrlError(RuntimeError):
    pass


class PgConfig(ctypes.Structure):
    """trl_pg_config: clip range and plan weight (paper: eps = 0.2, alpha = 0.1)."""
    _fields_ = [("eps_lo", ctypes.c_float), ("eps_hi", ctypes.c_float), ("alpha", ctypes.c_float),
                ("clip_form", ctypes.c_int), ("agg_mode", ctypes.c_int)]


def lib_path():
    """libtrl.so, or with TRL_DEBUG_BUILD=1 in the environment the bounds-checked build libtrl_debug.so
    (`python -m paper_2510_17891_b200.build --debug`)."""
    return os.path.join(_PKG, "libtrl_debug.so" if os.environ.get("TRL_DEBUG_BUILD") == "1" else "libtrl.so")


_vp, _sz, _i = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
_SIGNATURES = {
    "trl_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i]),
    "trl_workspace_bytes_min": (_sz, [_i, _i, _i, _i, _i, _i]),
    "trl_status_string": (ctypes.c_char_p, [_i]),
    "trl_kernel_launches": (ctypes.c_ulonglong, []),
    "trl_config_string": (ctypes.c_char_p, []),
    "trl_token_logprobs": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _sz, _vp, _vp]),
    "trl_hrd_advantages": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "trl_pg_loss_fwd": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, PgConfig, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "trl_pg_loss_fwd_static": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, PgConfig, _vp, _vp, _vp, _vp, _vp]),
    "trl_pg_step_fused": (_i, [_vp] * 8 + [_i] * 6 + [PgConfig] + [_vp] * 7 + [_vp, _sz, _vp, _vp]),
    "trl_pg_step_fused_banded": (_i, [_vp] * 8 + [_i] * 6 + [PgConfig] + [_vp] * 7 + [_i, _vp, _vp, _i] + [_vp, _sz, _vp, _vp]),
    "trl_pg_step_fused_banded_workspace_bytes": (_sz, [_i, _i, _i, _i, _i]),
    "trl_dw_band_plan": (_i, [_i, _i, _i, _vp]),
    "trl_pg_loss_bwd": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _vp, _vp, _vp, _sz, _vp, _vp]),
}


def exported_symbols():
    return sorted(_SIGNATURES)


def load_library():
    """Load libtrl.so (built in-tree by paper_2510_17891_b200.build).  Raises if absent."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise TrlError(f"{path} not found: build it with `python -m paper_2510_17891_b200.build` "
                           "(there is no fallback path)")
        lib = ctypes.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(rc, what):
    if rc != 0:
        raise TrlError(f"{what}: {load_library().trl_status_string(rc).decode()} (status {rc})")


def _dt(t):
    if t.dtype == torch.bfloat16:
        return TRL_BF16
    if t.dtype == torch.float32:
        return TRL_F32
    raise TrlError(f"unsupported dtype {t.dtype}")


def _dev(*ts):
    for t in ts:
        if t is not None and (not t.is_cuda or not t.is_contiguous()):
            raise TrlError("all tensors must be contiguous CUDA tensors")


def trl_workspace_bytes(which, B, T, H, V, dt):
    return load_library().trl_workspace_bytes(which, B, T, H, V, dt)


def trl_workspace_bytes_min(which, B, T, H, V, dt):
    return load_library().trl_workspace_bytes_min(which, B, T, H, V, dt)


def trl_status_string(code):
    return load_library().trl_status_string(code).decode()


def trl_config_string():
    return load_library().trl_config_string().decode()


def trl_kernel_launches():
    return load_library().trl_kernel_launches()


def _workspace(nbytes, device):
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def check_status(status):
    """Synchronising read of the device status word; raises on any device-detected error."""
    v = int(status.item())
    if v:
        msgs = [m for b, m in _STATUS_BITS.items() if v & (1 << b)]
        raise TrlError("device status: " + "; ".join(msgs or [hex(v)]))


def trl_token_logprobs(hidden, W, ids, lens, T, logp=None, lse=None, workspace=None, status=None, stream=None):
    """logp[n], lse[n] of the sampled tokens (see include/trl.h).  Returns (logp, lse)."""
    _dev(hidden, W, ids, lens, logp, lse, workspace, status)
    B = lens.numel()
    V, H = W.shape
    dt = _dt(hidden)
    if logp is None:
        logp = torch.empty(B * T, dtype=torch.float32, device=hidden.device)
    if lse is None:
        lse = torch.empty(B * T, dtype=torch.float32, device=hidden.device)
    if workspace is None:
        workspace = _workspace(trl_workspace_bytes(TRL_CALL_TOKEN_LOGPROBS, B, T, H, V, dt), hidden.device)
    rc = load_library().trl_token_logprobs(_ptr(hidden), _ptr(W), _ptr(ids), _ptr(lens), B, T, H, V, dt,
                                           _ptr(logp), _ptr(lse), _ptr(workspace), workspace.numel(),
                                           _ptr(status), _stream(stream))
    _check(rc, "trl_token_logprobs")
    return logp, lse


def trl_hrd_advantages(r_plan, r_code, lens, bnd, P, G, T, adv_mode=0, out=None, status=None, stream=None):
    """HRD advantages and segment labels.  Returns a dict of device tensors."""
    _dev(r_plan, r_code, lens, bnd, status)
    B, dev = P * G, r_plan.device
    if out is None:
        out = dict(A_plan=torch.empty(B, dtype=torch.float32, device=dev),
                   A_code=torch.empty(B, dtype=torch.float32, device=dev),
                   seg=torch.empty(B * T, dtype=torch.uint8, device=dev),
                   adv=torch.empty(B * T, dtype=torch.float32, device=dev),
                   n_plan=torch.empty(B, dtype=torch.int32, device=dev),
                   n_code=torch.empty(B, dtype=torch.int32, device=dev),
                   n_valid=torch.empty(1, dtype=torch.int64, device=dev))
    rc = load_library().trl_hrd_advantages(_ptr(r_plan), _ptr(r_code), _ptr(lens), _ptr(bnd), P, G, T, adv_mode,
                                           _ptr(out["A_plan"]), _ptr(out["A_code"]), _ptr(out["seg"]),
                                           _ptr(out["adv"]), _ptr(out["n_plan"]), _ptr(out["n_code"]),
                                           _ptr(out["n_valid"]), _ptr(status), _stream(stream))
    _check(rc, "trl_hrd_advantages")
    return out


def trl_pg_loss_fwd(logp, old_logp, adv, seg, lens, P, G, T, eps_lo=0.2, eps_hi=0.2, alpha=0.1,
                    loss=None, g=None, stats=None, workspace=None, status=None, stream=None, clip_form=0, agg_mode=0):
    """Clipped surrogate loss, d loss/d logp and clip statistics.  Returns (loss, g, stats)."""
    _dev(logp, old_logp, adv, seg, lens, loss, g, stats, workspace, status)
    dev = logp.device
    if loss is None:
        loss = torch.empty(1, dtype=torch.float32, device=dev)
    if g is None:
        g = torch.empty(P * G * T, dtype=torch.float32, device=dev)
    if stats is None:
        stats = torch.empty(4, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = _workspace(trl_workspace_bytes(TRL_CALL_PG_LOSS_FWD, P * G, T, 1, 1, TRL_F32), dev)
    rc = load_library().trl_pg_loss_fwd(_ptr(logp), _ptr(old_logp), _ptr(adv), _ptr(seg), _ptr(lens), P, G, T,
                                        PgConfig(eps_lo, eps_hi, alpha, clip_form, agg_mode), _ptr(loss), _ptr(g),
                                        _ptr(stats), _ptr(workspace), workspace.numel(), _ptr(status), _stream(stream))
    _check(rc, "trl_pg_loss_fwd")
    return loss, g, stats


def trl_pg_loss_fwd_static(logp, old_logp, adv, seg, lens, P, G, T, loss, g, stats, eps_lo=0.2, eps_hi=0.2,
                           alpha=0.1, status=None, stream=None, clip_form=0, agg_mode=0):
    """trl_pg_loss_fwd for callers that cannot allocate: the scratch is a fixed array inside the
    library, and this wrapper allocates nothing either, so `loss` [1], `g` [P*G*T] and `stats`
    [4] (or None) must be passed in.  Limit P*G*ceil(T/16384) <= 65536.  Calls that may overlap
    on the GPU must not share a device.  Returns (loss, g, stats)."""
    _dev(logp, old_logp, adv, seg, lens, loss, g, stats, status)
    rc = load_library().trl_pg_loss_fwd_static(_ptr(logp), _ptr(old_logp), _ptr(adv), _ptr(seg), _ptr(lens), P, G, T,
                                               PgConfig(eps_lo, eps_hi, alpha, clip_form, agg_mode), _ptr(loss), _ptr(g),
                                               _ptr(stats), _ptr(status), _stream(stream))
    _check(rc, "trl_pg_loss_fwd_static")
    return loss, g, stats


def trl_pg_loss_bwd(hidden, W, ids, lens, lse, g, T, dHidden=None, dW=None, workspace=None, status=None,
                    stream=None):
    """dHidden [N,H] (input dtype) and dW [V,H] fp32.  Returns (dHidden, dW)."""
    _dev(hidden, W, ids, lens, lse, g, dHidden, dW, workspace, status)
    B = lens.numel()
    V, H = W.shape
    dt = _dt(hidden)
    if dHidden is None:
        dHidden = torch.empty_like(hidden)
    if dW is None:
        dW = torch.empty(V, H, dtype=torch.float32, device=hidden.device)
    if workspace is None:
        workspace = _workspace(trl_workspace_bytes(TRL_CALL_PG_LOSS_BWD, B, T, H, V, dt), hidden.device)
    rc = load_library().trl_pg_loss_bwd(_ptr(hidden), _ptr(W), _ptr(ids), _ptr(lens), _ptr(lse), _ptr(g),
                                        B, T, H, V, dt, _ptr(dHidden), _ptr(dW), _ptr(workspace),
                                        workspace.numel(), _ptr(status), _stream(stream))
    _check(rc, "trl_pg_loss_bwd")
    return dHidden, dW


def trl_pg_step_fused(hidden, W, ids, lens, old_logp, lse_hint, adv, seg, P, G, T, eps_lo=0.2, eps_hi=0.2, alpha=0.1,
                      out=None, workspace=None, status=None, stream=None, clip_form=0, agg_mode=0):
    """Fused policy scoring + surrogate loss + backward (see include/trl.h).  `lse_hint` may be
    None.  Returns a dict with logp, lse, loss, g, stats, dHidden, dW."""
    _dev(hidden, W, ids, lens, old_logp, lse_hint, adv, seg, workspace, status)
    B = lens.numel()
    V, H = W.shape
    dt = _dt(hidden)
    dev = hidden.device
    o = {} if out is None else out
    f32 = dict(dtype=torch.float32, device=dev)
    for k, shape in (("logp", B * T), ("lse", B * T), ("g", B * T), ("loss", 1), ("stats", 4)):
        if o.get(k) is None:
            o[k] = torch.empty(shape, **f32)
    if o.get("dHidden") is None:
        o["dHidden"] = torch.empty_like(hidden)
    if o.get("dW") is None:
        o["dW"] = torch.empty(V, H, **f32)
    if workspace is None:
        workspace = _workspace(trl_workspace_bytes(TRL_CALL_PG_STEP_FUSED, B, T, H, V, dt), dev)
    rc = load_library().trl_pg_step_fused(_ptr(hidden), _ptr(W), _ptr(ids), _ptr(lens), _ptr(old_logp), _ptr(lse_hint),
                                          _ptr(adv), _ptr(seg), P, G, T, H, V, dt,
                                          PgConfig(eps_lo, eps_hi, alpha, clip_form, agg_mode),
                                          _ptr(o["logp"]), _ptr(o["lse"]), _ptr(o["loss"]), _ptr(o["g"]),
                                          _ptr(o["stats"]), _ptr(o["dHidden"]), _ptr(o["dW"]), _ptr(workspace),
                                          workspace.numel(), _ptr(status), _stream(stream))
    _check(rc, "trl_pg_step_fused")
    return o


def trl_dw_band_plan(V, H, n_bands_wanted):
    """Band boundaries (a list of n + 1 vocabulary rows) for trl_pg_step_fused_banded."""
    buf = (ctypes.c_int32 * (n_bands_wanted + 1))()
    n = load_library().trl_dw_band_plan(V, H, n_bands_wanted, buf)
    if n <= 0:
        raise TrlError("trl_dw_band_plan: invalid arguments")
    return [int(buf[i]) for i in range(n + 1)]


def trl_pg_step_fused_banded_workspace_bytes(B, T, H, V, rows_bound=0):
    return load_library().trl_pg_step_fused_banded_workspace_bytes(B, T, H, V, rows_bound)


def trl_pg_step_fused_banded(hidden, W, ids, lens, old_logp, lse_hint, adv, seg, P, G, T, band_begin, band_events=None,
                             rows_bound=0, eps_lo=0.2, eps_hi=0.2, alpha=0.1, out=None, workspace=None, status=None,
                             stream=None, clip_form=0, agg_mode=0):
    """trl_pg_step_fused with dW finished band by band (see include/trl.h).  `band_begin` is a list
    of n + 1 rows from trl_dw_band_plan; `band_events` a list of n recorded-at-least-once
    torch.cuda.Event objects (or None): event j is recorded on the stream when band j of dW is final."""
    _dev(hidden, W, ids, lens, old_logp, lse_hint, adv, seg, workspace, status)
    B = lens.numel()
    V, H = W.shape
    dt = _dt(hidden)
    dev = hidden.device
    o = {} if out is None else out
    f32 = dict(dtype=torch.float32, device=dev)
    for k, shape in (("logp", B * T), ("lse", B * T), ("g", B * T), ("loss", 1), ("stats", 4)):
        if o.get(k) is None:
            o[k] = torch.empty(shape, **f32)
    if o.get("dHidden") is None:
        o["dHidden"] = torch.empty_like(hidden)
    if o.get("dW") is None:
        o["dW"] = torch.empty(V, H, **f32)
    if workspace is None:
        workspace = _workspace(trl_pg_step_fused_banded_workspace_bytes(B, T, H, V, rows_bound), dev)
    n = len(band_begin) - 1
    bb = (ctypes.c_int32 * (n + 1))(*band_begin)
    ev = None
    if band_events is not None:
        ev = (ctypes.c_void_p * n)(*[None if e is None else e.cuda_event for e in band_events])
    rc = load_library().trl_pg_step_fused_banded(_ptr(hidden), _ptr(W), _ptr(ids), _ptr(lens), _ptr(old_logp), _ptr(lse_hint),
                                                 _ptr(adv), _ptr(seg), P, G, T, H, V, dt,
                                                 PgConfig(eps_lo, eps_hi, alpha, clip_form, agg_mode),
                                                 _ptr(o["logp"]), _ptr(o["lse"]), _ptr(o["loss"]), _ptr(o["g"]),
                                                 _ptr(o["stats"]), _ptr(o["dHidden"]), _ptr(o["dW"]),
                                                 n, bb, ev, rows_bound, _ptr(workspace), workspace.numel(), _ptr(status),
                                                 _stream(stream))
    _check(rc, "trl_pg_step_fused_banded")
    return o


def hrd_pg_step(batch, P, G, T, eps_lo=0.2, eps_hi=0.2, alpha=0.1, adv_mode=0, old_logp=None, bufs=None,
                status=None, stream=None, fused=False, use_hint=True, clip_form=0, agg_mode=0):
    """One pass of the whole path by calling the five C entry points in order: score under the
    current and the old policy, HRD advantages, surrogate loss, backward.  `bufs` may carry
    preallocated outputs / workspaces (keys as returned).  No arithmetic happens here."""
    bufs = {} if bufs is None else bufs
    if fused:
        old_lse = None
        if old_logp is None:
            old_logp, old_lse = trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], T,
                                                   bufs.get("old_logp"), bufs.get("old_lse"), bufs.get("ws_fwd"),
                                                   status, stream)
        hrd = trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], P, G, T, adv_mode,
                                 bufs.get("hrd"), status, stream)
        o = trl_pg_step_fused(batch["hidden"], batch["W"], batch["ids"], batch["lens"], old_logp,
                              old_lse if use_hint else None, hrd["adv"], hrd["seg"], P, G, T, eps_lo, eps_hi, alpha,
                              bufs.get("fused_out"), bufs.get("ws_fused"), status, stream, clip_form, agg_mode)
        return dict(old_logp=old_logp, hrd=hrd, **o)
    logp, lse = trl_token_logprobs(batch["hidden"], batch["W"], batch["ids"], batch["lens"], T,
                                   bufs.get("logp"), bufs.get("lse"), bufs.get("ws_fwd"), status, stream)
    if old_logp is None:
        old_logp, _ = trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], T,
                                         bufs.get("old_logp"), bufs.get("old_lse"), bufs.get("ws_fwd"), status, stream)
    hrd = trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], P, G, T, adv_mode,
                             bufs.get("hrd"), status, stream)
    loss, g, stats = trl_pg_loss_fwd(logp, old_logp, hrd["adv"], hrd["seg"], batch["lens"], P, G, T, eps_lo, eps_hi,
                                     alpha, bufs.get("loss"), bufs.get("g"), bufs.get("stats"), bufs.get("ws_loss"),
                                     status, stream, clip_form, agg_mode)
    dHidden, dW = trl_pg_loss_bwd(batch["hidden"], batch["W"], batch["ids"], batch["lens"], lse, g, T,
                                  bufs.get("dHidden"), bufs.get("dW"), bufs.get("ws_bwd"), status, stream)
    return dict(logp=logp, lse=lse, old_logp=old_logp, hrd=hrd, loss=loss, g=g, stats=stats, dHidden=dHidden, dW=dW)
