"""Stand-ins for a memory checker: guard bands around every output and workspace must stay
untouched, and repeated runs must give bit-identical results (no data race, no use of
uninitialised scratch)."""
import pytest
import torch

from paper_2510_17891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 4096           # bytes on each side
SENTINEL = 0xA5


class Guarded:
    """A tensor view inside a byte buffer with sentinel-filled guard bands on both sides."""

    def __init__(self, nbytes, dtype=torch.uint8, shape=None):
        nbytes = (int(nbytes) + 255) // 256 * 256
        self.raw = torch.full((nbytes + 2 * GUARD,), SENTINEL, dtype=torch.uint8, device=DEV)
        body = self.raw[GUARD:GUARD + nbytes]
        self.t = body.view(dtype) if shape is None else body.view(dtype)[: int(torch.tensor(shape).prod())].view(*shape)
        self.nbytes = nbytes

    def intact(self):
        return bool((self.raw[:GUARD] == SENTINEL).all()) and bool((self.raw[GUARD + self.nbytes:] == SENTINEL).all())


@pytest.fixture(scope="module")
def trl():
    import paper_2510_17891_b200 as t
    t.load_library()
    return t


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_no_write_outside_outputs_and_workspaces(trl, dtype):
    # ragged shape: partial last row block, partial last vocabulary tile, H not a multiple of 64
    w = synth.scaled(synth.CONFIGS[2], name=f"guard_{dtype}", P=2, G=3, T=200, H=72, V=1000, dtype=dtype, len_lo=0.1)
    b = synth.make_batch(w, device=DEV)
    dt = trl.TRL_BF16 if dtype == "bf16" else trl.TRL_F32
    esz = 2 if dtype == "bf16" else 4
    N, B, T, H, V = w.N, w.B, w.T, w.H, w.V
    f32 = torch.float32
    g = {k: Guarded(N * 4, f32, (N,)) for k in ("logp", "lse", "old_logp", "old_lse", "g", "adv")}
    g.update(loss=Guarded(4, f32, (1,)), stats=Guarded(16, f32, (4,)), seg=Guarded(N, torch.uint8, (N,)),
             A_plan=Guarded(B * 4, f32, (B,)), A_code=Guarded(B * 4, f32, (B,)),
             n_plan=Guarded(B * 4, torch.int32, (B,)), n_code=Guarded(B * 4, torch.int32, (B,)),
             n_valid=Guarded(8, torch.int64, (1,)),
             dHidden=Guarded(N * H * esz, b["hidden"].dtype, (N, H)), dW=Guarded(V * H * 4, f32, (V, H)),
             ws_fwd=Guarded(trl.trl_workspace_bytes(trl.TRL_CALL_TOKEN_LOGPROBS, B, T, H, V, dt)),
             ws_loss=Guarded(trl.trl_workspace_bytes(trl.TRL_CALL_PG_LOSS_FWD, B, T, 1, 1, trl.TRL_F32)),
             ws_bwd=Guarded(trl.trl_workspace_bytes_min(trl.TRL_CALL_PG_LOSS_BWD, B, T, H, V, dt)),
             ws_fused=Guarded(trl.trl_workspace_bytes_min(trl.TRL_CALL_PG_STEP_FUSED, B, T, H, V, dt)))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    hrd = {k: g[k].t for k in ("A_plan", "A_code", "seg", "adv", "n_plan", "n_code", "n_valid")}
    trl.trl_token_logprobs(b["hidden"], b["W"], b["ids"], b["lens"], T, g["logp"].t, g["lse"].t, g["ws_fwd"].t, status)
    trl.trl_token_logprobs(b["hidden_old"], b["W_old"], b["ids"], b["lens"], T, g["old_logp"].t, g["old_lse"].t,
                           g["ws_fwd"].t, status)
    trl.trl_hrd_advantages(b["r_plan"], b["r_code"], b["lens"], b["bnd"], w.P, w.G, T, 0, hrd, status)
    trl.trl_pg_loss_fwd(g["logp"].t, g["old_logp"].t, g["adv"].t, g["seg"].t, b["lens"], w.P, w.G, T, 0.2, 0.2, 0.1,
                        g["loss"].t, g["g"].t, g["stats"].t, g["ws_loss"].t, status)
    trl.trl_pg_loss_bwd(b["hidden"], b["W"], b["ids"], b["lens"], g["lse"].t, g["g"].t, T, g["dHidden"].t, g["dW"].t,
                        g["ws_bwd"].t, status)
    out = {k: g[k].t for k in ("logp", "lse", "g", "loss", "stats", "dHidden", "dW")}
    trl.trl_pg_step_fused(b["hidden"], b["W"], b["ids"], b["lens"], g["old_logp"].t, g["old_lse"].t, g["adv"].t,
                          g["seg"].t, w.P, w.G, T, 0.2, 0.2, 0.1, out, g["ws_fused"].t, status)
    trl.trl_pg_step_fused(b["hidden"], b["W"], b["ids"], b["lens"], g["old_logp"].t, None, g["adv"].t,
                          g["seg"].t, w.P, w.G, T, 0.2, 0.2, 0.1, out,
                          Guarded(trl.trl_workspace_bytes(trl.TRL_CALL_PG_STEP_FUSED, B, T, H, V, dt)).t, status)
    torch.cuda.synchronize()
    trl.check_status(status)
    broken = [k for k, v in g.items() if not v.intact()]
    assert not broken, broken
    assert torch.isfinite(g["dW"].t).all() and torch.isfinite(g["loss"].t).all()


def test_repeated_runs_are_bit_identical(trl):
    w = synth.scaled(synth.CONFIGS[2], name="determinism", P=3, G=4, T=500, H=512, V=4096, degenerate_frac=0.34)
    b = synth.make_batch(w, device=DEV)
    runs = []
    for fused in (True, True, False, False):
        # poison fresh outputs/workspaces differently each time: results must not depend on them
        o = trl.hrd_pg_step(b, w.P, w.G, w.T, fused=fused)
        torch.cuda.synchronize()
        runs.append({k: o[k].clone() for k in ("logp", "lse", "old_logp", "loss", "g", "stats", "dHidden", "dW")})
        torch.cuda.empty_cache()
        junk = torch.full((64 << 20,), float("nan"), device=DEV)    # dirty the allocator's free blocks
        del junk
    for a, c in ((runs[0], runs[1]), (runs[2], runs[3])):
        for k in a:
            assert torch.equal(a[k], c[k]), k


def test_step_replays_from_a_cuda_graph(trl):
    """The calls enqueue work on the caller's stream only (no allocation, no host sync), so a
    whole step can be captured once and replayed with new input values in the same buffers."""
    w = synth.scaled(synth.CONFIGS[2], name="graph", P=2, G=4, T=300, H=256, V=2048)
    b = synth.make_batch(w, device=DEV)
    B, T, H, V = w.B, w.T, w.H, w.V
    f32 = dict(dtype=torch.float32, device=DEV)
    ws = lambda call: torch.empty(trl.trl_workspace_bytes(call, B, T, H, V, trl.TRL_BF16), dtype=torch.uint8, device=DEV)
    bufs = dict(old_logp=torch.empty(w.N, **f32), old_lse=torch.empty(w.N, **f32), ws_fwd=ws(trl.TRL_CALL_TOKEN_LOGPROBS),
                ws_fused=ws(trl.TRL_CALL_PG_STEP_FUSED),
                fused_out=dict(logp=torch.empty(w.N, **f32), lse=torch.empty(w.N, **f32), g=torch.empty(w.N, **f32),
                               loss=torch.empty(1, **f32), stats=torch.empty(4, **f32),
                               dHidden=torch.empty_like(b["hidden"]), dW=torch.empty(V, H, **f32)))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    out = trl.hrd_pg_step(b, w.P, w.G, T, fused=True, bufs=bufs, status=status)       # eager (also warms up)
    bufs["hrd"] = out["hrd"]
    torch.cuda.synchronize()
    eager = {k: out[k].clone() for k in ("logp", "loss", "dHidden", "dW")}
    stream = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(stream):
        with torch.cuda.graph(graph, stream=stream):
            trl.hrd_pg_step(b, w.P, w.G, T, fused=True, bufs=bufs, status=status, stream=stream)
    for k in ("logp", "loss", "dHidden", "dW"):
        out[k].fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    for k in eager:
        assert torch.equal(out[k], eager[k]), k
    # new inputs in the same buffers: the replay follows them
    b2 = synth.make_batch(synth.scaled(w, name="graph2"), device=DEV)
    for k in ("hidden", "W", "W_old", "ids", "lens", "bnd", "r_plan", "r_code"):
        b[k].copy_(b2[k])
    graph.replay()
    torch.cuda.synchronize()
    replayed = {k: out[k].clone() for k in eager}
    ref = trl.hrd_pg_step(b2, w.P, w.G, T, fused=True, status=status)
    torch.cuda.synchronize()
    trl.check_status(status)
    for k in eager:
        assert torch.equal(replayed[k], ref[k]), k
