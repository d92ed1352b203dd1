"""trl_pg_step_fused_banded: dW finished band by band for data-parallel overlap.  One GPU: results
must equal trl_pg_step_fused bit for bit, and a band must not change after its event."""
import numpy as np
import pytest
import torch

from paper_2510_17891_b200 import synth, dp

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def trl():
    import paper_2510_17891_b200 as t
    t.load_library()
    return t


def _inputs(trl, w):
    batch = synth.make_batch(w, device=DEV)
    old_logp, old_lse = trl.trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], w.T)
    hrd = trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], w.P, w.G, w.T)
    return batch, (batch["hidden"], batch["W"], batch["ids"], batch["lens"], old_logp, old_lse, hrd["adv"], hrd["seg"],
                   w.P, w.G, w.T)


def _same(a, b):
    for k in ("logp", "lse", "g", "loss", "stats", "dHidden", "dW"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("shape", [(2, 4, 300, 320, 1000), (3, 6, 384, 512, 3000), (1, 2, 64, 64, 256)])
@pytest.mark.parametrize("use_hint", [True, False])
def test_banded_schedule_is_bit_identical_and_bands_are_final_at_their_events(trl, shape, use_hint):
    P, G, T, H, V = shape
    w = synth.scaled(synth.CONFIGS[2], name=f"banded_{V}", P=P, G=G, T=T, H=H, V=V, degenerate_frac=0.3)
    batch, args = _inputs(trl, w)
    if not use_hint:
        args = args[:5] + (None,) + args[6:]
    ref = trl.trl_pg_step_fused(*args)
    bands = trl.trl_dw_band_plan(V, H, 4)
    assert bands[0] == 0 and bands[-1] == V
    n = len(bands) - 1
    events = [torch.cuda.Event() for _ in range(n)]
    for e in events:
        e.record()
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    n_valid = int(batch["lens"].sum())
    snap = torch.full((V, H), float("nan"), device=DEV)
    side = torch.cuda.Stream()
    torch.cuda.synchronize()
    out = trl.trl_pg_step_fused_banded(*args, bands, events, rows_bound=n_valid, status=status)
    # a side stream copies each band as soon as its event has fired, while later bands still run
    for j in range(n):
        side.wait_event(events[j])
        with torch.cuda.stream(side):
            snap[bands[j]:bands[j + 1]].copy_(out["dW"][bands[j]:bands[j + 1]], non_blocking=True)
    torch.cuda.synchronize()
    trl.check_status(status)
    _same(out, ref)
    assert torch.equal(snap, out["dW"])
    assert all(e.query() for e in events)
    # no events, no bound: same again
    out2 = trl.trl_pg_step_fused_banded(*args, bands)
    torch.cuda.synchronize()
    _same(out2, ref)


def test_rows_bound_too_small_is_flagged_without_faulting(trl):
    w = synth.scaled(synth.CONFIGS[2], name="banded_bound", P=2, G=4, T=300, H=320, V=1000, len_lo=0.9)
    batch, args = _inputs(trl, w)
    n_valid = int(batch["lens"].sum())
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    trl.trl_pg_step_fused_banded(*args, trl.trl_dw_band_plan(w.V, w.H, 2), rows_bound=n_valid - 300, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << 10
    with pytest.raises(trl.TrlError, match="rows_bound"):
        trl.check_status(status)


def test_host_checks_of_the_band_arguments(trl):
    w = synth.scaled(synth.CONFIGS[2], name="banded_args", P=1, G=2, T=128, H=64, V=512)
    batch, args = _inputs(trl, w)
    for bad in ([0, 128, 512], [0, 256, 256, 512], [256, 512], [0, 256]):
        with pytest.raises(trl.TrlError, match="invalid argument"):
            trl.trl_pg_step_fused_banded(*args, bad)
    with pytest.raises(trl.TrlError, match="workspace"):
        trl.trl_pg_step_fused_banded(*args, [0, 256, 512], workspace=torch.empty(4096, dtype=torch.uint8, device=DEV))


def test_reducer_on_one_gpu_is_a_no_op_around_the_banded_call(trl):
    """world_size = 1: the reducer hands out events and a band split, starts nothing, and dW is the
    fused step's dW bit for bit."""
    w = synth.scaled(synth.CONFIGS[2], name="banded_dp1", P=2, G=4, T=200, H=256, V=1536)
    batch, args = _inputs(trl, w)
    ref = trl.trl_pg_step_fused(*args)
    dW = torch.empty(w.V, w.H, device=DEV)
    red = dp.BandedGradReducer(dW, trl.trl_dw_band_plan(w.V, w.H, 3), w.P)
    out = trl.trl_pg_step_fused_banded(*args, red.band_begin, red.events, out=dict(dW=dW))
    red.start(out["loss"])
    red.finish()
    torch.cuda.synchronize()
    assert out["dW"] is dW and torch.equal(dW, ref["dW"]) and torch.equal(out["loss"], ref["loss"])
