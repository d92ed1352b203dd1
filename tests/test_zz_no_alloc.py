"""trl_pg_loss_fwd_static (the entry point for callers that cannot allocate device memory, e.g.
a trainer whose arena owns the whole GPU) must give what trl_pg_loss_fwd gives.  Collected
last on purpose: a run that stops at the first failure has then already run everything else."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _inputs(P, G, T, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    N = P * G * T
    lens = torch.randint(0, T + 1, (P * G,), generator=g, device="cuda", dtype=torch.int32)
    bnd = (lens.float() * torch.rand(P * G, generator=g, device="cuda")).to(torch.int32)
    t = torch.arange(T, device="cuda").repeat(P * G)
    L, Bd = lens.repeat_interleave(T), bnd.repeat_interleave(T)
    seg = torch.where(t < Bd, 1, torch.where(t < L, 2, 0)).to(torch.uint8)
    adv = torch.randn(P * G, generator=g, device="cuda").repeat_interleave(T) * (seg != 0)
    old = -torch.rand(N, generator=g, device="cuda") * 5
    logp = old + 0.15 * torch.randn(N, generator=g, device="cuda")
    return logp, old, adv, seg, lens


def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row():
    import paper_2510_17891_b200 as trl
    trl.load_library()
    # two calls in a row with different shapes and data: the second one runs over whatever
    # the first left in the shared scratch array
    # (the first case spans three partial-sum slots per rollout, the last one a single slot)
    from oracle import trl_oracle as orc
    for (P, G, T, seed) in ((2, 3, 40000, 3), (3, 5, 9000, 1), (2, 4, 300, 2)):
        logp, old, adv, seg, lens = _inputs(P, G, T, seed)
        ref_loss, ref_g, ref_stats = trl.trl_pg_loss_fwd(logp, old, adv, seg, lens, P, G, T, 0.2, 0.2, 0.1)
        loss = torch.full((1,), float("nan"), device="cuda")
        g = torch.full((P * G * T,), float("nan"), device="cuda")
        stats = torch.full((4,), float("nan"), device="cuda")
        before = torch.cuda.memory_allocated()
        trl.trl_pg_loss_fwd_static(logp, old, adv, seg, lens, P, G, T, loss, g, stats, 0.2, 0.2, 0.1)
        assert torch.cuda.memory_allocated() == before
        torch.cuda.synchronize()
        # same kernels, same order of summation: the tolerance of the loss parity tests is ample
        assert abs(float(loss) - float(ref_loss)) <= 1e-3 * abs(float(ref_loss)) + 1e-9
        np.testing.assert_allclose(g.cpu().numpy(), ref_g.cpu().numpy(), rtol=1e-6, atol=1e-12)
        np.testing.assert_allclose(stats.cpu().numpy(), ref_stats.cpu().numpy(), rtol=1e-6)
        # and against the fp64 oracle, at the tolerance of the loss parity tests
        f64 = lambda t: t.cpu().double().numpy()
        o_loss, o_g, o_stats = orc.pg_loss_fwd(f64(logp), f64(old), f64(adv), seg.cpu().numpy(), lens.cpu().numpy(), P, G, T)
        assert abs(float(loss) - o_loss) <= 1e-3 * abs(o_loss) + 1e-9
        assert np.linalg.norm(f64(g) - o_g) <= 1e-5 * np.linalg.norm(o_g)
        np.testing.assert_allclose(f64(stats), o_stats, rtol=1e-4, atol=1e-6)


def test_static_scratch_variant_rejects_oversize():
    import paper_2510_17891_b200 as trl
    P, G, T = 1, 60000, 32768         # 60000 * 2 tiles > 65536 slots
    dummy = torch.zeros(8, device="cuda")
    with pytest.raises(trl.TrlError, match="workspace too small"):
        trl.trl_pg_loss_fwd_static(dummy, dummy, dummy, dummy.to(torch.uint8), dummy.to(torch.int32), P, G, T,
                                   dummy, dummy, dummy)
