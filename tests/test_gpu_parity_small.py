"""CUDA path vs fp64 oracle, element by element, on shapes the oracle finishes in seconds.
All calls go through the C ABI (ctypes binding)."""
import numpy as np
import pytest
import torch

from oracle import trl_oracle as orc
from paper_2510_17891_b200 import synth
from tests._util import f64, oracle_inputs, rel_fro, TOL_LOGP, TOL_LOSS, TOL_GRAD

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def trl():
    import paper_2510_17891_b200 as t
    t.load_library()
    assert torch.cuda.is_available()
    return t


def run_and_compare(trl, w, batch=None, explicit_old=False, alpha=0.1, eps=0.2, adv_mode=0, fused=False,
                    use_hint=True, clip_form=0, agg_mode=0, eps_hi=None):
    eps_hi = eps if eps_hi is None else eps_hi
    dev = "cuda:0"
    batch = synth.make_batch(w, device=dev) if batch is None else batch
    oi = oracle_inputs(batch)
    old_logp_o = None
    old_logp_g = None
    if explicit_old:      # old logp = oracle logp + N(0, sigma): an input to both sides
        lp, _ = orc.token_logprobs(oi["hidden"], oi["W"], oi["ids"], oi["lens"], w.T)
        old_logp_o = (lp + oi["old_noise"]).astype(np.float32).astype(np.float64)
        old_logp_g = torch.tensor(old_logp_o, dtype=torch.float32, device=dev)
    ref = orc.full_step(oi["hidden"], oi["W"], oi["hidden_old"], oi["W_old"], oi["ids"], oi["lens"], oi["bnd"],
                        oi["r_plan"], oi["r_code"], w.P, w.G, w.T, eps, eps_hi, alpha, adv_mode, old_logp=old_logp_o,
                        clip_form=clip_form, agg_mode=agg_mode)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out = trl.hrd_pg_step(batch, w.P, w.G, w.T, eps, eps_hi, alpha, adv_mode, old_logp=old_logp_g, status=status,
                          fused=fused, use_hint=use_hint, clip_form=clip_form, agg_mode=agg_mode)
    torch.cuda.synchronize()
    trl.check_status(status)
    hrd = out["hrd"]
    # integers: bit exact
    np.testing.assert_array_equal(hrd["seg"].cpu().numpy(), ref["seg"])
    np.testing.assert_array_equal(hrd["n_plan"].cpu().numpy(), ref["n_plan"])
    np.testing.assert_array_equal(hrd["n_code"].cpu().numpy(), ref["n_code"])
    assert int(hrd["n_valid"].item()) == ref["n_valid"]
    np.testing.assert_allclose(f64(hrd["A_plan"]), ref["A_plan"], rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(f64(hrd["A_code"]), ref["A_code"], rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(f64(hrd["adv"]), ref["adv"], rtol=1e-6, atol=1e-7)
    # floating point
    assert np.abs(f64(out["logp"]) - ref["logp"]).max() <= TOL_LOGP
    assert np.abs(f64(out["lse"]) - ref["lse"]).max() <= TOL_LOGP
    if not explicit_old:
        assert np.abs(f64(out["old_logp"]) - ref["old_logp"]).max() <= TOL_LOGP
    assert abs(float(out["loss"]) - ref["loss"]) <= TOL_LOSS * abs(ref["loss"]) + 1e-9
    valid = ref["seg"] != 0
    assert not f64(out["g"])[~valid].any() and not f64(out["logp"])[~valid].any()
    assert rel_fro(f64(out["g"]), ref["g"]) <= TOL_GRAD
    dH = f64(out["dHidden"])
    assert not dH[~valid].any()
    if np.linalg.norm(ref["dHidden"]) > 0:
        assert rel_fro(dH, ref["dHidden"]) <= TOL_GRAD
        assert rel_fro(f64(out["dW"]), ref["dW"]) <= TOL_GRAD
    else:
        assert not dH.any() and not f64(out["dW"]).any()
    st = f64(out["stats"])
    np.testing.assert_allclose(st[:3], ref["stats"][:3], atol=2e-3)
    assert st[3] == ref["stats"][3]
    return out, ref


def test_config0_f32_end_to_end(trl):
    run_and_compare(trl, synth.CONFIGS[0])
    run_and_compare(trl, synth.CONFIGS[0], explicit_old=True)


def test_config0_literal_boundary_reading(trl):
    run_and_compare(trl, synth.scaled(synth.CONFIGS[0], name="cfg0_bnd_of_T", bnd_of_T=True), explicit_old=True)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_ragged_multi_tile(trl, dtype):
    # rows: 3 blocks per rollout with a ragged tail; K: 5 k-blocks; V: 4 tiles, the last one partial
    w = synth.scaled(synth.CONFIGS[2], name=f"twin_ragged_{dtype}", P=2, G=4, T=300, H=320, V=1000, dtype=dtype)
    run_and_compare(trl, w)
    run_and_compare(trl, w, explicit_old=True, alpha=0.5, eps=0.1)


def test_bf16_many_tiles_real_plan_reward(trl):
    # more tiles than SMs in the forward, several waves, 2 raster bands; non-binary plan reward
    w = synth.scaled(synth.CONFIGS[2], name="twin_wide", P=3, G=6, T=384, H=512, V=3000, real_plan_reward=True,
                     len_lo=0.1)
    run_and_compare(trl, w)


def test_long_reasoning_twin_bf16(trl):
    w = synth.scaled(synth.CONFIGS[3], name="twin_cfg3", P=2, G=8, T=512, H=256, V=2048)
    run_and_compare(trl, w)
    run_and_compare(trl, synth.scaled(w, name="twin_cfg3_lit", bnd_of_T=True))


def test_sweep_twin_degenerate_groups_and_std_mode(trl):
    for G in (4, 16):
        w = synth.scaled(synth.CONFIGS[2], name=f"twin_sweep_G{G}", P=64 // G, G=G, T=128, H=256, V=1536,
                         degenerate_frac=0.25)
        run_and_compare(trl, w)
    run_and_compare(trl, synth.scaled(synth.CONFIGS[2], name="twin_std", P=4, G=4, T=128, H=256, V=1024), adv_mode=1)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_edge_cases_empty_rollouts_and_boundaries(trl, dtype):
    w = synth.scaled(synth.CONFIGS[2], name=f"edge_{dtype}", P=2, G=4, T=160, H=128, V=512, dtype=dtype)
    batch = synth.make_batch(w, device="cuda:0")
    lens = torch.tensor([0, 160, 1, 128, 129, 77, 0, 5], dtype=torch.int32)
    bnd = torch.tensor([0, 0, 1, 128, 64, 77, 0, 2], dtype=torch.int32)   # no plan / no code / both
    batch["lens"], batch["bnd"] = lens.cuda(), bnd.cuda()
    run_and_compare(trl, w, batch=batch)
    # everything padded: all outputs zero
    batch["lens"], batch["bnd"] = torch.zeros(8, dtype=torch.int32).cuda(), torch.zeros(8, dtype=torch.int32).cuda()
    out, _ = run_and_compare(trl, w, batch=batch)
    assert float(out["loss"]) == 0.0


def test_all_equal_rewards_give_exact_zero(trl):
    w = synth.scaled(synth.CONFIGS[2], name="degenerate_all", P=2, G=4, T=128, H=128, V=512)
    batch = synth.make_batch(w, device="cuda:0")
    batch["r_plan"] = torch.tensor([0.7] * 4 + [1.3] * 4, device="cuda:0")
    batch["r_code"] = torch.tensor([1.0] * 4 + [0.0] * 4, device="cuda:0")
    out, _ = run_and_compare(trl, w, batch=batch)
    assert float(out["loss"]) == 0.0 and not out["g"].any() and not out["dW"].any() and not out["dHidden"].any()


def test_group_size_one(trl):
    w = synth.scaled(synth.CONFIGS[0], name="g1", P=6, G=1, T=64, H=64, V=256)
    out, _ = run_and_compare(trl, w)
    assert float(out["loss"]) == 0.0


def test_uniform_logits_closed_form(trl):
    # W = 0: logp = -ln V exactly representable to fp32 rounding on both paths
    for dtype, tdt in (("bf16", torch.bfloat16), ("f32", torch.float32)):
        w = synth.scaled(synth.CONFIGS[2], name="uniform", P=1, G=2, T=128, H=64, V=1000, dtype=dtype)
        batch = synth.make_batch(w, device="cuda:0")
        batch["W"] = torch.zeros_like(batch["W"])
        logp, lse = trl.trl_token_logprobs(batch["hidden"], batch["W"], batch["ids"], batch["lens"], w.T)
        torch.cuda.synchronize()
        L = int(batch["lens"][0])
        assert abs(float(lse[0]) - np.log(1000.0)) < 1e-5 and abs(float(logp[L - 1]) + np.log(1000.0)) < 1e-5


def test_device_detected_bad_inputs_set_status_without_faulting(trl):
    w = synth.scaled(synth.CONFIGS[2], name="bad", P=1, G=2, T=128, H=64, V=512)
    batch = synth.make_batch(w, device="cuda:0")
    batch["ids"][3] = 100000          # outside [0, V)
    batch["lens"][:] = torch.tensor([128, 90], dtype=torch.int32)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    logp, _ = trl.trl_token_logprobs(batch["hidden"], batch["W"], batch["ids"], batch["lens"], w.T, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & (1 << 7) and float(logp[3]) == 0.0
    with pytest.raises(trl.TrlError):
        trl.check_status(status)
    status.zero_()
    batch["bnd"][0] = 500             # beyond len
    trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], 1, 2, w.T, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & (1 << 7)


def test_host_argument_errors(trl):
    w = synth.scaled(synth.CONFIGS[2], name="args", P=1, G=2, T=128, H=64, V=512)
    batch = synth.make_batch(w, device="cuda:0")
    tiny = torch.empty(256, dtype=torch.uint8, device="cuda:0")
    with pytest.raises(trl.TrlError, match="workspace"):
        trl.trl_token_logprobs(batch["hidden"], batch["W"], batch["ids"], batch["lens"], w.T, workspace=tiny)
    with pytest.raises(trl.TrlError, match="shape"):
        trl.trl_token_logprobs(batch["hidden"][:, :60].contiguous(), batch["W"][:, :60].contiguous(), batch["ids"],
                               batch["lens"], w.T)      # H % 8 != 0 in bf16


@pytest.mark.parametrize("use_hint", [True, False])
def test_fused_step_matches_oracle(trl, use_hint):
    """trl_pg_step_fused (forward GEMM stores E = exp(z - c), no recompute) against the oracle,
    with the old policy's lse as the shift and with no hint."""
    w = synth.scaled(synth.CONFIGS[2], name="fused_ragged", P=2, G=4, T=300, H=320, V=1000)
    run_and_compare(trl, w, fused=True, use_hint=use_hint)
    run_and_compare(trl, w, fused=True, use_hint=use_hint, explicit_old=True, alpha=0.5, eps=0.1)
    w = synth.scaled(synth.CONFIGS[2], name="fused_wide", P=3, G=6, T=384, H=512, V=3000, real_plan_reward=True,
                     len_lo=0.1, degenerate_frac=0.34)
    run_and_compare(trl, w, fused=True, use_hint=use_hint)
    run_and_compare(trl, synth.CONFIGS[0], fused=True, use_hint=use_hint)          # fp32: three calls inside


def test_fused_step_edge_cases(trl):
    w = synth.scaled(synth.CONFIGS[2], name="fused_edge", P=2, G=4, T=160, H=128, V=512)
    batch = synth.make_batch(w, device="cuda:0")
    batch["lens"] = torch.tensor([0, 160, 1, 128, 129, 77, 0, 5], dtype=torch.int32).cuda()
    batch["bnd"] = torch.tensor([0, 0, 1, 128, 64, 77, 0, 2], dtype=torch.int32).cuda()
    run_and_compare(trl, w, batch=batch, fused=True)
    batch["lens"], batch["bnd"] = torch.zeros(8, dtype=torch.int32).cuda(), torch.zeros(8, dtype=torch.int32).cuda()
    out, _ = run_and_compare(trl, w, batch=batch, fused=True)
    assert float(out["loss"]) == 0.0


def test_fused_step_any_reasonable_hint_gives_same_result_and_bad_hint_is_flagged(trl):
    w = synth.scaled(synth.CONFIGS[2], name="fused_hint", P=2, G=4, T=200, H=256, V=1536)
    batch = synth.make_batch(w, device="cuda:0")
    old_logp, old_lse = trl.trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], w.T)
    hrd = trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], w.P, w.G, w.T)
    args = (batch["hidden"], batch["W"], batch["ids"], batch["lens"], old_logp)
    ref = trl.trl_pg_step_fused(*args, None, hrd["adv"], hrd["seg"], w.P, w.G, w.T)
    shifted = old_lse + 10.0 * (torch.rand_like(old_lse) - 0.5)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    out = trl.trl_pg_step_fused(*args, shifted, hrd["adv"], hrd["seg"], w.P, w.G, w.T, status=status)
    torch.cuda.synchronize()
    trl.check_status(status)
    assert (out["logp"] - ref["logp"]).abs().max() <= 1e-4
    assert abs(float(out["loss"]) - float(ref["loss"])) <= 1e-4 * abs(float(ref["loss"]))
    assert rel_fro(f64(out["dW"]), f64(ref["dW"])) <= 1e-2 and rel_fro(f64(out["dHidden"]), f64(ref["dHidden"])) <= 1e-2
    trl.trl_pg_step_fused(*args, old_lse - 500.0, hrd["adv"], hrd["seg"], w.P, w.G, w.T, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) & (1 << 9)


@pytest.mark.parametrize("fused", [False, True])
def test_documented_loss_variants(trl, fused):
    """Appendix clip form A*min{s, clip(s)} (uniform-reward GRPO as printed: one reward for both
    classes, alpha = 1) and token-mean aggregation, against the oracle."""
    w = synth.scaled(synth.CONFIGS[2], name="variants", P=2, G=4, T=200, H=256, V=1536, sigma_old=0.15)
    batch = synth.make_batch(w, device="cuda:0")
    run_and_compare(trl, w, batch=batch, fused=fused, clip_form=1)
    run_and_compare(trl, w, batch=batch, fused=fused, agg_mode=1)
    batch["r_code"] = batch["r_plan"] = 0.7 * batch["r_code"] + 0.3 * batch["r_plan"]     # beta = 0.7 mixture
    run_and_compare(trl, w, batch=batch, fused=fused, clip_form=1, alpha=1.0)
    run_and_compare(trl, synth.CONFIGS[0], fused=fused, clip_form=1, agg_mode=1)


def test_fused_step_minimum_workspace_chunks(trl):
    """One 128-row chunk at a time must give what one big chunk gives."""
    w = synth.scaled(synth.CONFIGS[2], name="fused_chunks", P=1, G=3, T=300, H=128, V=520)
    batch = synth.make_batch(w, device="cuda:0")
    old_logp, old_lse = trl.trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], w.T)
    hrd = trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], w.P, w.G, w.T)
    args = (batch["hidden"], batch["W"], batch["ids"], batch["lens"], old_logp, old_lse, hrd["adv"], hrd["seg"], w.P, w.G, w.T)
    ref = trl.trl_pg_step_fused(*args)
    nmin = trl.trl_workspace_bytes_min(trl.TRL_CALL_PG_STEP_FUSED, w.B, w.T, w.H, w.V, trl.TRL_BF16)
    assert nmin < trl.trl_workspace_bytes(trl.TRL_CALL_PG_STEP_FUSED, w.B, w.T, w.H, w.V, trl.TRL_BF16)
    out = trl.trl_pg_step_fused(*args, workspace=torch.empty(nmin, dtype=torch.uint8, device="cuda:0"))
    torch.cuda.synchronize()
    assert torch.equal(out["logp"], ref["logp"]) and torch.equal(out["g"], ref["g"]) and torch.equal(out["dHidden"], ref["dHidden"])
    assert float(out["loss"]) == float(ref["loss"])
    assert rel_fro(f64(out["dW"]), f64(ref["dW"])) < 1e-5


@pytest.mark.parametrize("fused", [False, True])
def test_many_rollouts_and_odd_length(trl, fused):
    """More rollouts than the threads of the row-packing scan (1024), and a T that is not a multiple
    of 4 (scalar paths of the advantage / loss kernels, rollouts that do not start 16-byte aligned)."""
    w = synth.scaled(synth.CONFIGS[2], name="many_rollouts", P=150, G=8, T=12, H=64, V=256, len_lo=0.0)
    run_and_compare(trl, w, fused=fused)
    w = synth.scaled(synth.CONFIGS[2], name="odd_T", P=2, G=3, T=75, H=128, V=520, len_lo=0.3)
    run_and_compare(trl, w, fused=fused)
    run_and_compare(trl, synth.scaled(w, name="odd_T_f32", dtype="f32"), fused=fused)


@pytest.mark.parametrize("shape", [(1, 1, 1, 8, 8), (1, 2, 3, 8, 1000), (2, 2, 5, 1024, 8), (1, 3, 130, 16, 24),
                                   (1, 1, 128, 64, 256), (1, 1, 129, 64, 264)])
def test_smallest_legal_shapes(trl, shape):
    """Tensors smaller than one TMA box / one tile in every dimension (H = V = 8, T = 1), and shapes
    one past a tile edge."""
    P, G, T, H, V = shape
    w = synth.scaled(synth.CONFIGS[2], name=f"tiny_{P}_{G}_{T}_{H}_{V}", P=P, G=G, T=T, H=H, V=V, len_lo=0.5)
    run_and_compare(trl, w)
    run_and_compare(trl, w, fused=True)


def test_minimum_workspace_gives_same_backward(trl):
    # chunked backward (one 128-row block per chunk) equals the one-chunk result
    w = synth.scaled(synth.CONFIGS[2], name="chunks", P=1, G=3, T=200, H=128, V=512)
    batch = synth.make_batch(w, device="cuda:0")
    logp, lse = trl.trl_token_logprobs(batch["hidden"], batch["W"], batch["ids"], batch["lens"], w.T)
    g = torch.randn(w.N, device="cuda:0") * (torch.arange(w.N, device="cuda:0") % w.T < batch["lens"].repeat_interleave(w.T))
    dH1, dW1 = trl.trl_pg_loss_bwd(batch["hidden"], batch["W"], batch["ids"], batch["lens"], lse, g, w.T)
    nmin = trl.trl_workspace_bytes_min(trl.TRL_CALL_PG_LOSS_BWD, w.B, w.T, w.H, w.V, trl.TRL_BF16)
    ws = torch.empty(nmin, dtype=torch.uint8, device="cuda:0")
    dH2, dW2 = trl.trl_pg_loss_bwd(batch["hidden"], batch["W"], batch["ids"], batch["lens"], lse, g, w.T, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(dH1, dH2)
    assert rel_fro(f64(dW2), f64(dW1)) < 1e-5


# ---------------------------------------------------------------- a confident (trained) policy
def _confident(name, scale, dtype="bf16"):
    return synth.scaled(synth.CONFIGS[2], name=f"{name}_{scale}_{dtype}", P=2, G=4, T=300, H=320, V=1000, dtype=dtype,
                        logit_scale=float(scale), greedy_ids=True)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("scale,med_lo,med_hi", [(8, 0.55, 0.85), (20, 0.96, 0.995), (32, 0.997, 0.9999)])
def test_confident_policy_every_element_and_most_confident_rows(trl, dtype, fused, scale, med_lo, med_hi):
    """Peaked softmax: the sampled token is the arg-max and carries most of the probability
    (median p_t about 0.7, 0.98, 0.998), the regime of a trained policy.  Every output against the
    oracle at the usual tolerances, then dHidden row by row on the most confident rows that still
    have a gradient: there the one-hot entry g (1 - p_t) is a small difference of nearly equal
    numbers, and the row is only right if that entry is formed without cancellation."""
    w = _confident("confident", scale, dtype)
    out, ref = run_and_compare(trl, w, fused=fused)
    valid = ref["seg"] != 0
    p_t = np.exp(ref["logp"])
    assert med_lo <= np.median(p_t[valid]) <= med_hi
    live = np.nonzero(valid & (ref["g"] != 0))[0]
    # The fused step forms the entry as -sum_{v != t} E_v and is exact however small 1 - p_t is.  The
    # separate backward recomputes p_t = exp(z_t - lse) from an lse it receives in fp32, so its entry
    # carries an absolute error of about ulp(lse): rows with 1 - p_t below ~1e-3 are left to the
    # Frobenius check above, where their (tiny) gradients weigh nothing.
    floor = 1e-7 if (fused and dtype == "bf16") else 2e-3
    cand = live[(1.0 - p_t[live]) >= floor]
    top = cand[np.argsort(p_t[cand])[::-1][:48]]
    assert top.size >= 16 and (1.0 - p_t[top]).min() < 2e-2
    dH = f64(out["dHidden"])[top]
    err = np.linalg.norm(dH - ref["dHidden"][top], axis=1) / np.linalg.norm(ref["dHidden"][top], axis=1)
    assert err.max() <= 2e-2, (err.max(), float(p_t[top[np.argmax(err)]]))


def test_fused_step_is_as_accurate_as_the_separate_calls_on_a_confident_policy(trl):
    """Relative Frobenius error of dHidden and dW: the fused schedule (E stored in bf16) must stay
    within 1.5x of the four-call schedule (dS stored in bf16), both far inside the tolerance."""
    for scale in (8, 20, 32):
        w = _confident("confident_cmp", scale)
        errs = {}
        for fused in (False, True):
            out, ref = run_and_compare(trl, w, fused=fused)
            errs[fused] = (rel_fro(f64(out["dHidden"]), ref["dHidden"]), rel_fro(f64(out["dW"]), ref["dW"]))
        for k in (0, 1):
            assert errs[True][k] <= max(1.5 * errs[False][k], 3e-3), (scale, errs)


def test_asymmetric_clip_range(trl):
    """eps_lo != eps_hi, old policy far enough away that both clip sides fire."""
    w = synth.scaled(synth.CONFIGS[2], name="asym_clip", P=2, G=4, T=200, H=256, V=1536, sigma_old=0.25)
    for fused in (False, True):
        out, ref = run_and_compare(trl, w, fused=fused, eps=0.1, eps_hi=0.3)
        assert ref["stats"][0] > 0.01 and ref["stats"][1] > 0.05          # both sides clip somewhere
        assert ref["stats"][1] > 1.5 * ref["stats"][0]                    # and the narrow side clips more
    run_and_compare(trl, w, eps=0.3, eps_hi=0.05, clip_form=1)
    run_and_compare(trl, synth.scaled(w, name="asym_clip_f32", dtype="f32"), eps=0.3, eps_hi=0.05)


@pytest.mark.parametrize("offset", [-60.0, -35.0, -20.0, 20.0, 45.0, 60.0])
def test_fused_step_hint_tens_of_units_off(trl, offset):
    """A shift c that misses the true log-partition by 20 to 60 (E then lives around e^-offset)
    must still give the oracle's results: the header promises any hint within ~80."""
    w = synth.scaled(synth.CONFIGS[2], name="fused_hint_far", P=2, G=4, T=200, H=256, V=1536)
    batch = synth.make_batch(w, device="cuda:0")
    oi = oracle_inputs(batch)
    ref = orc.full_step(oi["hidden"], oi["W"], oi["hidden_old"], oi["W_old"], oi["ids"], oi["lens"], oi["bnd"],
                        oi["r_plan"], oi["r_code"], w.P, w.G, w.T)
    old_logp, old_lse = trl.trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], w.T)
    hrd = trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], w.P, w.G, w.T)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    hint = old_lse + offset + 5.0 * (torch.rand_like(old_lse) - 0.5)
    out = trl.trl_pg_step_fused(batch["hidden"], batch["W"], batch["ids"], batch["lens"], old_logp, hint, hrd["adv"],
                                hrd["seg"], w.P, w.G, w.T, status=status)
    torch.cuda.synchronize()
    trl.check_status(status)
    assert np.abs(f64(out["logp"]) - ref["logp"]).max() <= TOL_LOGP
    assert abs(float(out["loss"]) - ref["loss"]) <= TOL_LOSS * abs(ref["loss"])
    assert rel_fro(f64(out["dHidden"]), ref["dHidden"]) <= TOL_GRAD and rel_fro(f64(out["dW"]), ref["dW"]) <= TOL_GRAD


# ---------------------------------------------------------------- long rollouts: several token tiles per rollout
@pytest.mark.parametrize("T", [16384, 20000, 40001])
def test_advantages_and_loss_over_several_token_tiles(trl, T):
    """Responses up to the paper's 16,384-token limit and beyond: the advantage kernel then covers a
    rollout with several CTAs (8192 tokens each) and the loss kernel with several partial sums
    (16384 tokens each); T % 16 == 0, T % 4 == 0 and odd T take the three store paths."""
    P, G = 2, 3
    B, N = P * G, P * G * T
    g = torch.Generator().manual_seed(T)
    lens = torch.randint(T // 3, T + 1, (B,), generator=g, dtype=torch.int32)
    lens[1], lens[4] = T, 8192
    bnd = (lens.double() * torch.rand(B, generator=g, dtype=torch.float64)).to(torch.int32)
    r_plan = torch.rand(B, generator=g) * 2.0
    r_code = (torch.rand(B, generator=g) < 0.5).float()
    old = -torch.rand(N, generator=g) * 6
    logp = old + 0.15 * torch.randn(N, generator=g)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    dev = lambda t: t.to("cuda:0")
    hrd = trl.trl_hrd_advantages(dev(r_plan), dev(r_code), dev(lens), dev(bnd), P, G, T, status=status)
    loss, gg, stats = trl.trl_pg_loss_fwd(dev(logp), dev(old), hrd["adv"], hrd["seg"], dev(lens), P, G, T, status=status)
    torch.cuda.synchronize()
    trl.check_status(status)
    ref = orc.hrd_advantages(f64(r_plan), f64(r_code), lens.numpy(), bnd.numpy(), P, G, T)
    np.testing.assert_array_equal(hrd["seg"].cpu().numpy(), ref["seg"])
    np.testing.assert_array_equal(hrd["n_plan"].cpu().numpy(), ref["n_plan"])
    np.testing.assert_array_equal(hrd["n_code"].cpu().numpy(), ref["n_code"])
    assert int(hrd["n_valid"].item()) == ref["n_valid"]
    np.testing.assert_allclose(f64(hrd["adv"]), ref["adv"], rtol=1e-6, atol=1e-7)
    rl, rg, rs = orc.pg_loss_fwd(f64(logp), f64(old), ref["adv"], ref["seg"], lens.numpy(), P, G, T)
    assert abs(float(loss) - rl) <= TOL_LOSS * abs(rl)
    assert rel_fro(f64(gg), rg) <= 1e-5
    np.testing.assert_allclose(f64(stats), rs, rtol=1e-4, atol=1e-6)


def test_fused_step_leaves_a_bad_id_row_out_of_loss_g_and_gradients(trl):
    """A token id outside [0, V): flagged, and the row is treated as padding by everything the
    fused call returns (same results as with that row's advantage set to zero)."""
    w = synth.scaled(synth.CONFIGS[2], name="bad_fused", P=1, G=2, T=128, H=64, V=512)
    batch = synth.make_batch(w, device="cuda:0")
    batch["lens"] = torch.tensor([100, 128], dtype=torch.int32, device="cuda:0")
    batch["bnd"] = torch.tensor([40, 60], dtype=torch.int32, device="cuda:0")
    batch["r_plan"] = torch.tensor([1.0, 0.0], device="cuda:0")
    batch["r_code"] = torch.tensor([0.0, 1.0], device="cuda:0")
    old_logp, old_lse = trl.trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], w.T)
    hrd = trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], w.P, w.G, w.T)
    assert float(hrd["adv"][5]) != 0.0
    bad = batch["ids"].clone()
    bad[5] = 70000
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    out = trl.trl_pg_step_fused(batch["hidden"], batch["W"], bad, batch["lens"], old_logp, old_lse, hrd["adv"], hrd["seg"],
                                w.P, w.G, w.T, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 1 << 7
    adv0 = hrd["adv"].clone()
    adv0[5] = 0.0
    ref = trl.trl_pg_step_fused(batch["hidden"], batch["W"], batch["ids"], batch["lens"], old_logp, old_lse, adv0, hrd["seg"],
                                w.P, w.G, w.T)
    torch.cuda.synchronize()
    assert float(out["g"][5]) == 0.0 and float(out["logp"][5]) == 0.0 and not out["dHidden"][5].any()
    assert float(out["loss"]) == float(ref["loss"]) and torch.equal(out["dHidden"], ref["dHidden"])
    assert torch.equal(out["g"], ref["g"]) and rel_fro(f64(out["dW"]), f64(ref["dW"])) < 1e-6


@pytest.mark.parametrize("fused", [False, True])
def test_inactive_row_blocks_between_active_ones(trl, fused):
    """Zero-advantage groups in the middle of the batch make whole 128-row blocks inactive between
    active ones (an odd number of them, at odd positions, plus a plan-only stretch): the gradient
    GEMMs form their tiles over the active blocks only.  Every element against the oracle."""
    w = synth.scaled(synth.CONFIGS[2], name="holes", P=5, G=2, T=448, H=128, V=768, len_lo=1.0, len_hi=1.0)
    batch = synth.make_batch(w, device="cuda:0")
    # groups 1 and 3: all-equal rewards in both classes (7 blocks of zero rows each); group 2: equal
    # plan rewards only (its plan tokens are inactive, its code tokens are not); group 4 ends the batch inactive
    batch["r_plan"] = torch.tensor([1.0, 0.0, 0.5, 0.5, 1.0, 1.0, 0.0, 0.0, 2.0, 2.0], device="cuda:0")
    batch["r_code"] = torch.tensor([0.0, 1.0, 1.0, 1.0, 1.0, 0.0, 0.0, 0.0, 1.0, 1.0], device="cuda:0")
    batch["bnd"] = torch.tensor([100, 300, 200, 10, 384, 256, 5, 440, 128, 0], dtype=torch.int32, device="cuda:0")
    out, ref = run_and_compare(trl, w, batch=batch, fused=fused)
    g = f64(out["g"]).reshape(w.B, w.T)
    assert not g[2:4].any() and not g[6:10].any() and g[0].any() and g[4, 384:].any() and not g[4, :384].any()
