"""Pins for the fp64 oracle: values worked by hand, closed forms, invariants, brute force,
a library routine (scipy logsumexp) and finite differences.  None of these re-type the
oracle's own formulas with the oracle's own primitives; each would fail for a plausible
mistake (dropped term, wrong sign/index, transposed operand, wrong normaliser)."""
import math
import os

import numpy as np
import pytest
from scipy.special import logsumexp

from oracle import trl_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_fixture(name):
    d = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            d[k] = np.array([float(x) for x in v])
    return d


def _rng(seed):
    return np.random.default_rng(seed)


def _tiny_problem(seed, P=2, G=3, T=5, H=6, V=11):
    r = _rng(seed)
    B = P * G
    hidden = r.standard_normal((B * T, H))
    W = r.standard_normal((V, H)) * H ** -0.5
    ids = r.integers(0, V, B * T)
    lens = r.integers(1, T + 1, B)
    lens[0] = T
    bnd = np.array([r.integers(0, L + 1) for L in lens])
    r_plan = r.random(B) * 2.0
    r_code = (r.random(B) < 0.5).astype(float)
    return dict(P=P, G=G, T=T, H=H, V=V, hidden=hidden, W=W, ids=ids, lens=lens, bnd=bnd,
                r_plan=r_plan, r_code=r_code)


# ----------------------------------------------------------------------------- scoring

def test_logprob_hand_worked_fixture():
    fx = _read_fixture("logprob_worked_example.txt")
    H, V = int(fx["H"][0]), int(fx["V"][0])
    hidden = fx["hidden"].reshape(2, H)
    W = fx["W"].reshape(V, H)
    logp, lse = orc.token_logprobs(hidden, W, fx["ids"].astype(int), np.array([2]), T=2)
    np.testing.assert_allclose(lse, fx["lse"], rtol=0, atol=1e-14)
    np.testing.assert_allclose(logp, fx["logp"], rtol=0, atol=1e-14)


def test_uniform_logits_give_minus_log_V():
    V, H, T = 37, 5, 4
    r = _rng(0)
    ids = r.integers(0, V, 2 * T)
    # W = 0 and hidden = 0 both give uniform logits
    for hidden, W in ((r.standard_normal((2 * T, H)), np.zeros((V, H))),
                      (np.zeros((2 * T, H)), r.standard_normal((V, H)))):
        logp, lse = orc.token_logprobs(hidden, W, ids, np.array([T, T]), T)
        np.testing.assert_allclose(lse, math.log(V), atol=1e-14)
        np.testing.assert_allclose(logp, -math.log(V), atol=1e-14)


def test_logprob_against_python_loops_and_scipy():
    p = _tiny_problem(1)
    logp, lse = orc.token_logprobs(p["hidden"], p["W"], p["ids"], p["lens"], p["T"])
    for b in range(p["P"] * p["G"]):
        for t in range(p["T"]):
            n = b * p["T"] + t
            if t >= p["lens"][b]:
                assert logp[n] == 0.0 and lse[n] == 0.0
                continue
            z = [sum(p["hidden"][n, k] * p["W"][v, k] for k in range(p["H"])) for v in range(p["V"])]
            ref_lse = logsumexp(z)
            assert abs(lse[n] - ref_lse) < 1e-12
            assert abs(logp[n] - (z[p["ids"][n]] - ref_lse)) < 1e-12


def test_logprob_large_logit_is_stable_and_dominant():
    V, H = 9, 3
    hidden = np.array([[1.0, 0.0, 0.0]])
    W = np.zeros((V, H))
    W[4, 0] = 800.0            # naive exp would overflow
    logp, lse = orc.token_logprobs(hidden, W, np.array([4]), np.array([1]), T=1)
    assert abs(lse[0] - 800.0) < 1e-12 and abs(logp[0]) < 1e-12
    logp, _ = orc.token_logprobs(hidden, W, np.array([2]), np.array([1]), T=1)
    assert abs(logp[0] + 800.0) < 1e-9


def test_logprob_shift_and_permutation_invariance():
    p = _tiny_problem(2)
    logp, lse = orc.token_logprobs(p["hidden"], p["W"], p["ids"], p["lens"], p["T"])
    c = _rng(3).standard_normal(p["H"])
    logp2, _ = orc.token_logprobs(p["hidden"], p["W"] + c[None, :], p["ids"], p["lens"], p["T"])
    np.testing.assert_allclose(logp2, logp, atol=1e-12)      # softmax is shift invariant
    perm = _rng(4).permutation(p["V"])                        # new index of old row perm[k] is k
    inv = np.argsort(perm)
    logp3, lse3 = orc.token_logprobs(p["hidden"], p["W"][perm], inv[p["ids"]], p["lens"], p["T"])
    np.testing.assert_allclose(logp3, logp, atol=1e-12)
    np.testing.assert_allclose(lse3, lse, atol=1e-12)


# -------------------------------------------------------------------------- advantages

def test_hrd_hand_worked_fixture():
    fx = _read_fixture("hrd_worked_example.txt")
    P, G, T = int(fx["P"][0]), int(fx["G"][0]), int(fx["T"][0])
    lens, bnd = fx["lens"].astype(int), fx["bnd"].astype(int)
    hrd = orc.hrd_advantages(fx["r_plan"], fx["r_code"], lens, bnd, P, G, T)
    np.testing.assert_array_equal(hrd["A_plan"], fx["A_plan"])
    np.testing.assert_array_equal(hrd["A_code"], fx["A_code"])
    np.testing.assert_array_equal(hrd["seg"], fx["seg"].astype(np.uint8))
    np.testing.assert_array_equal(hrd["adv"], fx["adv"])
    old_logp = _rng(5).standard_normal(P * G * T) - 3.0
    logp = old_logp + np.log(fx["ratio"])
    loss, g, stats = orc.pg_loss_fwd(logp, old_logp, hrd["adv"], hrd["seg"], lens, P, G, T,
                                     fx["eps"][0], fx["eps"][0], fx["alpha"][0])
    assert abs(loss - fx["loss"][0]) < 1e-14
    np.testing.assert_allclose(g, fx["g"], rtol=0, atol=1e-14)
    assert abs(stats[0] - fx["clip_frac_hi"][0]) < 1e-14
    assert abs(stats[1] - fx["clip_frac_lo"][0]) < 1e-14
    assert abs(stats[2] - fx["mean_ratio"][0]) < 1e-13
    assert stats[3] == 6


def test_advantage_textbook_group():
    # r = (1,0,0,0): A = (.75,-.25,-.25,-.25); a second group with all-equal rewards: A = 0 exactly
    r = np.array([1, 0, 0, 0, 0.3, 0.3, 0.3, 0.3])
    lens = np.full(8, 3)
    hrd = orc.hrd_advantages(r, r[::-1].copy(), lens, np.full(8, 1), P=2, G=4, T=3)
    np.testing.assert_array_equal(hrd["A_plan"], [.75, -.25, -.25, -.25, 0, 0, 0, 0])
    np.testing.assert_array_equal(hrd["A_code"], [0, 0, 0, 0, -.25, -.25, -.25, .75])
    # plan tokens carry the plan advantage, code tokens the code advantage
    adv = hrd["adv"].reshape(8, 3)
    np.testing.assert_array_equal(adv[:, 0], hrd["A_plan"])
    np.testing.assert_array_equal(adv[:, 1], hrd["A_code"])
    np.testing.assert_array_equal(adv[:, 2], hrd["A_code"])


def test_advantage_invariants():
    p = _tiny_problem(6, P=3, G=5)
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], p["P"], p["G"], p["T"])
    for A in (hrd["A_plan"], hrd["A_code"]):
        np.testing.assert_allclose(A.reshape(p["P"], p["G"]).sum(axis=1), 0, atol=1e-14)
    shift = np.repeat(_rng(7).standard_normal(p["P"]), p["G"])
    hrd2 = orc.hrd_advantages(p["r_plan"] + shift, p["r_code"], p["lens"], p["bnd"], p["P"], p["G"], p["T"])
    np.testing.assert_allclose(hrd2["A_plan"], hrd["A_plan"], atol=1e-14)
    one = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], p["P"] * p["G"], 1, p["T"])
    assert not one["A_plan"].any() and not one["A_code"].any() and not one["adv"].any()   # G = 1
    # std-normalised option: unit population variance per non-degenerate group, scale invariant
    n1 = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], p["P"], p["G"], p["T"], adv_mode=1)
    n2 = orc.hrd_advantages(7 * p["r_plan"], p["r_code"], p["lens"], p["bnd"], p["P"], p["G"], p["T"], adv_mode=1)
    np.testing.assert_allclose((n1["A_plan"].reshape(p["P"], p["G"]) ** 2).mean(axis=1), 1, atol=1e-4)
    np.testing.assert_allclose(n1["A_plan"], n2["A_plan"], atol=1e-5)


def test_segments_and_counts_closed_form():
    T = 7
    lens = np.array([7, 0, 3, 5, 1, 7])
    bnd = np.array([0, 0, 3, 2, 1, 7])       # no plan / empty / no code / both / single / all plan
    hrd = orc.hrd_advantages(np.arange(6.0), np.arange(6.0) * 2, lens, bnd, P=2, G=3, T=T)
    seg = hrd["seg"].reshape(6, T)
    for b in range(6):
        expect = [1 if t < bnd[b] else 2 if t < lens[b] else 0 for t in range(T)]
        assert seg[b].tolist() == expect
    np.testing.assert_array_equal(hrd["n_plan"], bnd)
    np.testing.assert_array_equal(hrd["n_code"], lens - bnd)
    assert hrd["n_valid"] == lens.sum()
    assert hrd["seg"].dtype == np.uint8 and hrd["n_plan"].dtype == np.int32


# --------------------------------------------------------------------------------- loss

def test_ratio_one_closed_form_and_zero_clip_fraction():
    p = _tiny_problem(8, P=3, G=4, T=9)
    P, G, T = p["P"], p["G"], p["T"]
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], P, G, T)
    logp = -_rng(9).random(P * G * T) * 5
    alpha = 0.37
    loss, g, stats = orc.pg_loss_fwd(logp, logp.copy(), hrd["adv"], hrd["seg"], p["lens"], P, G, T, 0.2, 0.2, alpha)
    # s = 1: J = (1/P) sum_i (1/G) sum_j [alpha A^plan n_plan + A^code n_code] / len
    J = 0.0
    for b in range(P * G):
        L = p["lens"][b]
        J += (alpha * hrd["A_plan"][b] * p["bnd"][b] + hrd["A_code"][b] * (L - p["bnd"][b])) / L
    J /= P * G
    assert abs(loss + J) < 1e-13
    assert stats[0] == 0 and stats[1] == 0 and abs(stats[2] - 1) < 1e-15 and stats[3] == p["lens"].sum()


def test_all_equal_group_gives_exactly_zero_loss_and_gradient():
    P, G, T = 2, 4, 6
    lens = np.array([6, 5, 4, 3, 6, 6, 2, 1])
    bnd = lens // 2
    r_plan = np.repeat([0.7, 1.3], G)
    r_code = np.repeat([1.0, 0.0], G)
    hrd = orc.hrd_advantages(r_plan, r_code, lens, bnd, P, G, T)
    r = _rng(10)
    loss, g, _ = orc.pg_loss_fwd(-r.random(P * G * T), -r.random(P * G * T), hrd["adv"], hrd["seg"], lens, P, G, T)
    assert loss == 0.0 and not g.any()


@pytest.mark.parametrize("s,A,u,active", [
    (1.5, 2.0, 2.0 * 1.2, False),     # A>0, s above 1+eps: saturates at 1+eps, no gradient
    (0.5, -2.0, -2.0 * 0.8, False),   # A<0, s below 1-eps: saturates at 1-eps, no gradient
    (0.5, 2.0, 2.0 * 0.5, True),      # A>0, s small: unclipped
    (1.5, -2.0, -2.0 * 1.5, True),    # A<0, s large: unclipped (no dual clip)
    (1.1, 2.0, 2.0 * 1.1, True),
    (0.9, -2.0, -2.0 * 0.9, True),
])
def test_clip_saturation_single_token(s, A, u, active):
    # one prompt, one rollout, one code token: loss = -u, g = -A s if active
    loss, g, _ = orc.pg_loss_fwd(np.array([math.log(s) - 1.0]), np.array([-1.0]), np.array([A]),
                                 np.array([2], dtype=np.uint8), np.array([1]), 1, 1, 1, 0.2, 0.2, 0.1)
    assert abs(loss + u) < 1e-14
    assert abs(g[0] - (-A * s if active else 0.0)) < 1e-14


def test_loss_linear_in_reward_scale_alpha_zero_and_uniform_case():
    p = _tiny_problem(11, P=2, G=4, T=8)
    P, G, T = p["P"], p["G"], p["T"]
    r = _rng(12)
    old = -r.random(P * G * T) * 4
    logp = old + r.standard_normal(P * G * T) * 0.3
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], P, G, T)
    hrd3 = orc.hrd_advantages(3 * p["r_plan"], 3 * p["r_code"], p["lens"], p["bnd"], P, G, T)
    l1, g1, _ = orc.pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T)
    l3, g3, _ = orc.pg_loss_fwd(logp, old, hrd3["adv"], hrd3["seg"], p["lens"], P, G, T)
    assert abs(l3 - 3 * l1) < 1e-13
    np.testing.assert_allclose(g3, 3 * g1, atol=1e-14)
    # alpha = 0 removes the plan term: equals the loss with the plan advantages zeroed
    adv_code_only = np.where(hrd["seg"] == 2, hrd["adv"], 0.0)
    la, _, _ = orc.pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T, alpha=0.0)
    lb, _, _ = orc.pg_loss_fwd(logp, old, adv_code_only, hrd["seg"], p["lens"], P, G, T, alpha=0.5)
    assert abs(la - lb) < 1e-14
    # alpha = 1 with r_plan = r_code is uniform-reward GRPO (appendix on uniform reward
    # assignment, with the min taken as in Section 2.3): brute-force loops
    hu = orc.hrd_advantages(p["r_plan"], p["r_plan"], p["lens"], p["bnd"], P, G, T)
    lu, _, _ = orc.pg_loss_fwd(logp, old, hu["adv"], hu["seg"], p["lens"], P, G, T, 0.2, 0.2, 1.0)
    J = 0.0
    for i in range(P):
        mu = sum(p["r_plan"][i * G + j] for j in range(G)) / G
        for j in range(G):
            b = i * G + j
            A = p["r_plan"][b] - mu
            acc = 0.0
            for t in range(p["lens"][b]):
                s = math.exp(logp[b * T + t] - old[b * T + t])
                acc += min(A * s, A * min(max(s, 0.8), 1.2))
            J += acc / p["lens"][b] / G
    assert abs(lu + J / P) < 1e-13


def test_loss_permutation_of_rollouts_within_group():
    p = _tiny_problem(13, P=2, G=4, T=6)
    P, G, T = p["P"], p["G"], p["T"]
    r = _rng(14)
    old = -r.random(P * G * T)
    logp = old + r.standard_normal(P * G * T) * 0.2
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], P, G, T)
    l1, _, _ = orc.pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T)
    perm = np.concatenate([r.permutation(G), G + r.permutation(G)])
    rows = (perm[:, None] * T + np.arange(T)[None, :]).ravel()
    hrd2 = orc.hrd_advantages(p["r_plan"][perm], p["r_code"][perm], p["lens"][perm], p["bnd"][perm], P, G, T)
    l2, _, _ = orc.pg_loss_fwd(logp[rows], old[rows], hrd2["adv"], hrd2["seg"], p["lens"][perm], P, G, T)
    assert abs(l1 - l2) < 1e-14


# ---------------------------------------------------------------------------- gradients

def _loss_of(p, hidden, W, old_logp, adv, seg, alpha=0.3):
    logp, lse = orc.token_logprobs(hidden, W, p["ids"], p["lens"], p["T"])
    loss, g, _ = orc.pg_loss_fwd(logp, old_logp, adv, seg, p["lens"], p["P"], p["G"], p["T"], 0.2, 0.2, alpha)
    return loss, g, lse, logp


def test_finite_difference_gradients():
    p = _tiny_problem(15, P=2, G=3, T=4, H=5, V=7)
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], p["P"], p["G"], p["T"])
    logp0, _ = orc.token_logprobs(p["hidden"], p["W"], p["ids"], p["lens"], p["T"])
    # ratios spread over clipped / unclipped regions but away from the kinks at 1 +- eps
    r = _rng(16)
    ratio = r.choice([0.5, 0.7, 0.9, 1.0, 1.1, 1.35, 1.6], size=logp0.shape)
    old = logp0 - np.log(ratio)
    loss, g, lse, _ = _loss_of(p, p["hidden"], p["W"], old, hrd["adv"], hrd["seg"])
    assert (g == 0).sum() > p["P"] * p["G"] * p["T"] - p["lens"].sum()     # some clipped tokens
    dH, dW = orc.pg_loss_bwd(p["hidden"], p["W"], p["ids"], p["lens"], lse, g, p["T"])
    h = 1e-6
    # d loss / d logp
    for n in range(0, logp0.size, 3):
        lp = logp0.copy(); lm = logp0.copy()
        lp[n] += h; lm[n] -= h
        fp, _, _ = orc.pg_loss_fwd(lp, old, hrd["adv"], hrd["seg"], p["lens"], p["P"], p["G"], p["T"], 0.2, 0.2, 0.3)
        fm, _, _ = orc.pg_loss_fwd(lm, old, hrd["adv"], hrd["seg"], p["lens"], p["P"], p["G"], p["T"], 0.2, 0.2, 0.3)
        assert abs((fp - fm) / (2 * h) - g[n]) < 1e-8
    for (arr, grad, name) in ((p["hidden"], dH, "hidden"), (p["W"], dW, "W")):
        fd = np.zeros_like(arr)
        for idx in np.ndindex(arr.shape):
            a = arr.copy(); a[idx] += h
            b = arr.copy(); b[idx] -= h
            if name == "hidden":
                fp = _loss_of(p, a, p["W"], old, hrd["adv"], hrd["seg"])[0]
                fm = _loss_of(p, b, p["W"], old, hrd["adv"], hrd["seg"])[0]
            else:
                fp = _loss_of(p, p["hidden"], a, old, hrd["adv"], hrd["seg"])[0]
                fm = _loss_of(p, p["hidden"], b, old, hrd["adv"], hrd["seg"])[0]
            fd[idx] = (fp - fm) / (2 * h)
        err = np.linalg.norm(fd - grad) / np.linalg.norm(grad)
        assert err < 1e-6, (name, err)


def test_backward_invariants_and_cross_entropy_special_case():
    p = _tiny_problem(17, P=1, G=2, T=6, H=4, V=9)
    N = p["G"] * p["T"]
    logp, lse = orc.token_logprobs(p["hidden"], p["W"], p["ids"], p["lens"], p["T"])
    g = _rng(18).standard_normal(N)
    valid = (np.arange(p["T"])[None, :] < p["lens"][:, None]).ravel()
    g[~valid] = 0
    dH, dW = orc.pg_loss_bwd(p["hidden"], p["W"], p["ids"], p["lens"], lse, g, p["T"])
    np.testing.assert_allclose(dW.sum(axis=0), 0, atol=1e-13)        # sum_v dS[n,v] = 0
    assert not dH[~valid].any()
    # with g = -1 this is the gradient of sum_n NLL_n: textbook (softmax - onehot)
    gm = np.where(valid, -1.0, 0.0)
    dH2, dW2 = orc.pg_loss_bwd(p["hidden"], p["W"], p["ids"], p["lens"], lse, gm, p["T"])
    dH_ref = np.zeros_like(dH2); dW_ref = np.zeros_like(dW2)
    for n in np.nonzero(valid)[0]:
        z = p["W"] @ p["hidden"][n]
        sm = np.exp(z - logsumexp(z))
        sm[p["ids"][n]] -= 1.0
        dH_ref[n] = sm @ p["W"]
        dW_ref += np.outer(sm, p["hidden"][n])
    np.testing.assert_allclose(dH2, dH_ref, atol=1e-13)
    np.testing.assert_allclose(dW2, dW_ref, atol=1e-13)
    # single-row helper agrees with the batched routine
    n = int(np.nonzero(valid)[0][3])
    np.testing.assert_allclose(orc.row_dhidden(p["hidden"][n], p["W"], p["ids"][n], g[n]), dH[n], atol=1e-13)


def test_backward_closed_form_at_uniform_logits():
    # W = 0: p = 1/V, dHidden = 0, dW[v] = sum_n g_n (1[v=id_n] - 1/V) hidden[n]
    r = _rng(19)
    T, H, V = 5, 3, 4
    hidden = r.standard_normal((T, H))
    ids = r.integers(0, V, T)
    g = r.standard_normal(T)
    dH, dW = orc.pg_loss_bwd(hidden, np.zeros((V, H)), ids, np.array([T]), np.full(T, math.log(V)), g, T)
    assert not dH.any()
    for v in range(V):
        for k in range(H):
            ref = sum(g[n] * ((1.0 if ids[n] == v else 0.0) - 1.0 / V) * hidden[n, k] for n in range(T))
            assert abs(dW[v, k] - ref) < 1e-14


@pytest.mark.parametrize("given_old", [False, True])
@pytest.mark.parametrize("opts", [dict(), dict(alpha=0.37, adv_mode=1), dict(clip_form=1, agg_mode=1, eps_lo=0.1, eps_hi=0.3),
                                  dict(alpha=0.0, eps_lo=0.3, eps_hi=0.05)])
def test_full_step_is_the_four_functions_wired_in_order(given_old, opts):
    """Every output of full_step equals the four pinned functions composed by hand: a wrong wiring
    (swapped policy / old-policy inputs, an option not passed on, lse of the wrong model in the
    backward, old_logp ignored or not) changes at least one of them."""
    p = _tiny_problem(20, P=2, G=4, T=7)
    P, G, T = p["P"], p["G"], p["T"]
    r = _rng(21)
    Wo = p["W"] + 0.3 * r.standard_normal(p["W"].shape) * p["H"] ** -0.5
    ho = p["hidden"] + 0.2 * r.standard_normal(p["hidden"].shape)
    given = (-r.random(P * G * T) * 3.0) if given_old else None
    out = orc.full_step(p["hidden"], p["W"], ho, Wo, p["ids"], p["lens"], p["bnd"], p["r_plan"], p["r_code"], P, G, T,
                        old_logp=given, **opts)
    logp, lse = orc.token_logprobs(p["hidden"], p["W"], p["ids"], p["lens"], T)
    old = given if given_old else orc.token_logprobs(ho, Wo, p["ids"], p["lens"], T)[0]
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], P, G, T, opts.get("adv_mode", 0))
    loss, g, stats = orc.pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T, opts.get("eps_lo", 0.2),
                                     opts.get("eps_hi", 0.2), opts.get("alpha", 0.1), opts.get("clip_form", 0),
                                     opts.get("agg_mode", 0))
    dH, dW = orc.pg_loss_bwd(p["hidden"], p["W"], p["ids"], p["lens"], lse, g, T)
    assert np.abs(g).max() > 0 and (not given_old or np.abs(old - orc.token_logprobs(ho, Wo, p["ids"], p["lens"], T)[0]).max() > 0.1)
    for k, v in dict(logp=logp, lse=lse, old_logp=old, g=g, stats=stats, dHidden=dH, dW=dW, seg=hrd["seg"],
                     adv=hrd["adv"], A_plan=hrd["A_plan"], A_code=hrd["A_code"], n_plan=hrd["n_plan"],
                     n_code=hrd["n_code"]).items():
        np.testing.assert_array_equal(out[k], v, err_msg=k)
    assert out["loss"] == loss and out["n_valid"] == hrd["n_valid"]
    # and the options do change the result (so passing them on is observable)
    if opts:
        base = orc.full_step(p["hidden"], p["W"], ho, Wo, p["ids"], p["lens"], p["bnd"], p["r_plan"], p["r_code"], P, G, T,
                             old_logp=given)
        assert base["loss"] != out["loss"]


def test_dW_rows_is_the_row_subset_of_the_full_gradient_and_matches_loops():
    """dW_rows against (i) the rows of pg_loss_bwd's dW (itself pinned by finite differences) with
    arbitrary lse / g inputs, including duplicated and never-sampled vocabulary rows, and (ii) plain
    Python loops over the definition."""
    p = _tiny_problem(40, P=2, G=3, T=6, H=5, V=13)
    T, V = p["T"], p["V"]
    r = _rng(41)
    N = p["P"] * p["G"] * T
    lse = r.standard_normal(N) + 2.0           # not the true lse on purpose: both routines take it as given
    g = r.standard_normal(N)
    _, dW = orc.pg_loss_bwd(p["hidden"], p["W"], p["ids"], p["lens"], lse, g, T)
    vsel = np.array([12, 0, 7, 7, 3])
    got = orc.dW_rows(p["hidden"], p["W"][vsel], vsel, p["ids"], p["lens"], lse, g, T)
    np.testing.assert_allclose(got, dW[vsel], atol=1e-13)
    for k, v in enumerate(vsel):
        for h in range(p["H"]):
            acc = 0.0
            for b in range(p["P"] * p["G"]):
                for t in range(p["lens"][b]):
                    n = b * T + t
                    z = sum(p["hidden"][n, q] * p["W"][v, q] for q in range(p["H"]))
                    acc += g[n] * ((1.0 if p["ids"][n] == v else 0.0) - math.exp(z - lse[n])) * p["hidden"][n, h]
            assert abs(got[k, h] - acc) < 1e-12


# ------------------------------------------------------------ documented variants of the loss

@pytest.mark.parametrize("s,A,u,active", [
    (1.5, 2.0, 2.0 * 1.2, False),     # same as the main form for A > 0
    (0.5, 2.0, 2.0 * 0.5, True),
    (1.5, -2.0, -2.0 * 1.2, False),   # A < 0: s above 1+eps saturates (unlike the main form)
    (0.5, -2.0, -2.0 * 0.5, True),    # A < 0: s below 1-eps does not saturate (unlike the main form)
])
def test_appendix_clip_form_single_token(s, A, u, active):
    loss, g, _ = orc.pg_loss_fwd(np.array([math.log(s) - 1.0]), np.array([-1.0]), np.array([A]),
                                 np.array([2], dtype=np.uint8), np.array([1]), 1, 1, 1, 0.2, 0.2, 0.1, clip_form=1)
    assert abs(loss + u) < 1e-14
    assert abs(g[0] - (-A * s if active else 0.0)) < 1e-14


def test_appendix_form_is_uniform_grpo_as_printed_and_fd_gradient():
    # alpha = 1, r_plan = r_code, clip_form = 1: L_GRPO of the appendix, A * min{s, clip(s)}, by loops
    p = _tiny_problem(31, P=2, G=4, T=8)
    P, G, T = p["P"], p["G"], p["T"]
    r = _rng(32)
    old = -r.random(P * G * T) * 4
    logp = old + r.standard_normal(P * G * T) * 0.3
    hu = orc.hrd_advantages(p["r_plan"], p["r_plan"], p["lens"], p["bnd"], P, G, T)
    lu, g, _ = orc.pg_loss_fwd(logp, old, hu["adv"], hu["seg"], p["lens"], P, G, T, 0.2, 0.2, 1.0, clip_form=1)
    J = 0.0
    for i in range(P):
        mu = sum(p["r_plan"][i * G + j] for j in range(G)) / G
        for j in range(G):
            b = i * G + j
            A = p["r_plan"][b] - mu
            acc = sum(A * min(math.exp(logp[b * T + t] - old[b * T + t]),
                              min(max(math.exp(logp[b * T + t] - old[b * T + t]), 0.8), 1.2))
                      for t in range(p["lens"][b]))
            J += acc / p["lens"][b] / G
    assert abs(lu + J / P) < 1e-13
    h = 1e-6
    for n in range(0, logp.size, 5):
        s = math.exp(logp[n] - old[n])
        if abs(s - 1.2) < 1e-3:
            continue
        lp = logp.copy(); lm = logp.copy()
        lp[n] += h; lm[n] -= h
        fp = orc.pg_loss_fwd(lp, old, hu["adv"], hu["seg"], p["lens"], P, G, T, 0.2, 0.2, 1.0, clip_form=1)[0]
        fm = orc.pg_loss_fwd(lm, old, hu["adv"], hu["seg"], p["lens"], P, G, T, 0.2, 0.2, 1.0, clip_form=1)[0]
        assert abs((fp - fm) / (2 * h) - g[n]) < 1e-8


def test_token_mean_aggregation_closed_form_and_fd():
    p = _tiny_problem(33, P=3, G=4, T=9)
    P, G, T = p["P"], p["G"], p["T"]
    hrd = orc.hrd_advantages(p["r_plan"], p["r_code"], p["lens"], p["bnd"], P, G, T)
    logp = -_rng(34).random(P * G * T) * 5
    alpha = 0.37
    loss, g, _ = orc.pg_loss_fwd(logp, logp.copy(), hrd["adv"], hrd["seg"], p["lens"], P, G, T, 0.2, 0.2, alpha, agg_mode=1)
    # s = 1: loss = -sum_b [alpha A_plan n_plan + A_code n_code] / sum_b len
    num = sum(alpha * hrd["A_plan"][b] * p["bnd"][b] + hrd["A_code"][b] * (p["lens"][b] - p["bnd"][b]) for b in range(P * G))
    assert abs(loss + num / p["lens"].sum()) < 1e-13
    h = 1e-6
    old = logp - 0.05
    _, g, _ = orc.pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T, 0.2, 0.2, alpha, agg_mode=1)
    for n in range(0, logp.size, 7):
        lp = logp.copy(); lm = logp.copy()
        lp[n] += h; lm[n] -= h
        fp = orc.pg_loss_fwd(lp, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T, 0.2, 0.2, alpha, agg_mode=1)[0]
        fm = orc.pg_loss_fwd(lm, old, hrd["adv"], hrd["seg"], p["lens"], P, G, T, 0.2, 0.2, alpha, agg_mode=1)[0]
        assert abs((fp - fm) / (2 * h) - g[n]) < 1e-8
