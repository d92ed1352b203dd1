"""Property tests of the oracle on random tiny problems (hypothesis): invariants that hold for
any input, complementing the fixed pins."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import trl_oracle as orc


@st.composite
def problems(draw):
    P, G = draw(st.integers(1, 3)), draw(st.integers(1, 4))
    T, H, V = draw(st.integers(1, 6)), draw(st.integers(1, 5)), draw(st.integers(2, 9))
    seed = draw(st.integers(0, 2 ** 31 - 1))
    r = np.random.default_rng(seed)
    B = P * G
    lens = r.integers(0, T + 1, B)
    bnd = np.array([r.integers(0, L + 1) for L in lens])
    return dict(P=P, G=G, T=T, H=H, V=V, hidden=r.standard_normal((B * T, H)), W=r.standard_normal((V, H)),
                ids=r.integers(0, V, B * T), lens=lens, bnd=bnd, r_plan=r.random(B) * 2, r_code=r.integers(0, 2, B).astype(float),
                old_shift=r.standard_normal(B * T) * 0.3, alpha=float(r.choice([0.0, 0.1, 1.0])))


@settings(max_examples=40, deadline=None)
@given(problems())
def test_invariants(p):
    P, G, T = p["P"], p["G"], p["T"]
    old_logp = orc.token_logprobs(p["hidden"], p["W"], p["ids"], p["lens"], T)[0] + p["old_shift"]
    out = orc.full_step(p["hidden"], p["W"], None, None, p["ids"], p["lens"], p["bnd"], p["r_plan"], p["r_code"], P, G, T,
                        alpha=p["alpha"], old_logp=old_logp)
    valid = (np.arange(T)[None, :] < p["lens"][:, None]).ravel()
    # padding: every per-token output is zero, every gradient row is zero
    for k in ("logp", "lse", "g", "adv"):
        assert not out[k][~valid].any()
    assert not out["seg"][~valid].any() and (out["seg"][valid] > 0).all()
    assert not out["dHidden"][~valid].any()
    # log-probs are <= 0 and lse >= max logit
    assert (out["logp"][valid] <= 1e-12).all()
    # advantages of a group sum to zero; segments partition the valid tokens
    assert np.allclose(out["A_plan"].reshape(P, G).sum(1), 0, atol=1e-12)
    assert np.allclose(out["A_code"].reshape(P, G).sum(1), 0, atol=1e-12)
    assert (out["n_plan"] + out["n_code"] == p["lens"]).all() and out["n_valid"] == p["lens"].sum()
    # sum_v dS[n,v] = 0  =>  column sums of dW vanish
    assert np.allclose(out["dW"].sum(0), 0, atol=1e-10)
    # g has the sign of -adv (or is zero), and is zero wherever adv is zero
    assert (out["g"] * out["adv"] <= 1e-300).all() and not out["g"][out["adv"] == 0].any()
    # the loss is what g predicts to first order: directional derivative along a random direction
    d = np.random.default_rng(1).standard_normal(out["logp"].shape) * valid
    h = 1e-7
    old = out["old_logp"]
    lp = orc.pg_loss_fwd(out["logp"] + h * d, old, out["adv"], out["seg"], p["lens"], P, G, T, alpha=p["alpha"])[0]
    lm = orc.pg_loss_fwd(out["logp"] - h * d, old, out["adv"], out["seg"], p["lens"], P, G, T, alpha=p["alpha"])[0]
    s = np.exp(out["logp"] - old)
    if np.abs(np.abs(s[valid] - 1.0) - 0.2).min(initial=1.0) > 1e-4:      # away from the clip kinks
        assert abs((lp - lm) / (2 * h) - float(out["g"] @ d)) < 1e-6


@settings(max_examples=25, deadline=None)
@given(problems(), st.floats(0.1, 10.0))
def test_scalings(p, c):
    P, G, T = p["P"], p["G"], p["T"]
    base = orc.full_step(p["hidden"], p["W"], p["hidden"], p["W"] * 0.97, p["ids"], p["lens"], p["bnd"], p["r_plan"],
                         p["r_code"], P, G, T, alpha=p["alpha"])
    scaled = orc.full_step(p["hidden"], p["W"], p["hidden"], p["W"] * 0.97, p["ids"], p["lens"], p["bnd"], c * p["r_plan"],
                           c * p["r_code"], P, G, T, alpha=p["alpha"])
    # everything downstream of the advantages is linear in a common reward scale
    assert np.isclose(scaled["loss"], c * base["loss"], rtol=1e-10, atol=1e-14)
    assert np.allclose(scaled["dW"], c * base["dW"], rtol=1e-9, atol=1e-13)
    assert np.allclose(scaled["dHidden"], c * base["dHidden"], rtol=1e-9, atol=1e-13)
    # scoring does not depend on the rewards at all
    assert np.array_equal(scaled["logp"], base["logp"])
