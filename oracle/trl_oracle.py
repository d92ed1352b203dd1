"""fp64 CPU oracle for the HRD policy-gradient scoring path (TritonRL, Section 2.3).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the CUDA
library is checked against.  It shares no code with the CUDA path and must never be
imported by it; only tests, the smoke check and the benchmark's CPU-baseline leg call it.

Everything is numpy float64.  Inputs stored in a narrower type (bf16 / fp32) are
converted exactly to float64 by the caller before they arrive here.  There is no
blocking or fusion: the only loop is over rollouts (rows are independent), and the
matrix products are numpy `@`.

Notation (Section 2.3 and the notation appendix): P prompts q_i, G rollouts o_{i,j} per
prompt, B = P*G rollouts, each right-padded to T response tokens, N = B*T rows, row
n = b*T + t.  `lens[b]` = |o_{i,j}| is the number of valid tokens, `bnd[b]` the index of
the first code token: tokens t < bnd are the plan segment T^plan, bnd <= t < len the code
segment T^code.  `hidden[n,:]` is the final hidden state that predicts token `ids[n]`;
`W[v,:]` is the LM-head row of vocabulary entry v (no bias, temperature 1).

Parity pins: every function here is pinned by tests/test_oracle_pins.py (closed forms,
hand-worked fixtures under tests/golden/, finite differences, brute-force loops,
scipy's logsumexp).  No function is "parity unpinned".
"""
import numpy as np

SEG_PAD, SEG_PLAN, SEG_CODE = 0, 1, 2


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def token_logprobs(hidden, W, ids, lens, T):
    """log pi(o_t | .) of the sampled token and the log-partition, per row.

    The policy is the softmax over the vocabulary of z[n,v] = sum_k hidden[n,k] W[v,k]
    (the token probabilities pi_theta(o_{i,j,t} | q_i, o_{i,j,<t}) that enter the ratio
    s_{i,j,t} of Section 2.3).  lse[n] = log sum_v exp z[n,v], logp[n] = z[n,ids[n]] - lse[n].
    Padded rows (t >= lens[b]) get logp = lse = 0.

    Returns (logp[N], lse[N]) float64.
    """
    hidden = _f64(hidden)
    W = _f64(W)
    ids = np.asarray(ids, dtype=np.int64)
    lens = np.asarray(lens, dtype=np.int64)
    B = lens.shape[0]
    N = B * T
    assert hidden.shape[0] == N and ids.shape[0] == N
    logp = np.zeros(N, dtype=np.float64)
    lse = np.zeros(N, dtype=np.float64)
    for b in range(B):
        L = int(lens[b])
        if L == 0:
            continue
        rows = slice(b * T, b * T + L)
        z = hidden[rows] @ W.T                      # [L, V]
        m = z.max(axis=1)
        l = m + np.log(np.exp(z - m[:, None]).sum(axis=1))
        lse[rows] = l
        logp[rows] = z[np.arange(L), ids[rows]] - l
    return logp, lse


def hrd_advantages(r_plan, r_code, lens, bnd, P, G, T, adv_mode=0):
    """Hierarchical Reward Decomposition: segment labels and group-relative advantages.

    A^c_{i,j} = r^c_{i,j} - (1/G) sum_j r^c_{i,j}  for c in {plan, code}  (Section 2.3,
    the sentence introducing Eq. 2; also the notation appendix).  r^plan is the speedup
    reward, r^code the correctness reward (Eq. 2); both are inputs here.
    adv_mode 1 additionally divides by (population std of the group + 1e-6); the paper
    does not do this, it is the common GRPO variant and is kept as an option.

    seg[n] = 1 for plan tokens (t < bnd[b]), 2 for code tokens (bnd[b] <= t < lens[b]),
    0 for padding; adv[n] = A^plan or A^code of the rollout according to seg, 0 for padding.

    Returns dict with A_plan[B], A_code[B] (f64), seg[N] (u8), adv[N] (f64),
    n_plan[B], n_code[B] (i32), n_valid (int).
    """
    r_plan = _f64(r_plan)
    r_code = _f64(r_code)
    lens = np.asarray(lens, dtype=np.int64)
    bnd = np.asarray(bnd, dtype=np.int64)
    B = P * G
    assert r_plan.shape == (B,) and r_code.shape == (B,) and lens.shape == (B,) and bnd.shape == (B,)
    assert np.all((0 <= lens) & (lens <= T)) and np.all((0 <= bnd) & (bnd <= lens))

    def centred(r):
        A = np.empty(B, dtype=np.float64)
        for i in range(P):
            grp = r[i * G:(i + 1) * G]
            mu = grp.sum() / G
            a = grp - mu
            if adv_mode == 1:
                sd = np.sqrt(((grp - mu) ** 2).sum() / G)
                a = a / (sd + 1e-6)
            A[i * G:(i + 1) * G] = a
        return A

    A_plan = centred(r_plan)
    A_code = centred(r_code)
    seg = np.zeros(B * T, dtype=np.uint8)
    adv = np.zeros(B * T, dtype=np.float64)
    for b in range(B):
        o = b * T
        seg[o:o + bnd[b]] = SEG_PLAN
        seg[o + bnd[b]:o + lens[b]] = SEG_CODE
        adv[o:o + bnd[b]] = A_plan[b]
        adv[o + bnd[b]:o + lens[b]] = A_code[b]
    return dict(A_plan=A_plan, A_code=A_code, seg=seg, adv=adv,
                n_plan=bnd.astype(np.int32), n_code=(lens - bnd).astype(np.int32),
                n_valid=int(lens.sum()))


def pg_loss_fwd(logp, old_logp, adv, seg, lens, P, G, T, eps_lo=0.2, eps_hi=0.2, alpha=0.1, clip_form=0,
                agg_mode=0):
    """Clipped importance-ratio surrogate with the plan/code weighting, and d loss / d logp.

    J = (1/P) sum_i [ alpha J^plan_i + J^code_i ],
    J^c_i = (1/G) sum_j (1/|o_ij|) sum_{t in T^c_ij} min[ A s, A clip(s, 1-eps, 1+eps) ],
    s = pi_theta / pi_theta_old = exp(logp - old_logp)   (the two displayed objective
    equations of Section 2.3; the expectation over prompts is the mean over the P prompts
    of the call).  loss = -J.  Both classes are normalised by the full response length
    |o_ij| = lens[b]; rollouts with lens = 0 contribute nothing but still count in 1/G.

    g[n] = d loss / d logp[n] = -w A s / (P G len_b) when the unclipped branch is the
    minimum (A s <= A clip(s)), else 0; w = alpha for plan tokens, 1 for code tokens.

    clip_form 1 replaces the min by A * min{s, clip(s, 1-eps, 1+eps)}, the form printed in the
    appendix on uniform reward assignment (it differs from the above for A < 0).
    agg_mode 1 replaces the (1/P)(1/G)(1/|o|) weights by one mean over all valid tokens of the
    call (not in the paper).

    stats = [fraction of valid tokens with s > 1+eps_hi, fraction with s < 1-eps_lo,
             mean s over valid tokens, number of valid tokens].

    Returns (loss float, g[N] f64, stats[4] f64).
    """
    logp = _f64(logp)
    old_logp = _f64(old_logp)
    adv = _f64(adv)
    seg = np.asarray(seg)
    lens = np.asarray(lens, dtype=np.int64)
    B = P * G
    N = B * T
    assert logp.shape == (N,) and old_logp.shape == (N,) and adv.shape == (N,) and seg.shape == (N,)
    g = np.zeros(N, dtype=np.float64)
    J = 0.0
    n_hi = n_lo = 0
    sum_s = 0.0
    n_tok = 0
    n_total = int(np.clip(lens, 0, T).sum())
    for i in range(P):
        Ji = 0.0
        for j in range(G):
            b = i * G + j
            L = int(lens[b])
            if L == 0:
                continue
            rows = slice(b * T, b * T + L)
            s = np.exp(logp[rows] - old_logp[rows])
            A = adv[rows]
            w = np.where(seg[rows] == SEG_PLAN, alpha, np.where(seg[rows] == SEG_CODE, 1.0, 0.0))
            unclipped = A * s
            if clip_form == 0:
                clipped = A * np.clip(s, 1.0 - eps_lo, 1.0 + eps_hi)
                u = np.minimum(unclipped, clipped)
                active = unclipped <= clipped
            else:
                u = A * np.minimum(s, np.clip(s, 1.0 - eps_lo, 1.0 + eps_hi))
                active = s <= 1.0 + eps_hi
            norm = (P * G * L) if agg_mode == 0 else n_total
            Ji += (w * u).sum() / (L if agg_mode == 0 else 1.0)
            g[rows] = np.where(active, -w * A * s / norm, 0.0)
            n_hi += int((s > 1.0 + eps_hi).sum())
            n_lo += int((s < 1.0 - eps_lo).sum())
            sum_s += float(s.sum())
            n_tok += L
        J += Ji / (G if agg_mode == 0 else 1.0)
    J /= (P if agg_mode == 0 else max(n_total, 1))
    stats = np.array([n_hi / max(n_tok, 1), n_lo / max(n_tok, 1), sum_s / max(n_tok, 1), float(n_tok)])
    return -J, g, stats


def pg_loss_bwd(hidden, W, ids, lens, lse, g, T):
    """Gradient of the loss with respect to the LM-head inputs.

    Chain rule through logp[n] = z[n,ids[n]] - lse[n], z = hidden W^T:
      dS[n,v]    = g[n] (1[v = ids[n]] - exp(z[n,v] - lse[n]))
      dHidden[n] = sum_v dS[n,v] W[v,:]          dW[v] = sum_n dS[n,v] hidden[n,:]
    (the paper relies on automatic differentiation of the objective of Section 2.3; this is
    that derivative written out).  Padded rows of dHidden are exactly 0.

    Returns (dHidden[N,H] f64, dW[V,H] f64).
    """
    hidden = _f64(hidden)
    W = _f64(W)
    ids = np.asarray(ids, dtype=np.int64)
    lens = np.asarray(lens, dtype=np.int64)
    lse = _f64(lse)
    g = _f64(g)
    B = lens.shape[0]
    N = B * T
    V, H = W.shape
    dHidden = np.zeros((N, H), dtype=np.float64)
    dW = np.zeros((V, H), dtype=np.float64)
    for b in range(B):
        L = int(lens[b])
        if L == 0:
            continue
        rows = slice(b * T, b * T + L)
        z = hidden[rows] @ W.T
        dS = -np.exp(z - lse[rows][:, None])
        dS[np.arange(L), ids[rows]] += 1.0
        dS *= g[rows][:, None]
        dHidden[rows] = dS @ W
        dW += dS.T @ hidden[rows]
    return dHidden, dW


def row_dhidden(hidden_row, W, tok, g_n):
    """dHidden for one row from scratch (own lse), for sampled-row checks at full size."""
    W = _f64(W)
    z = W @ _f64(hidden_row)
    m = z.max()
    p = np.exp(z - (m + np.log(np.exp(z - m).sum())))
    dS = -p
    dS[int(tok)] += 1.0
    return g_n * (dS @ W)


def dW_rows(hidden, W_rows, vsel, ids, lens, lse, g, T):
    """Selected rows of dW: dW[v] = sum_n g[n] (1[v = ids[n]] - exp(z[n,v] - lse[n])) hidden[n,:] for
    v in `vsel`, summed over all valid rows n, with z[n,v] = hidden[n] . W_rows[k] for v = vsel[k]
    (the same chain rule as pg_loss_bwd, restricted to a few vocabulary rows so that it can be
    evaluated at full size).  `lse` and `g` are given per row.  Returns [len(vsel), H] float64."""
    hidden = _f64(hidden)
    W_rows = _f64(W_rows)
    vsel = np.asarray(vsel, dtype=np.int64)
    ids = np.asarray(ids, dtype=np.int64)
    lens = np.asarray(lens, dtype=np.int64)
    lse = _f64(lse)
    g = _f64(g)
    out = np.zeros((vsel.shape[0], hidden.shape[1]), dtype=np.float64)
    for b in range(lens.shape[0]):
        L = int(lens[b])
        if L == 0:
            continue
        rows = slice(b * T, b * T + L)
        z = hidden[rows] @ W_rows.T                                   # [L, len(vsel)]
        dS = (ids[rows][:, None] == vsel[None, :]).astype(np.float64) - np.exp(z - lse[rows][:, None])
        dS *= g[rows][:, None]
        out += dS.T @ hidden[rows]
    return out


def full_step(hidden, W, hidden_old, W_old, ids, lens, bnd, r_plan, r_code, P, G, T,
              eps_lo=0.2, eps_hi=0.2, alpha=0.1, adv_mode=0, old_logp=None, clip_form=0, agg_mode=0):
    """One pass of the whole path: score under pi_theta and pi_theta_old, HRD advantages,
    surrogate loss, backward.  If `old_logp` is given it replaces the pi_theta_old scoring."""
    logp, lse = token_logprobs(hidden, W, ids, lens, T)
    if old_logp is None:
        old_logp, _ = token_logprobs(hidden_old, W_old, ids, lens, T)
    hrd = hrd_advantages(r_plan, r_code, lens, bnd, P, G, T, adv_mode)
    loss, g, stats = pg_loss_fwd(logp, old_logp, hrd["adv"], hrd["seg"], lens, P, G, T, eps_lo, eps_hi, alpha,
                                 clip_form, agg_mode)
    dHidden, dW = pg_loss_bwd(hidden, W, ids, lens, lse, g, T)
    return dict(logp=logp, lse=lse, old_logp=old_logp, loss=loss, g=g, stats=stats,
                dHidden=dHidden, dW=dW, **hrd)
