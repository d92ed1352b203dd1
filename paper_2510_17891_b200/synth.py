"""Seeded synthetic rollout batches.

This module only *draws inputs*; it contains none of the method's arithmetic (no
log-softmax, no advantages, no loss).  Both the CUDA tests/benchmark and the CPU oracle
receive the arrays produced here.  The one matrix product below exists solely to sample
token ids from softmax(hidden W^T) with the Gumbel-max trick, as the workload recipe asks.

Workload recipe (stands in for Qwen3-8B rollouts on KernelBook prompts, which are not
available offline): hidden ~ N(0,1), W ~ N(0,1/H) so logits are ~N(0,1); ids sampled from
the policy's own softmax; valid lengths uniform in [len_lo*T, len_hi*T] with right padding;
the reasoning/code boundary at a uniform fraction f in [bnd_lo, bnd_hi] of the valid length
(or of T, clipped to the length, when `bnd_of_T`); plan / code rewards Bernoulli(p_plan),
Bernoulli(p_code) (optionally a fraction of prompts gets all-equal rewards);
the old policy pi_theta_old shares the hidden states and has a perturbed LM head,
W_old = W + sigma*N(0,1/H), which makes every logit differ by ~N(0, sigma) and hence the
log-prob differences ~N(0, sigma), sigma = 0.05.

Two generator-only knobs move the batch from this flat regime (no token above p ~ 1e-3) to the
peaked one of a trained policy, where most sampled tokens carry almost all the probability:
`logit_scale` multiplies the LM head (logits ~ N(0, logit_scale^2); the old policy's
perturbation is not scaled, so log-prob differences stay ~N(0, sigma)), and `greedy_ids`
takes ids = argmax of the logits instead of sampling.
"""
from dataclasses import dataclass, replace
import zlib

import torch

BASE_SEED = 20251017


@dataclass(frozen=True)
class Workload:
    name: str
    P: int
    G: int
    T: int
    H: int
    V: int
    dtype: str = "bf16"           # storage type of hidden / W: "bf16" or "f32"
    len_lo: float = 0.25
    len_hi: float = 1.0
    bnd_lo: float = 0.2
    bnd_hi: float = 0.8
    bnd_of_T: bool = False        # True: boundary = floor(f*T) clipped to len (literal reading)
    p_plan: float = 0.3
    p_code: float = 0.6
    degenerate_frac: float = 0.0  # fraction of prompts whose rewards are all equal
    real_plan_reward: bool = False  # plan reward Bernoulli * U(0.2, 2): the clipped speedup range
    sigma_old: float = 0.05
    logit_scale: float = 1.0      # W ~ N(0, logit_scale^2 / H): larger = more confident policy
    greedy_ids: bool = False      # ids = argmax of the logits instead of a sample from their softmax

    @property
    def B(self):
        return self.P * self.G

    @property
    def N(self):
        return self.P * self.G * self.T


# The five benchmark configurations (index = config number).
CONFIGS = {
    0: Workload("cfg0_tiny_f32", P=2, G=4, T=64, H=256, V=1024, dtype="f32",
                len_lo=0.5, len_hi=1.0, p_plan=0.5, p_code=0.5),
    1: Workload("cfg1_8b_fwd", P=8, G=8, T=2048, H=4096, V=151936),
    2: Workload("cfg2_8b_fwdbwd", P=8, G=8, T=2048, H=4096, V=151936),
    3: Workload("cfg3_long_reasoning", P=4, G=8, T=8192, H=4096, V=151936,
                len_lo=0.125, bnd_lo=0.5, bnd_hi=0.9),
    # one representative point of the config-4 sweep (the full grid is sweep_workloads())
    4: Workload("cfg4_V151936_H4096_G8", P=8, G=8, T=1024, H=4096, V=151936, degenerate_frac=0.25),
}


def sweep_workloads():
    """Config 4: 64 rollouts x T=1024 over the (V, H, G) grid, 25 % degenerate groups."""
    out = []
    for V in (32000, 65536, 151936, 256000):
        for H in (2048, 4096, 5120):
            for G in (4, 8, 16):
                out.append(Workload(f"cfg4_V{V}_H{H}_G{G}", P=64 // G, G=G, T=1024, H=H, V=V,
                                    degenerate_frac=0.25))
    return out


def scaled(w: Workload, **kw) -> Workload:
    """Same distributions, smaller shape (for element-by-element oracle comparisons)."""
    return replace(w, **kw)


def _gen(w: Workload, tensor: str, device, seed_offset=0):
    seed = (BASE_SEED + zlib.crc32(f"{w.name}/{tensor}".encode()) + seed_offset) % (2 ** 63 - 1)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _store_dtype(w: Workload):
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def sample_ids(hidden, W, gen, chunk_rows=2048, greedy=False):
    """ids[n] ~ Categorical(softmax(hidden[n] W^T)) by Gumbel-max, in row chunks (greedy: the
    argmax itself)."""
    N = hidden.shape[0]
    ids = torch.empty(N, dtype=torch.int32, device=hidden.device)
    mm_dtype = hidden.dtype if hidden.is_cuda else torch.float32
    Wm = W.to(mm_dtype)
    for r0 in range(0, N, chunk_rows):
        z = (hidden[r0:r0 + chunk_rows].to(mm_dtype) @ Wm.T).float()
        if not greedy:
            u = torch.rand(z.shape, generator=gen, device=z.device, dtype=torch.float32)
            u = u.clamp_(1e-20, 1.0 - 1e-7)
            z.sub_(torch.log(-torch.log(u)))
            del u
        ids[r0:r0 + chunk_rows] = z.argmax(dim=1).to(torch.int32)
        del z
    return ids


def make_batch(w: Workload, device="cpu", seed_offset=0, with_old_model=True):
    """Draw one batch.  Returns a dict of tensors on `device`:

    hidden [N,H], W [V,H] (storage dtype), hidden_old, W_old (same shapes; hidden_old is
    hidden itself), ids [N] i32, lens [B] i32, bnd [B] i32, r_plan [B] f32, r_code [B] f32,
    old_noise [N] f32 ~ N(0, sigma_old) (tests that supply old_logp explicitly add it to a
    log-prob vector of their own).
    """
    dev = torch.device(device)
    dt = _store_dtype(w)
    B, N, T, H, V = w.B, w.N, w.T, w.H, w.V

    hidden = torch.randn(N, H, generator=_gen(w, "hidden", dev, seed_offset), device=dev,
                         dtype=torch.float32).to(dt)
    W32 = torch.randn(V, H, generator=_gen(w, "W", dev, seed_offset), device=dev,
                      dtype=torch.float32).mul_(w.logit_scale * H ** -0.5)
    W = W32.to(dt)
    out = dict(hidden=hidden, W=W)
    if with_old_model:
        dW = torch.randn(V, H, generator=_gen(w, "W_old", dev, seed_offset), device=dev,
                         dtype=torch.float32).mul_(w.sigma_old * H ** -0.5)
        out["W_old"] = (W32 + dW).to(dt)
        out["hidden_old"] = hidden
        del dW
    del W32

    out["ids"] = sample_ids(hidden, W, _gen(w, "ids", dev, seed_offset), greedy=w.greedy_ids)

    gc = _gen(w, "lens", torch.device("cpu"), seed_offset)
    lo, hi = int(w.len_lo * T), int(w.len_hi * T)
    lens = torch.randint(lo, hi + 1, (B,), generator=gc, dtype=torch.int64)
    f = torch.rand(B, generator=gc, dtype=torch.float64) * (w.bnd_hi - w.bnd_lo) + w.bnd_lo
    if w.bnd_of_T:
        bnd = torch.minimum((f * T).floor().to(torch.int64), lens)
    else:
        bnd = (f * lens.double()).floor().to(torch.int64)
    r_plan = (torch.rand(B, generator=gc) < w.p_plan).float()
    if w.real_plan_reward:
        r_plan = r_plan * (torch.rand(B, generator=gc) * 1.8 + 0.2)
    r_code = (torch.rand(B, generator=gc) < w.p_code).float()
    if w.degenerate_frac > 0:
        n_deg = int(round(w.degenerate_frac * w.P))
        deg = torch.randperm(w.P, generator=gc)[:n_deg]
        for i in deg.tolist():
            r_plan[i * w.G:(i + 1) * w.G] = r_plan[i * w.G]
            r_code[i * w.G:(i + 1) * w.G] = r_code[i * w.G]
    out["lens"] = lens.to(torch.int32).to(dev)
    out["bnd"] = bnd.to(torch.int32).to(dev)
    out["r_plan"] = r_plan.to(dev)
    out["r_code"] = r_code.to(dev)
    out["old_noise"] = torch.randn(N, generator=_gen(w, "old_noise", dev, seed_offset), device=dev,
                                   dtype=torch.float32).mul_(w.sigma_old)
    return out
