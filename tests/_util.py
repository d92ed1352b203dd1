"""Shared helpers for the parity tests (no method arithmetic here)."""
import numpy as np
import torch


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


def oracle_inputs(batch):
    """Exact float64 / integer numpy copies of a synthetic batch."""
    out = {}
    for k, v in batch.items():
        out[k] = f64(v) if v.is_floating_point() else v.cpu().numpy()
    return out


def rel_fro(a, ref):
    return float(np.linalg.norm(np.asarray(a, dtype=np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))


# tolerances of the parity bar
TOL_LOGP = 5e-3       # |delta logp| per token
TOL_LOSS = 1e-3       # relative
TOL_GRAD = 1e-2       # relative Frobenius, dHidden and dW
