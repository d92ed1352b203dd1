"""Data-parallel plumbing for N > 1 ranks (one process per GPU).

The path shards by prompt group: every rank scores its own rollout groups with its own copy
of the LM head, so the data path has no exchange step; only the benchmark's bookkeeping
(time = max over ranks, tokens = sum over ranks) crosses ranks."""
import torch
import torch.distributed as dist


def rank_seed_offset(rank: int) -> int:
    """Seed offset that gives every rank a different synthetic batch of the same workload."""
    return int(rank)


def aggregate_throughput(elapsed_ms: float, tokens_per_step: int, steps: int, device="cpu"):
    """Whole-job tokens/s: (sum over ranks of tokens) * steps / (max over ranks of time).
    Works with any initialised backend (nccl with a CUDA device, gloo with "cpu"); with no
    process group it is the single-rank value.  Returns (tokens_per_s, max_ms, total_tokens)."""
    if dist.is_available() and dist.is_initialized():
        t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
        n = torch.tensor([int(tokens_per_step)], dtype=torch.int64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
        elapsed_ms, tokens_per_step = float(t.item()), int(n.item())
    return tokens_per_step * steps / (elapsed_ms * 1e-3), elapsed_ms, tokens_per_step
