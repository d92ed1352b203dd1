"""Data-parallel plumbing for N > 1 ranks (one process per GPU).

The path shards by prompt group: every rank scores its own rollout groups with its own copy
of the LM head, so scoring, advantages, loss and backward have no exchange step.  What a
data-parallel trainer exchanges afterwards is the LM-head gradient (and the scalar loss):
`allreduce_step_outputs` does that with the process group's all-reduce (NCCL over NVLink on
GPUs, gloo on CPU), in buckets so the first buckets can be reduced while later ones are
still being enqueued.  `BandedGradReducer` goes one step further together with
`trl_pg_step_fused_banded`: the dW GEMM finishes dW band by band and records an event per band,
and each band's all-reduce is started on a side stream behind that event while later bands are
still being computed.  The benchmark keeps both off by default (ranks are independent replicas
there); its bookkeeping (time = max over ranks, tokens = sum) is in `aggregate_throughput`."""
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


def allreduce_step_outputs(dW: torch.Tensor, loss: torch.Tensor, n_prompts_local: int, bucket_bytes: int = 256 << 20):
    """Combine the per-rank results of one step into the global-batch gradient and loss, in place.

    Each rank computed its loss as a mean over its own P_r prompts, so the global mean over
    sum_r P_r prompts is sum_r (P_r / P_total) * loss_r, and the same weights apply to dW.
    dW is reduced bucket by bucket with asynchronous all-reduces; the call returns when all of
    them have completed on the current stream.  Without a process group it is the identity.
    Returns the global number of prompts."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return n_prompts_local
    tot = torch.tensor([float(n_prompts_local)], dtype=torch.float64, device=dW.device)
    dist.all_reduce(tot, op=dist.ReduceOp.SUM)
    weight = n_prompts_local / float(tot.item())
    flat = dW.view(-1)
    flat.mul_(weight)
    loss.mul_(weight)
    step = max(1, bucket_bytes // flat.element_size())
    works = [dist.all_reduce(flat[i:i + step], op=dist.ReduceOp.SUM, async_op=True) for i in range(0, flat.numel(), step)]
    works.append(dist.all_reduce(loss, op=dist.ReduceOp.SUM, async_op=True))
    for wk in works:
        wk.wait()
    return int(round(tot.item()))


class BandedGradReducer:
    """Sums dW (and the loss) over the ranks band by band, each band as soon as it is final.

    Use with trl_pg_step_fused_banded: pass `band_begin` and `events` to it; when it has returned
    (everything is enqueued, nothing has run yet necessarily) call `start(loss)`: for every band j, in
    band order on every rank, the side stream waits for event j, scales rows
    band_begin[j]..band_begin[j+1] of dW by this rank's share of the prompts and starts their
    all-reduce.  `finish()` makes the current stream wait for all of them; call it before dW is
    read and before the next step overwrites it.  Each rank computed its loss and gradient as a mean
    over its own P_r prompts, so the global mean over sum_r P_r prompts is
    sum_r (P_r / P_total) * (rank r's result).

    On CPU tensors (gloo) there are no streams or events: the bands are reduced in the same order
    with the same weights, which is what the two-rank CPU test checks.  Without a process group
    (or with one rank) nothing is communicated and dW is left untouched.
    """

    def __init__(self, dW: torch.Tensor, band_begin, n_prompts_local: int, group=None):
        self.dW, self.band_begin, self.group = dW, list(band_begin), group
        self.active = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
        self.cuda = dW.is_cuda
        self.n_prompts_total = n_prompts_local
        self.weight = 1.0
        if self.active:                       # one-off host round trip; the prompt split is fixed for a run
            tot = torch.tensor([float(n_prompts_local)], dtype=torch.float64, device=dW.device)
            dist.all_reduce(tot, op=dist.ReduceOp.SUM, group=group)
            self.n_prompts_total = int(round(tot.item()))
            self.weight = n_prompts_local / float(self.n_prompts_total)
        n = len(self.band_begin) - 1
        self.events, self.side = None, None
        if self.cuda:
            self.events = [torch.cuda.Event() for _ in range(n)]
            for e in self.events:             # an event has a handle to pass on once it has been recorded
                e.record()
            self.side = torch.cuda.Stream(device=dW.device, priority=-1)
        self.works = []
        self.order = []                       # bands in the order their reduction was started (for tests)

    def start(self, loss: torch.Tensor):
        self.works, self.order = [], []
        if not self.active:
            return
        for j in range(len(self.band_begin) - 1):
            band = self.dW[self.band_begin[j]:self.band_begin[j + 1]]
            if self.cuda:
                self.side.wait_event(self.events[j])
                with torch.cuda.stream(self.side):
                    band.mul_(self.weight)
                    self.works.append(dist.all_reduce(band, op=dist.ReduceOp.SUM, group=self.group, async_op=True))
            else:
                band.mul_(self.weight)
                self.works.append(dist.all_reduce(band, op=dist.ReduceOp.SUM, group=self.group, async_op=True))
            self.order.append(j)
        loss.mul_(self.weight)
        self.works.append(dist.all_reduce(loss, op=dist.ReduceOp.SUM, group=self.group, async_op=True))

    def finish(self):
        for wk in self.works:
            wk.wait()
        self.works = []
