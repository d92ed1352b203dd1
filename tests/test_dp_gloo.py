"""N > 1 bookkeeping with two gloo ranks on CPU: different batches per rank, whole-job
throughput = summed tokens over the slowest rank's time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2510_17891_b200 import dp, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.scaled(synth.CONFIGS[0], name="dp_cpu", H=32, V=64)
    batch = synth.make_batch(w, device="cpu", seed_offset=dp.rank_seed_offset(rank))
    tokens = int(batch["lens"].sum())
    elapsed = 10.0 * (rank + 1)                    # rank 1 is the slow one
    tps, max_ms, total = dp.aggregate_throughput(elapsed, tokens, steps=4)
    # gather every rank's token count and a fingerprint of its batch to check sharding
    info = [None] * world
    dist.all_gather_object(info, (tokens, float(batch["hidden"].double().sum())))
    if rank == 0:
        out.put((tps, max_ms, total, info))
    dist.destroy_process_group()


def test_two_rank_aggregation_and_distinct_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    tps, max_ms, total, info = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert max_ms == 20.0
    assert total == info[0][0] + info[1][0]
    assert abs(tps - total * 4 / 0.020) < 1e-6
    assert info[0][1] != info[1][1]                # the two ranks drew different batches


def _grad_worker(rank, world, port, out):
    """Each rank runs the fp64 oracle on its own prompts; the all-reduced gradient must equal the
    oracle run on the concatenated batch."""
    import numpy as np
    from oracle import trl_oracle as orc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    P_local = [1, 3][rank]                         # unequal shards: the weights matter
    w = synth.scaled(synth.CONFIGS[0], name="dp_grad", P=P_local, G=2, T=6, H=8, V=12)
    b = synth.make_batch(w, device="cpu", seed_offset=dp.rank_seed_offset(rank))
    f = lambda t: t.double().numpy()
    # every rank must use the same LM head: take rank 0's
    Ws = [b["W"].clone(), b["W_old"].clone()]
    for t in Ws:
        dist.broadcast(t, src=0)
    ref = orc.full_step(f(b["hidden"]), f(Ws[0]), f(b["hidden"]), f(Ws[1]), b["ids"].numpy(), b["lens"].numpy(),
                        b["bnd"].numpy(), f(b["r_plan"]), f(b["r_code"]), w.P, w.G, w.T)
    dW = torch.tensor(ref["dW"])
    loss = torch.tensor([ref["loss"]], dtype=torch.float64)
    total_P = dp.allreduce_step_outputs(dW, loss, w.P, bucket_bytes=64)     # tiny buckets: several all-reduces
    parts = [None] * world
    dist.all_gather_object(parts, {k: (v.numpy() if torch.is_tensor(v) else v) for k, v in b.items()})
    if rank == 0:
        cat = {k: np.concatenate([p[k] for p in parts]) for k in ("hidden", "ids", "lens", "bnd", "r_plan", "r_code")}
        full = orc.full_step(cat["hidden"].astype(np.float64), f(Ws[0]), cat["hidden"].astype(np.float64), f(Ws[1]),
                             cat["ids"], cat["lens"], cat["bnd"], cat["r_plan"].astype(np.float64),
                             cat["r_code"].astype(np.float64), total_P, w.G, w.T)
        out.put((total_P, float(loss), full["loss"], float(np.abs(dW.numpy() - full["dW"]).max()),
                 float(np.abs(full["dW"]).max())))
    dist.destroy_process_group()


def test_allreduced_gradient_equals_global_batch_oracle():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_grad_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    total_P, loss, full_loss, err, scale = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert total_P == 4
    assert abs(loss - full_loss) < 1e-12
    assert err < 1e-12 * max(scale, 1.0)


def test_single_process_is_identity():
    tps, ms, tok = dp.aggregate_throughput(50.0, 1000, steps=2)
    assert (tps, ms, tok) == (1000 * 2 / 0.05, 50.0, 1000)
