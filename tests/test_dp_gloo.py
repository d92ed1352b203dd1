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


def _banded_worker(rank, world, port, out):
    """The banded reducer on two CPU ranks with unequal shards: bands are reduced in band order with
    weights P_r / P_total, and the result equals the oracle on the concatenated batch."""
    import numpy as np
    from oracle import trl_oracle as orc
    import paper_2510_17891_b200 as trl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    P_local = [3, 1][rank]
    w = synth.scaled(synth.CONFIGS[0], name="dp_banded", P=P_local, G=2, T=6, H=8, V=1000)
    b = synth.make_batch(w, device="cpu", seed_offset=dp.rank_seed_offset(rank))
    f = lambda t: t.double().numpy()
    Ws = [b["W"].clone(), b["W_old"].clone()]
    for t in Ws:
        dist.broadcast(t, src=0)
    ref = orc.full_step(f(b["hidden"]), f(Ws[0]), f(b["hidden"]), f(Ws[1]), b["ids"].numpy(), b["lens"].numpy(),
                        b["bnd"].numpy(), f(b["r_plan"]), f(b["r_code"]), w.P, w.G, w.T)
    dW = torch.tensor(ref["dW"])
    local = dW.clone()
    loss = torch.tensor([ref["loss"]], dtype=torch.float64)
    bands = trl.trl_dw_band_plan(w.V, w.H, 3)          # the library's own split (host-only call)
    red = dp.BandedGradReducer(dW, bands, w.P)
    red.start(loss)
    red.finish()
    parts = [None] * world
    dist.all_gather_object(parts, dict(local=local.numpy(), P=w.P,
                                       **{k: v.numpy() for k, v in b.items() if k in ("hidden", "ids", "lens", "bnd", "r_plan", "r_code")}))
    if rank == 0:
        cat = {k: np.concatenate([p[k] for p in parts]) for k in ("hidden", "ids", "lens", "bnd", "r_plan", "r_code")}
        Pt = sum(p["P"] for p in parts)
        full = orc.full_step(cat["hidden"].astype(np.float64), f(Ws[0]), cat["hidden"].astype(np.float64), f(Ws[1]),
                             cat["ids"], cat["lens"], cat["bnd"], cat["r_plan"].astype(np.float64),
                             cat["r_code"].astype(np.float64), Pt, w.G, w.T)
        weighted = sum(p["local"] * (p["P"] / Pt) for p in parts)
        out.put(dict(bands=bands, order=red.order, P_total=red.n_prompts_total, weight=red.weight,
                     err_oracle=float(np.abs(dW.numpy() - full["dW"]).max()), scale=float(np.abs(full["dW"]).max()),
                     err_weighted=float(np.abs(dW.numpy() - weighted).max()), loss=float(loss), full_loss=full["loss"]))
    dist.destroy_process_group()


def test_banded_reducer_band_order_weights_and_global_batch_oracle():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_banded_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    bands = res["bands"]
    assert bands[0] == 0 and bands[-1] == 1000 and all(b % 256 == 0 for b in bands[:-1]) and len(bands) >= 3
    assert res["order"] == list(range(len(bands) - 1))           # band order, the same on every rank
    assert res["P_total"] == 4 and abs(res["weight"] - 0.75) < 1e-15
    assert res["err_weighted"] < 1e-15 * max(res["scale"], 1.0) + 1e-18
    assert res["err_oracle"] < 1e-12 * max(res["scale"], 1.0)
    assert abs(res["loss"] - res["full_loss"]) < 1e-12


def test_banded_reducer_without_a_process_group_leaves_dW_alone():
    dW = torch.arange(12.0).reshape(6, 2)
    loss = torch.ones(1)
    red = dp.BandedGradReducer(dW.clone(), [0, 4, 6], 5)
    red.start(loss)
    red.finish()
    assert torch.equal(red.dW, dW) and float(loss) == 1.0 and red.order == []


def test_single_process_is_identity():
    tps, ms, tok = dp.aggregate_throughput(50.0, 1000, steps=2)
    assert (tps, ms, tok) == (1000 * 2 / 0.05, 50.0, 1000)
