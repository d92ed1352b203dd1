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


def test_single_process_is_identity():
    tps, ms, tok = dp.aggregate_throughput(50.0, 1000, steps=2)
    assert (tps, ms, tok) == (1000 * 2 / 0.05, 50.0, 1000)
