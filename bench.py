#!/usr/bin/env python
"""Benchmark of the HRD policy-gradient scoring path on B200.

A step is one pass of the whole path over one synthetic batch: scoring under the current
and the old policy, HRD advantages, clipped surrogate, backward to dHidden and dW.
Metric: scored (valid) rollout tokens per second, fwd+bwd, at H=4096, V=151,936.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 is launched with torch.distributed.run (one rank per GPU); ranks process independent
batches (weak scaling, no data-path collective); time is the max over ranks.
`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "scored_rollout_tokens_per_sec_fwd_bwd"
UNIT = "tokens/s"
WORKLOAD_ID = 2          # 8B-scale fwd+bwd: 8 prompts x 8 rollouts, T=2048, H=4096, V=151,936
# DRAM bytes (read + write) of one tc_gemm_kernel<LSE> launch at WORKLOAD_ID, from a one-pass ncu
# capture (dram__bytes_read.sum + dram__bytes_write.sum) of that launch inside this very command:
# 28.14 GB read + 0.42 GB written = the packed hidden rows once + W once per raster band of 32 row
# blocks (22 bands); the capture's summary is committed under profiles/
LSE_TRAFFIC_BYTES = 2.856e10


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        out = dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                   source="measured")
        mhz = (p.get("clocks_under_load") or {}).get("sm_mhz_median")
        if mhz:
            out["sm_mhz_at_peak"] = mhz           # SM clock the sustained figure was measured at
        return out
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], None, [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax = float(f[2]); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=smax,
                    power_w_max=max(power) if power else None, samples=len(sm), reasons=sorted(reasons))


def oracle_sample_throughput(w, rollouts, T_sample, seed_offset=0):
    """Time the fp64 oracle, as it stands, on `rollouts` rollouts of length T_sample with the
    full H and V of workload `w`.  Returns (tokens/s, tokens, seconds, threads)."""
    import numpy as np
    import torch
    from threadpoolctl import threadpool_info
    from oracle import trl_oracle as orc
    from paper_2510_17891_b200 import synth
    ws = synth.scaled(w, name=w.name + "_cpu_sample", P=1, G=rollouts, T=T_sample)
    b = synth.make_batch(ws, device="cpu", seed_offset=seed_offset)
    f64 = lambda t: t.to(torch.float64).numpy()
    hidden, W, W_old = f64(b["hidden"]), f64(b["W"]), f64(b["W_old"])
    ids, lens, bnd = b["ids"].numpy(), b["lens"].numpy(), b["bnd"].numpy()
    rp, rc = f64(b["r_plan"]), f64(b["r_code"])
    t0 = time.perf_counter()
    orc.full_step(hidden, W, hidden, W_old, ids, lens, bnd, rp, rc, 1, rollouts, T_sample)
    dt = time.perf_counter() - t0
    threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    tokens = int(lens.sum())
    return tokens / dt, tokens, dt, threads


def run_reference(args, rank, world):
    """Reference arm = the oracle on the host cores (rank 0 only).  One batch of short rollouts
    with the full H and V is drawn once; every step runs the whole path on two of them."""
    if rank != 0:
        return
    import torch
    from threadpoolctl import threadpool_info
    from oracle import trl_oracle as orc
    from paper_2510_17891_b200 import synth
    w = synth.CONFIGS[WORKLOAD_ID]
    per_step, T_sample = 2, 16
    n_steps = args.steps + args.warmup
    ws = synth.scaled(w, name=w.name + "_cpu_reference", P=n_steps, G=per_step, T=T_sample)
    b = synth.make_batch(ws, device="cpu")
    f64 = lambda t: t.to(torch.float64).numpy()
    W, W_old, hidden = f64(b["W"]), f64(b["W_old"]), f64(b["hidden"])
    ids, lens, bnd = b["ids"].numpy(), b["lens"].numpy(), b["bnd"].numpy()
    rp, rc = f64(b["r_plan"]), f64(b["r_code"])
    tok = 0
    sec = 0.0
    for i in range(n_steps):
        r = slice(i * per_step, (i + 1) * per_step)
        rows = slice(i * per_step * T_sample, (i + 1) * per_step * T_sample)
        t0 = time.perf_counter()
        orc.full_step(hidden[rows], W, hidden[rows], W_old, ids[rows], lens[r], bnd[r], rp[r], rc[r], 1, per_step, T_sample)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            tok += int(lens[r].sum()); sec += dt
    threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    value = tok / sec
    sample = (f"{per_step} rollouts x T={T_sample} per step (valid tokens only), full H={w.H} V={w.V}, "
              f"policy + old-policy scoring, advantages, loss, backward in numpy fp64")
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=1e3 * sec / max(args.steps, 1), higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic", impl="reference",
                config=dict(workload=w.name, P=w.P, G=w.G, T=w.T, H=w.H, V=w.V, note="oracle on a bounded sample"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=threads, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def run_reductions(trl, torch, dev, peaks, args):
    """HBM roofline of the memory-bound calls at a size where launch latency no longer hides it:
    512 rollouts x 131,072 tokens = 2^26 tokens (the benchmark configs move < 5 MB through them)."""
    P, G, T = 64, 8, 131072
    B, N = P * G, P * G * T
    g = torch.Generator(device=dev).manual_seed(1)
    lens = torch.randint(T // 4, T + 1, (B,), generator=g, device=dev, dtype=torch.int32)
    bnd = (lens.float() * (0.2 + 0.6 * torch.rand(B, generator=g, device=dev))).to(torch.int32)
    r_plan = (torch.rand(B, generator=g, device=dev) < 0.3).float()
    r_code = (torch.rand(B, generator=g, device=dev) < 0.6).float()
    old = -torch.rand(N, generator=g, device=dev) * 5
    logp = old + 0.05 * torch.randn(N, generator=g, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    hrd = trl.trl_hrd_advantages(r_plan, r_code, lens, bnd, P, G, T, status=status)
    loss, gg, stats = trl.trl_pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], lens, P, G, T, status=status)
    ws = torch.empty(trl.trl_workspace_bytes(trl.TRL_CALL_PG_LOSS_FWD, B, T, 1, 1, trl.TRL_F32), dtype=torch.uint8, device=dev)
    n_valid = int(lens.sum())

    def timed(fn, n=20):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    t_adv = timed(lambda: trl.trl_hrd_advantages(r_plan, r_code, lens, bnd, P, G, T, 0, hrd, status))
    t_loss = timed(lambda: trl.trl_pg_loss_fwd(logp, old, hrd["adv"], hrd["seg"], lens, P, G, T, 0.2, 0.2, 0.1,
                                               loss, gg, stats, ws, status))
    trl.check_status(status)
    # algorithmic bytes: advantages write seg (1 B) + adv (4 B) per padded token; the loss reads
    # logp, old_logp, adv (12 B) + seg (1 B) per valid token and writes g (4 B) per padded token
    b_adv = 5.0 * N
    b_loss = 13.0 * n_valid + 4.0 * N
    line = dict(metric="reduction_kernels_hbm", tokens=N, valid_tokens=n_valid,
                hrd_advantages=dict(ms=t_adv, bytes=b_adv, gbs=b_adv / t_adv / 1e6, frac=b_adv / t_adv / 1e6 / peaks["hbm_gbs"]),
                pg_loss_fwd=dict(ms=t_loss, bytes=b_loss, gbs=b_loss / t_loss / 1e6, frac=b_loss / t_loss / 1e6 / peaks["hbm_gbs"]),
                peak_gbs=peaks["hbm_gbs"], peak_source=peaks["source"] + " copy bandwidth")
    print(json.dumps(line))


class StepRunner:
    """Preallocated buffers and the C-ABI call sequence of one step for one workload."""

    def __init__(self, trl, torch, w, batch, dev, path, dist=None, dp_allreduce=False):
        self.trl, self.torch, self.w, self.batch, self.dev, self.path = trl, torch, w, batch, dev, path
        self.dist, self.dp_allreduce = dist, dp_allreduce
        B, T, H, V = w.B, w.T, w.H, w.V
        dt_code = trl.TRL_BF16 if w.dtype == "bf16" else trl.TRL_F32
        f32 = dict(dtype=torch.float32, device=dev)
        ws = lambda call: torch.empty(max(trl.trl_workspace_bytes(call, B, T, H, V, dt_code), 256), dtype=torch.uint8, device=dev)
        # preallocated outputs and workspaces (the library allocates nothing)
        self.bufs = dict(logp=torch.empty(B * T, **f32), lse=torch.empty(B * T, **f32), old_logp=torch.empty(B * T, **f32),
                         old_lse=torch.empty(B * T, **f32), loss=torch.empty(1, **f32), g=torch.empty(B * T, **f32),
                         stats=torch.empty(4, **f32), dHidden=torch.empty_like(batch["hidden"]),
                         dW=torch.empty(V, H, **f32), ws_fwd=ws(trl.TRL_CALL_TOKEN_LOGPROBS),
                         ws_loss=ws(trl.TRL_CALL_PG_LOSS_FWD),
                         ws_bwd=ws(trl.TRL_CALL_PG_LOSS_BWD if path == "four_call" else trl.TRL_CALL_PG_STEP_FUSED)
                         if not (dp_allreduce and path == "fused") else None)
        # data-parallel training: dW is finished band by band and every band is all-reduced on a side
        # stream as soon as it is final (with one rank: the banded schedule alone)
        self.reducer = None
        if dp_allreduce and path == "fused":
            from paper_2510_17891_b200 import dp
            self.rows_bound = int(batch["lens"].sum().item())
            self.bufs["ws_bwd"] = torch.empty(trl.trl_pg_step_fused_banded_workspace_bytes(B, T, H, V, self.rows_bound),
                                              dtype=torch.uint8, device=dev)
            self.reducer = dp.BandedGradReducer(self.bufs["dW"], trl.trl_dw_band_plan(V, H, 16), w.P)
        self.fused_out = {k: self.bufs[k] for k in ("logp", "lse", "g", "loss", "stats", "dHidden", "dW")}
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.stream = torch.cuda.current_stream()
        self.names = (["token_logprobs_old", "hrd_advantages", "pg_step_fused"] if path == "fused" else
                      ["token_logprobs_policy", "token_logprobs_old", "hrd_advantages", "pg_loss_fwd", "pg_loss_bwd"])

    def rec(self):
        e = self.torch.cuda.Event(enable_timing=True)
        e.record(self.stream)
        return e

    def step(self, ev=None, batch=None):
        """One pass of the whole path.  `ev` collects CUDA events around each C-ABI call."""
        trl, w, bufs, status, stream = self.trl, self.w, self.bufs, self.status, self.stream
        batch = self.batch if batch is None else batch
        P, G, T = w.P, w.G, w.T
        mark = (lambda: None) if ev is None else (lambda: ev.append(self.rec()))
        mark()
        if self.path == "four_call":
            trl.trl_token_logprobs(batch["hidden"], batch["W"], batch["ids"], batch["lens"], T, bufs["logp"], bufs["lse"],
                                   bufs["ws_fwd"], status, stream)
            mark()
        trl.trl_token_logprobs(batch["hidden_old"], batch["W_old"], batch["ids"], batch["lens"], T, bufs["old_logp"],
                               bufs["old_lse"], bufs["ws_fwd"], status, stream)
        mark()
        hrd = trl.trl_hrd_advantages(batch["r_plan"], batch["r_code"], batch["lens"], batch["bnd"], P, G, T, 0,
                                     bufs.get("hrd"), status, stream)
        bufs["hrd"] = hrd
        mark()
        if self.reducer is not None:
            self.reducer.finish()          # the previous step's dW is reduced before this step overwrites it
            trl.trl_pg_step_fused_banded(batch["hidden"], batch["W"], batch["ids"], batch["lens"], bufs["old_logp"],
                                         bufs["old_lse"], hrd["adv"], hrd["seg"], P, G, T, self.reducer.band_begin,
                                         self.reducer.events, self.rows_bound, 0.2, 0.2, 0.1, self.fused_out, bufs["ws_bwd"],
                                         status, stream)
            self.reducer.start(bufs["loss"])
            self.reducer.finish()
        elif self.path == "fused":
            trl.trl_pg_step_fused(batch["hidden"], batch["W"], batch["ids"], batch["lens"], bufs["old_logp"], bufs["old_lse"],
                                  hrd["adv"], hrd["seg"], P, G, T, 0.2, 0.2, 0.1, self.fused_out, bufs["ws_bwd"], status, stream)
        else:
            trl.trl_pg_loss_fwd(bufs["logp"], bufs["old_logp"], hrd["adv"], hrd["seg"], batch["lens"], P, G, T, 0.2, 0.2, 0.1,
                                bufs["loss"], bufs["g"], bufs["stats"], bufs["ws_loss"], status, stream)
            mark()
            trl.trl_pg_loss_bwd(batch["hidden"], batch["W"], batch["ids"], batch["lens"], bufs["lse"], bufs["g"], T,
                                bufs["dHidden"], bufs["dW"], bufs["ws_bwd"], status, stream)
        mark()
        if self.dp_allreduce and self.reducer is None and self.dist is not None:      # four_call: all-reduce after the step
            from paper_2510_17891_b200 import dp
            dp.allreduce_step_outputs(bufs["dW"], bufs["loss"], P)

    def timed(self, steps, warmup, barrier):
        """`warmup` untimed steps, then `steps` steps between two events.  Returns (elapsed ms,
        per-call mean ms)."""
        for _ in range(warmup):
            self.step()
        self.torch.cuda.synchronize()
        self.trl.check_status(self.status)
        barrier()
        call_events = []
        t_start = self.rec()
        for _ in range(steps):
            ev = []
            self.step(ev)
            call_events.append(ev)
        t_end = self.rec()
        barrier()
        self.trl.check_status(self.status)
        call_ms = {n: statistics.mean(ev[i].elapsed_time(ev[i + 1]) for ev in call_events) for i, n in enumerate(self.names)}
        return t_start.elapsed_time(t_end), call_ms


def per_ghz(tflops, sm_mhz):
    return None if not sm_mhz else tflops / (sm_mhz * 1e-3)


def side_run(trl, torch, synth, dev, workload_id, path, peaks, barrier, steps=3, warmup=3):
    """A short timed run of another workload / schedule, reported under `other_runs` (not a headline).
    `workload_id` is a config number or a synth.Workload."""
    w = synth.CONFIGS[workload_id] if isinstance(workload_id, int) else workload_id
    batch = synth.make_batch(w, device=dev)
    batch["hidden_old"] = batch["hidden"].clone()
    n_valid = int(batch["lens"].sum().item())
    r = StepRunner(trl, torch, w, batch, dev, path)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    ms, call_ms = r.timed(steps, warmup, barrier)
    clocks = sampler.stop()
    tok_s = n_valid * steps / (ms * 1e-3)
    tf = 6.0 * w.H * w.V * tok_s / 1e12
    out = dict(workload=w.name, path=path, steps=steps, warmup=warmup, tokens_per_s=tok_s, ms_per_step=ms / steps,
               valid_tokens=n_valid, tflops_6NHV=tf, tflops_6NHV_per_ghz=per_ghz(tf, clocks.get("sm_mhz")),
               pct_of_nominal_bf16=100 * tf / 2250.0, pct_of_measured_sustained=100 * tf / peaks["bf16_sustained"],
               calls_ms=call_ms, sm_mhz=clocks.get("sm_mhz"), reasons=clocks.get("reasons"))
    del r, batch
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=WORKLOAD_ID, help="config number (default: the metric's)")
    ap.add_argument("--small-case", action="store_true",
                    help="run a 3 GB case of the same kernels instead (8 rollouts x T=2048, H=4096, V=32,768): "
                         "the size multi-pass profiler captures are taken on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-runs", action="store_true",
                    help="skip the short side runs (config 3 fused, config 2 four-call) that fill `other_runs`")
    ap.add_argument("--reductions", action="store_true",
                    help="time the two memory-bound calls (HRD advantages, surrogate loss) alone at 2^26 tokens")
    ap.add_argument("--sweep", action="store_true",
                    help="time the fused step on the 12 (V, H) shapes of the config-4 sweep (64 rollouts x T=1024, G=8, "
                         "25 %% all-equal reward groups) and print one JSON line with all of them")
    ap.add_argument("--dp-allreduce", action="store_true",
                    help="data-parallel training: run the banded schedule (dW final band by band) and, with N > 1, "
                         "all-reduce every band of dW and the loss across ranks on a side stream as it becomes final")
    ap.add_argument("--path", default="fused", choices=["fused", "four_call"],
                    help="fused: old-policy scoring, advantages, trl_pg_step_fused; four_call: the separate calls")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import paper_2510_17891_b200 as trl
    from paper_2510_17891_b200 import synth, dp
    trl.load_library()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    peaks = load_peaks()
    if args.reductions:
        run_reductions(trl, torch, dev, peaks, args)
        return
    if args.sweep:
        runs = [side_run(trl, torch, synth, dev, w4, args.path, peaks, lambda: torch.cuda.synchronize(),
                         steps=min(args.steps, 6), warmup=3)
                for w4 in synth.sweep_workloads() if w4.G == 8]
        print(json.dumps(dict(metric="config4_sweep_" + METRIC, unit=UNIT, path=args.path, runs=runs)))
        return
    w = synth.CONFIGS[args.workload]
    if args.small_case:
        w = synth.scaled(synth.CONFIGS[WORKLOAD_ID], name="small_case", P=1, G=8, T=2048, H=4096, V=32768)
    batch = synth.make_batch(w, device=dev, seed_offset=dp.rank_seed_offset(rank))
    batch["hidden_old"] = batch["hidden"].clone()        # the old policy's own activation buffer
    B, T, H, V, P, G = w.B, w.T, w.H, w.V, w.P, w.G
    n_valid = int(batch["lens"].sum().item())
    runner = StepRunner(trl, torch, w, batch, dev, args.path, dist, args.dp_allreduce)
    bufs, stream, step = runner.bufs, runner.stream, runner.step

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    launches0 = None
    warm = max(args.warmup, 3)
    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    launches0 = trl.trl_kernel_launches()
    sampler = ClockSampler(local_rank)
    sampler.start()
    elapsed_local, call_ms = runner.timed(args.steps, 0, barrier)
    clocks = sampler.stop()
    launches = trl.trl_kernel_launches() - launches0
    value, elapsed_ms, total_valid = dp.aggregate_throughput(elapsed_local, n_valid, args.steps, dev)

    # ---- end-to-end: host buffers in, loss out, copies inside the timed region.  Every step's
    # inputs (both models' hidden states, ids, len, bnd, rewards) come from pinned host memory
    # and its loss + statistics go back to the host; the upload of step i+1 runs on a copy
    # stream into a second set of device buffers while step i computes (what a trainer does).
    in_keys = ("hidden", "hidden_old", "ids", "lens", "bnd", "r_plan", "r_code")
    host = {k: batch[k].cpu().pin_memory() for k in in_keys}
    host_out = torch.empty(5, dtype=torch.float32).pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = host_out.numel() * 4
    e2e_steps = max(2, min(args.steps, 8))
    sets = [batch, {**batch, **{k: torch.empty_like(batch[k]) for k in in_keys}}]
    copy_stream = torch.cuda.Stream()
    uploaded = [torch.cuda.Event(), torch.cuda.Event()]
    consumed = [torch.cuda.Event(), torch.cuda.Event()]

    def upload(i):
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[i % 2])        # the step that last read this set has finished
            for k, v in host.items():
                sets[i % 2][k].copy_(v, non_blocking=True)
            uploaded[i % 2].record(copy_stream)

    def e2e_run(n):
        for e in consumed:
            e.record(stream)
        upload(0)
        for i in range(n):
            if i + 1 < n:
                upload(i + 1)
            stream.wait_event(uploaded[i % 2])
            step(None, sets[i % 2])
            consumed[i % 2].record(stream)
            host_out[:1].copy_(bufs["loss"], non_blocking=True)
            host_out[1:].copy_(bufs["stats"], non_blocking=True)
            stream.synchronize()                           # the step's result is on the host

    e2e_run(2)
    barrier()
    t0 = time.perf_counter()
    e2e_run(e2e_steps)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_value, _, _ = dp.aggregate_throughput(1e3 * e2e_s, n_valid, e2e_steps, dev)
    del sets, host

    # ---- roofline of the dominant kernel: the tcgen05 GEMM with the log-sum-exp epilogue
    # (the largest single launch of the step).  Its launch is timed through the
    # trl_token_logprobs call that contains it (plus two sub-millisecond helper kernels).
    flops_fwd = 2.0 * H * V * n_valid
    t_fwd_ms = call_ms["token_logprobs_old"]
    achieved = flops_fwd / (t_fwd_ms * 1e-3) / 1e12
    peak = peaks["bf16_sustained"]
    sm_mhz = clocks.get("sm_mhz")
    roofline = dict(bound="tensor", kernel="tc_gemm_kernel<LSE> (inside trl_token_logprobs)", achieved=achieved,
                    peak=peak, unit="TFLOP/s", frac=achieved / peak,
                    traffic=LSE_TRAFFIC_BYTES if (args.workload == WORKLOAD_ID and not args.small_case) else None,
                    peak_source=f"{peaks['source']} sustained cuBLAS bf16",
                    # the same comparison with the power cap's effect on the clock divided out: TFLOP/s per
                    # GHz of SM clock here (median sampled during the timed region) and for the peak (the
                    # clock its own measurement ran at)
                    achieved_per_ghz=per_ghz(achieved, sm_mhz),
                    peak_per_ghz=per_ghz(peak, peaks.get("sm_mhz_at_peak")),
                    peak_sm_mhz=peaks.get("sm_mhz_at_peak"))
    if roofline["achieved_per_ghz"] and roofline["peak_per_ghz"]:
        roofline["frac_per_clock"] = roofline["achieved_per_ghz"] / roofline["peak_per_ghz"]
    if args.path == "fused":     # policy forward + two gradient GEMMs = the metric's 6HV per token
        rest_alg = 6.0 * H * V * n_valid / (call_ms["pg_step_fused"] * 1e-3) / 1e12
        exec_flops = {"token_logprobs_old": 2.0, "pg_step_fused": 6.0}
    else:
        rest_alg = 4.0 * H * V * n_valid / (call_ms["pg_loss_bwd"] * 1e-3) / 1e12
        exec_flops = {"token_logprobs_policy": 2.0, "token_logprobs_old": 2.0, "pg_loss_bwd": 6.0}
    calls_tflops = {}
    for name, mult in exec_flops.items():      # executed GEMM FLOPs of each call (the recompute counts in four_call)
        tf = mult * H * V * n_valid / (call_ms[name] * 1e-3) / 1e12
        calls_tflops[name] = dict(tflops=tf, tflops_per_ghz=per_ghz(tf, sm_mhz))
    step_alg = 6.0 * H * V * value / world / 1e12

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v_cpu, tok, sec, threads = oracle_sample_throughput(w, 12, 64)
        cpu_baseline = dict(value=v_cpu, unit=UNIT, cores=threads, kind="oracle",
                            sample=f"12 rollouts x T=64 ({tok} valid tokens, {sec:.1f} s), full H={H} V={V}, whole path in numpy fp64")

    # ---- short side runs, so that the other configuration and the other schedule have a record
    # from the same process and GPU (3 timed steps each; not part of the headline)
    other_runs = None
    if rank == 0 and world == 1 and not args.no_other_runs and args.workload == WORKLOAD_ID and not args.small_case:
        del runner, bufs, step
        torch.cuda.empty_cache()
        other_runs = [side_run(trl, torch, synth, dev, 3, "fused", peaks, barrier),
                      side_run(trl, torch, synth, dev, WORKLOAD_ID, "four_call", peaks, barrier)]

    if rank == 0:
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=warm,
                    ms_per_step=elapsed_ms / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype=w.dtype, data="synthetic",
                    config=dict(workload=w.name, P=P, G=G, T=T, H=H, V=V, valid_tokens_per_rank=n_valid,
                                padded_rows_per_rank=B * T, l2="inputs larger than L2 (W alone is 1.2 GB); no flush",
                                parallelism=(f"data-parallel x{world}, dW all-reduced band by band behind the dW GEMM, loss all-reduced" if args.dp_allreduce
                                             else f"replicas x{world} (independent batches)")),
                    pct_of_bf16_peak_6NHV=dict(nominal=100 * step_alg / 2250.0,
                                               measured_sustained=100 * step_alg / peaks["bf16_sustained"],
                                               measured_burst=100 * step_alg / peaks["bf16_burst"],
                                               tflops=step_alg, tflops_per_ghz=per_ghz(step_alg, sm_mhz),
                                               note="6*H*V FLOP per scored token over the whole step (which also scores the old "
                                                    "policy: 8*H*V executed); nominal = 2250 TFLOP/s dense bf16, the measured "
                                                    "figures are cuBLAS on this pool's B200s under the same 1 kW cap"),
                    roofline=roofline,
                    calls_ms=call_ms,
                    calls_tflops=calls_tflops,
                    path=args.path,
                    algorithmic_tflops_of_last_call=rest_alg,
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             steps=e2e_steps),
                    gpu_launches=int(launches),
                    clocks=clocks,
                    cpu_baseline=cpu_baseline,
                    other_runs=other_runs,
                    loss=float(host_out[0]))
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
