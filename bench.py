#!/usr/bin/env python
"""Benchmark of the SureLock locked-forward step on B200.

One "step" = one pass of the whole hot path (compaction, embedding gather, L transformer blocks on the active
rows with K/V scatter and M x N attention, LM head, fused softmax-KL-lock) over one batch of synthetic
LLaDA-8B-shaped input.  Prints ONE JSON line (rank 0).  `value` is active tokens/s = packed active rows M
processed per second, inputs resident in HBM; `e2e` is the same through the host-buffer entry point with the
host<->device copies inside the timed region.  `sweep` repeats the measurement over M/N.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4|c3|c5|tiny] [--ratio 0.5]
                    [--ratios 1,0.5,0.25,0.125,0.05] [--impl ours|reference]

With --impl reference the CPU oracle is timed on the host cores on a bounded sample of the same workload.
For N > 1 (torchrun) every rank runs an independent replica of the workload (the path shards by sequence with
no exchange step): weak scaling, no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_06412_b200 import dist_util, inputs  # noqa: E402

WORKLOADS = {
    # name: (model shape, batch, N, prompt length, lock pattern)
    "c2": ("llada8b-layer", 1, 1024, 0, "random"),      # single-layer microbench: see run_single_layer()
    "c3": ("llada8b", 1, 512, 256, "random"),
    "c4": ("llada8b", 8, 1536, 512, "random"),
    "c5": ("llada8b", 4, 4096, 3584, "contiguous_plus_random"),
    "tiny": ("tiny", 1, 128, 64, "random"),
}
FALLBACK_PEAKS = dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0)


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def n_active_per_seq(B, N, ratio, seed):
    """Ragged per-sequence active counts around ratio*N (+-30 %, seeded); all N when ratio == 1."""
    if ratio >= 1.0:
        return [N] * B
    g = torch.Generator().manual_seed(seed)
    u = torch.rand(B, generator=g) * 2 - 1
    return [int(min(N, max(1, round(N * ratio * (1 + 0.3 * float(x)))))) for x in u]


def gemm_flops_per_row(cfg):
    d, F, V, L = cfg["d_model"], cfg["d_ff"], cfg["vocab"], cfg["n_layers"]
    hd = cfg["n_heads"] * cfg["head_dim"]
    return L * (2 * d * 3 * hd + 2 * hd * d + 2 * d * 2 * F + 2 * F * d) + 2 * d * V


def weight_bytes(cfg, esz=2):
    d, F, V, L = cfg["d_model"], cfg["d_ff"], cfg["vocab"], cfg["n_layers"]
    hd = cfg["n_heads"] * cfg["head_dim"]
    return esz * (L * (3 * hd * d + hd * d + 3 * d * F) + d * V)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.th.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], 0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = max(mx, float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=mx or None, reasons=sorted(reasons),
                    samples=len(sm))


# ----------------------------------------------------------------------------------------------------- CPU oracle leg
def oracle_sample(cfg, B, N, rows=512, head_rows=128, repeat=3):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: ONE of the L blocks on `rows`
    active rows of one sequence against an N-row cache, plus final norm + LM head + softmax/KL/lock test on
    `head_rows` rows; the block time is scaled by L.  Returns (tokens_per_s, seconds, threads, description)."""
    from oracle import surelock_oracle as O
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    oc = O.ModelCfg(**cfg)
    lw = {k: v.float().numpy() for k, v in inputs.make_layer_weights(cfg, 0, 1).items()}
    g = np.random.default_rng(0)
    d, H, dh, V = cfg["d_model"], cfg["n_heads"], cfg["head_dim"], cfg["vocab"]
    rows = min(rows, N)
    x = g.standard_normal((rows, d))
    pos = np.sort(g.choice(N, size=rows, replace=False))
    Kc, Vc = g.standard_normal((N, H, dh)), g.standard_normal((N, H, dh))
    t0 = time.perf_counter()
    for _ in range(repeat):
        O.layer_rows(oc, lw, x, pos, Kc, Vc)
    t_layer = (time.perf_counter() - t0) / repeat
    head = inputs._normal((V, d), 0.02, 3, torch.bfloat16, "cpu").float().numpy()
    xh = g.standard_normal((head_rows, d))
    zprev = g.standard_normal((head_rows, V)) * 3
    t0 = time.perf_counter()
    z = O.rmsnorm(xh, np.ones(d), cfg["rms_eps"]) @ np.asarray(head, np.float64).T
    O.posterior_stats(z)
    O.sure_test(O.kl_from_logits(z, zprev), np.zeros(head_rows), 1e-3)
    t_head = time.perf_counter() - t0
    per_row = cfg["n_layers"] * t_layer / rows + t_head / head_rows
    desc = (f"1 of {cfg['n_layers']} blocks on {rows} active rows of one N={N} sequence (x{cfg['n_layers']}) + LM head/"
            f"softmax-KL on {head_rows} rows; extrapolated per row")
    return 1.0 / per_row, repeat * t_layer + t_head, threads, desc


def workload_config(args, cfgname, cfg, B, N, pattern, M=None):
    """The `config` object, shared by both arms so that they describe the same workload."""
    return {"workload": f"{args.workload}: full {cfgname} stack ({cfg['n_layers']} layers, d={cfg['d_model']}, "
                        f"vocab={cfg['vocab']}), batch {B}, N={N}, M/N={args.ratio} ragged per sequence, "
                        f"{pattern} lock pattern", "batch": B, "seq_len": N, "active_rows": M,
            "l2": "inputs larger than L2 (every step streams all weights, %.1f GB)" % (weight_bytes(cfg) / 1e9),
            "multi_gpu": "replicas only (one independent batch per rank, no collective)"}


def c2_config(M0, N, wbytes):
    return {"workload": "c2: ONE LLaDA-8B-shaped layer (d=4096, 32 heads x 128, FFN 12288), batch 1, N=1024, "
                        f"M={M0} active rows (seeded random subset), through surelock_layer_step", "batch": 1,
            "seq_len": N, "active_rows": M0,
            "l2": "inputs larger than L2 (every call streams the layer's weights, %.0f MB)" % (wbytes / 1e6),
            "multi_gpu": "replicas only (one independent layer per rank, no collective)"}


def headline_rows(args, B, N):
    """M of the headline measurement: the ragged per-sequence active counts of replica 0 (the same seeded draw the
    GPU arm makes), so that both arms name the same workload."""
    seed = dist_util.replica_seed(1234, 0)
    return sum(n_active_per_seq(B, N, args.ratio, seed * 31 + int(args.ratio * 1000)))


def run_reference(args, cfgname, B, N, pattern):
    if args.workload == "c2":                                         # the single-layer microbench: the oracle's layer alone
        from oracle import surelock_oracle as O
        cfg = inputs.model_shape("llada8b", n_layers=1, vocab=0)
        oc = O.ModelCfg(**cfg)
        lw = {k: v.float().numpy() for k, v in inputs.make_layer_weights(cfg, 0, 1).items()}
        g = np.random.default_rng(0)
        rows, vals, secs = 128, [], 0.0
        Kc, Vc = (g.standard_normal((N, cfg["n_heads"], cfg["head_dim"])) for _ in range(2))
        for i in range(max(0, args.warmup) + max(1, args.steps)):
            x, pos = g.standard_normal((rows, cfg["d_model"])), np.sort(g.choice(N, size=rows, replace=False))
            t0 = time.perf_counter()
            O.layer_rows(oc, lw, x, pos, Kc, Vc)
            if i >= max(0, args.warmup):
                vals.append(rows / (time.perf_counter() - t0)); secs += time.perf_counter() - t0
        try:
            from threadpoolctl import threadpool_info
            threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        v = float(np.median(vals))
        desc = f"the layer on {rows} active rows against the N={N} cache per step"
        return {"impl": "reference", "metric": "active_tokens_per_s", "value": v, "unit": "tokens/s", "n_gpus": args.gpus,
                "steps": len(vals), "warmup": max(0, args.warmup), "ms_per_step": 1e3 * secs / len(vals),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": c2_config(512, N, 2 * (4 * cfg["n_heads"] * cfg["head_dim"] * cfg["d_model"]
                                                     + 3 * cfg["d_model"] * cfg["d_ff"])),
                "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
                "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    cfg = inputs.model_shape(cfgname)
    vals, secs = [], 0.0
    for _ in range(max(0, args.warmup)):                              # untimed, like the GPU arm's warm-up steps
        oracle_sample(cfg, B, N, rows=32, head_rows=8, repeat=1)
    for _ in range(max(1, args.steps)):                               # each step: a bounded sample of the workload
        v, s, threads, desc = oracle_sample(cfg, B, N, rows=128, head_rows=32, repeat=1)
        vals.append(v); secs += s
    v = float(np.median(vals))
    return {"impl": "reference", "metric": "active_tokens_per_s", "value": v, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": len(vals), "warmup": max(0, args.warmup), "ms_per_step": 1e3 * secs / len(vals), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args, cfgname, cfg, B, N, pattern, headline_rows(args, B, N)),
            "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


# ----------------------------------------------------------------------------------------------------- single layer
def run_single_layer(args, rank, world, local):
    """Single LLaDA-8B-shaped layer (RMSNorm, QKV + RoPE + cache scatter, M x N attention, O, SwiGLU FFN; no embedding,
    LM head or KL), batch 1, N = 1024, cache pre-filled by one full pass, seeded random active subsets of
    M in {1024, 512, 256, 128, 32} rows, through surelock_layer_step.  One "step" is one call."""
    from paper_2602_06412_b200 import binding as SL
    SL.lib()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    args.warmup = max(args.warmup, 3)
    cfg = inputs.model_shape("llada8b", n_layers=1, vocab=0)
    N, d, F = 1024, cfg["d_model"], cfg["d_ff"]
    seed = dist_util.replica_seed(1234, rank)
    w = dict(layers=[{k: v.to(dev) for k, v in inputs.make_layer_weights(cfg, 0, seed, dtype=torch.bfloat16).items()}])
    ctx = SL.surelock_init(cfg, w, N, 1)
    H0, H1 = inputs.hidden_states(N, d, 1).to(dev), inputs.hidden_states(N, d, 2).to(dev)
    out = torch.zeros((N, d), dtype=torch.float32, device=dev)
    SL.surelock_layer_step(ctx, 0, H0, torch.zeros((1, N), dtype=torch.uint8, device=dev), out)   # pre-fill of the cache
    torch.cuda.synchronize()
    pk, pk_kind = peaks()
    hd = cfg["n_heads"] * cfg["head_dim"]
    wbytes = 2 * (4 * hd * d + 3 * d * F)
    flops_row = 2 * d * 3 * hd + 2 * hd * d + 6 * d * F

    def timed(M, steps, warmup):
        lock = inputs.random_lock(1, N, [M], 100 + M).to(dev) if M < N else torch.zeros((1, N), dtype=torch.uint8, device=dev)
        for _ in range(warmup):
            SL.surelock_layer_step(ctx, 0, H1, lock, out)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            o = SL.surelock_layer_step(ctx, 0, H1, lock, out)
        e1.record()
        torch.cuda.synchronize()
        assert o.M() == M
        return dist_util.max_over_ranks(e0.elapsed_time(e1) / steps, dev), lock

    steps = max(args.steps, 20)
    M0 = 512
    sampler = ClockSampler(local)
    with sampler:
        ms, lock0 = timed(M0, 50 * steps, args.warmup)
    clocks = sampler.summary()
    launches = 50 * steps * SL.surelock_last_launch_count(ctx)
    SL.surelock_set_option(ctx, "time_kernels", 1)
    SL.surelock_layer_step(ctx, 0, H1, lock0, out)
    kt = SL.surelock_kernel_times(ctx)
    SL.surelock_set_option(ctx, "time_kernels", 0)
    total_k = sum(v[0] for v in kt.values())
    kernels = {k: dict(ms=round(v[0], 4), launches=v[1], share=round(v[0] / total_k, 4)) for k, v in kt.items()}
    gemm_ms = sum(v[0] for k, v in kt.items() if k.startswith("gemm"))
    gemm_n = sum(v[1] for k, v in kt.items() if k.startswith("gemm"))
    ach = M0 * flops_row / (gemm_ms * 1e-3) / 1e12
    roof = dict(kernel="gemm_tc (the four GEMM launches of the layer)", bound="tensor", achieved=ach,
                peak=pk["bf16_tflops"], unit="TFLOP/s", frac=ach / pk["bf16_tflops"],
                traffic=0.89 * (wbytes + M0 * (2 * d + 6 * hd + 2 * hd + 8 * d + 2 * d + 4 * F + 8 * d)) / max(gemm_n, 1),
                traffic_note="bytes per average launch, scaled from a small-case ncu capture",
                peak_kind=f"{pk_kind}, burst (kernels timed one by one)", launches_per_step=gemm_n,
                avg_launch_ms=gemm_ms / max(gemm_n, 1))
    # end to end: the hidden states come from pinned host memory and the packed output rows go back, every call
    hin = inputs.hidden_states(N, d, 2).pin_memory()
    hout = torch.zeros((N, d), dtype=torch.float32).pin_memory()
    hdev = torch.empty_like(H1)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        hdev.copy_(hin, non_blocking=True)
        SL.surelock_layer_step(ctx, 0, hdev, lock0, out)
        hout[:M0].copy_(out[:M0], non_blocking=True)
        torch.cuda.synchronize()
    e2e_ms = dist_util.max_over_ranks((time.perf_counter() - t0) * 1e3 / steps, dev)
    sweep = []
    for M in (1024, 512, 256, 128, 32):
        t, _ = timed(M, 20 * steps, 3)
        ideal = max(M * flops_row / (pk["bf16_tflops_sustained"] * 1e12) + 4.0 * M * N * hd / (pk["bf16_tflops_sustained"] * 1e12),
                    wbytes / (pk["hbm_gbs"] * 1e9)) * 1e3
        sweep.append(dict(M=M, ms_per_step=round(t, 5), tokens_per_s=round(dist_util.sum_over_ranks(M, dev) / (t * 1e-3), 1),
                          ideal_ms=round(ideal, 5), frac_of_ideal=round(ideal / t, 4)))
    line = {
        "metric": "active_tokens_per_s", "value": dist_util.sum_over_ranks(M0, dev) / (ms * 1e-3), "unit": "tokens/s",
        "n_gpus": world, "steps": 50 * steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": c2_config(M0, N, wbytes),
        "e2e": dict(value=dist_util.sum_over_ranks(M0, dev) / (e2e_ms * 1e-3), unit="tokens/s", ms_per_step=e2e_ms,
                    h2d_bytes_per_step=N * d * 2, d2h_bytes_per_step=M0 * d * 4),
        "gpu_launches": launches, "clocks": clocks, "roofline": roof, "kernels": kernels, "sweep": sweep,
        "device_status": SL.surelock_status_poll(ctx),
    }
    if rank == 0 and not args.no_cpu_baseline:
        from oracle import surelock_oracle as O
        oc = O.ModelCfg(**cfg)
        lw = {k: v.float().cpu().numpy() for k, v in w["layers"][0].items()}
        g = np.random.default_rng(0)
        rows = 256
        pos = np.sort(g.choice(N, size=rows, replace=False))
        Kc, Vc = g.standard_normal((N, cfg["n_heads"], cfg["head_dim"])), g.standard_normal((N, cfg["n_heads"], cfg["head_dim"]))
        x = g.standard_normal((rows, d))
        t0 = time.perf_counter()
        for _ in range(3):
            O.layer_rows(oc, lw, x, pos, Kc, Vc)
        secs = time.perf_counter() - t0
        try:
            from threadpoolctl import threadpool_info
            threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            threads = os.cpu_count() or 1
        line["cpu_baseline"] = {"value": 3 * rows / secs, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                                "sample": f"the layer on {rows} active rows against the N={N} cache, 3 times",
                                "seconds": round(secs, 2)}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


# ----------------------------------------------------------------------------------------------------- GPU leg
def spawn_ranks(n):
    """`python bench.py --gpus N` outside a launcher: start the N ranks here, one process per GPU, the way a launcher
    would (`python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 ...` with the same
    arguments).  Rank r binds GPU r; rank 0 prints the JSON line, which passes through unchanged.  NCCL's log is
    switched on and sent to stderr, so the communicator lines show the N ranks without touching stdout."""
    import socket
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    env.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd, env=env).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4", choices=sorted(WORKLOADS))
    ap.add_argument("--ratio", type=float, default=0.5, help="active fraction M/N of the headline measurement")
    ap.add_argument("--ratios", default="1,0.5,0.25,0.125,0.05", help="M/N sweep ('' = none)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sampler-steps", type=int, default=32,
                    help="diffusion steps of the decoding run (SureLock vs the no-locking baseline sampler); 0 = skip")
    args = ap.parse_args()
    if args.gpus > 1 and "RANK" not in os.environ:
        return spawn_ranks(args.gpus)
    rank, world, local = dist_util.env_rank_world()
    cfgname, B, N, n_prompt, pattern = WORKLOADS[args.workload]

    if args.impl == "reference":                   # the CPU oracle: rank 0 alone works, the others leave at once
        if rank == 0:
            args.gpus = max(args.gpus, world)
            print(json.dumps(run_reference(args, cfgname, B, N, pattern)), flush=True)
        return 0
    if world > 1 and torch.cuda.is_available() and local >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} wants GPU {local}, but only {torch.cuda.device_count()} GPU(s) are "
                         "visible: --gpus N needs N GPUs on this node (one replica per GPU)")

    if args.workload == "c2":
        return run_single_layer(args, rank, world, local)

    from paper_2602_06412_b200 import binding as SL
    SL.lib()                                       # fail loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    args.warmup = max(args.warmup, 3)
    cfg = inputs.model_shape(cfgname)
    dtype = torch.bfloat16 if cfgname != "tiny" else torch.float32
    seed = dist_util.replica_seed(1234, rank)
    w = inputs.make_weights(cfg, seed, dtype=dtype, device=dev)
    ctx = SL.surelock_init(cfg, w, N, B)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], seed)
    tokens_d, mask_d = tokens.to(dev), mask.to(dev)
    R = B * N
    lock_d = torch.zeros((B, N), dtype=torch.uint8, device=dev)

    def lock_pattern(ratio):
        na = n_active_per_seq(B, N, ratio, seed * 31 + int(ratio * 1000))
        f = inputs.contiguous_plus_random_lock if pattern == "contiguous_plus_random" else inputs.random_lock
        return f(B, N, na, seed), sum(na)

    # pre-fill: one full step (nothing locked) writes every cache row and the first "previous" logits
    SL.surelock_step(ctx, tokens_d, mask_d, lock_d, 1e-3)
    torch.cuda.synchronize()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    def timed(ratio, steps, warmup, sampler=None):
        lock0, M = lock_pattern(ratio)
        lock0 = lock0.to(dev)
        for _ in range(warmup):
            lock_d.copy_(lock0)
            out = SL.surelock_step(ctx, tokens_d, mask_d, lock_d, 1e-3)
        barrier()
        assert out.M() == M, (out.M(), M)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches = 0
        if sampler:
            sampler.__enter__()
        e0.record()
        for _ in range(steps):
            lock_d.copy_(lock0)                    # the sure test locks converged rows; restore so M stays fixed
            SL.surelock_step(ctx, tokens_d, mask_d, lock_d, 1e-3)
            launches += SL.surelock_last_launch_count(ctx)
        e1.record()
        barrier()
        if sampler:
            sampler.__exit__()
        ms = dist_util.max_over_ranks(e0.elapsed_time(e1) / steps, dev)
        return M, ms, launches, lock0

    pk, pk_kind = peaks()
    sampler = ClockSampler(local)
    M, ms, launches, lock0 = timed(args.ratio, args.steps, args.warmup, sampler)
    clocks = sampler.summary()
    value = dist_util.sum_over_ranks(M, dev) / (ms * 1e-3)    # all replicas' rows / slowest replica's time

    # per-kernel-class breakdown of the same step (separate pass: events around every launch)
    SL.surelock_set_option(ctx, "time_kernels", 1)
    acc = {}
    for _ in range(2):
        lock_d.copy_(lock0)
        SL.surelock_step(ctx, tokens_d, mask_d, lock_d, 1e-3)
        for k, (t, n) in SL.surelock_kernel_times(ctx).items():
            a = acc.setdefault(k, [0.0, 0])
            a[0] += t / 2; a[1] = n
    SL.surelock_set_option(ctx, "time_kernels", 0)
    gemm_ms = sum(acc[k][0] for k in acc if k.startswith("gemm"))
    gemm_launch = sum(acc[k][1] for k in acc if k.startswith("gemm"))
    flops = M * gemm_flops_per_row(cfg)
    wbytes = weight_bytes(cfg)
    # DRAM traffic per average GEMM launch: measured / algorithmic bytes of each of the step's five GEMM shapes from
    # one-launch ncu captures at this workload's own row count (M = 6587; profiles/gemm_tc_kernel_M6587_dram_traffic.md),
    # applied to the algorithmic bytes of the shapes at the M of this run
    d_, F_, V_, L_ = cfg["d_model"], cfg["d_ff"], cfg["vocab"], cfg["n_layers"]
    hd_ = cfg["n_heads"] * cfg["head_dim"]
    alg = {"qkv": 2 * M * d_ + 2 * 3 * hd_ * d_ + 2 * 3 * M * hd_, "o": 2 * M * hd_ + 2 * hd_ * d_ + 8 * M * d_,
           "gateup": 2 * M * d_ + 2 * 2 * d_ * F_ + 2 * M * F_, "down": 2 * M * F_ + 2 * F_ * d_ + 8 * M * d_,
           "head": 2 * M * d_ + 2 * d_ * V_ + 2 * M * V_}
    measured_over_alg = {"qkv": 1.54, "o": 1.19, "gateup": 2.10, "down": 2.30, "head": 2.53}
    traffic = (L_ * sum(alg[k] * measured_over_alg[k] for k in ("qkv", "o", "gateup", "down")) +
               alg["head"] * measured_over_alg["head"]) / max(gemm_launch, 1)
    traffic_alg = (L_ * sum(alg[k] for k in ("qkv", "o", "gateup", "down")) + alg["head"]) / max(gemm_launch, 1)
    ridge = pk["bf16_tflops_sustained"] * 1e12 / (pk["hbm_gbs"] * 1e9)
    if M >= ridge:
        ach = flops / (gemm_ms * 1e-3) / 1e12
        roof = dict(kernel="gemm_tc (all GEMM launches of the step)", bound="tensor", achieved=ach,
                    peak=pk["bf16_tflops_sustained"], unit="TFLOP/s", frac=ach / pk["bf16_tflops_sustained"],
                    traffic=traffic, traffic_algorithmic=traffic_alg,
                    traffic_note="DRAM bytes per average GEMM launch: per-shape measured/algorithmic ratios of one-launch ncu captures at M = 6587, applied to this run's algorithmic bytes",
                    peak_kind=f"{pk_kind}, sustained", launches_per_step=gemm_launch,
                    avg_launch_ms=gemm_ms / max(gemm_launch, 1))
    else:
        ach = wbytes / (gemm_ms * 1e-3) / 1e9
        chained = bool(SL.surelock_last_step_paths(ctx) & 1)        # few rows: the layer chain kernel ran the layers
        name = ("gemm_chain (one launch per layer: O, gate/up, down, next Q/K/V) + gemm_tc (LM head), weight streaming"
                if chained else "gemm_tc (all GEMM launches of the step, weight streaming)")
        roof = dict(kernel=name, bound="hbm", achieved=ach,
                    peak=pk["hbm_gbs"], unit="GB/s", frac=ach / pk["hbm_gbs"], traffic=traffic_alg,
                    traffic_algorithmic=traffic_alg,
                    traffic_note="weight-streaming regime: the weights are read once (ncu at M = 32: 102.0 MB read for a 100.7 MB matrix; 341 MB for the 335.5 MB of a chain launch), so algorithmic bytes per average launch", peak_kind=pk_kind,
                    launches_per_step=gemm_launch, avg_launch_ms=gemm_ms / max(gemm_launch, 1))
    total_k = sum(v[0] for v in acc.values())
    kernels = {k: dict(ms=round(v[0], 4), launches=v[1], share=round(v[0] / total_k, 4)) for k, v in acc.items()}

    # end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    tk, mk = tokens.pin_memory(), mask.pin_memory()
    lk0 = lock0.cpu()
    lk = lk0.clone().pin_memory()
    n_h = torch.zeros(1, dtype=torch.int32).pin_memory()
    ai = torch.zeros(R, dtype=torch.int32).pin_memory()
    klh, cfh = torch.zeros(R).pin_memory(), torch.zeros(R).pin_memory()
    amh = torch.zeros(R, dtype=torch.int32).pin_memory()
    for _ in range(2):
        lk.copy_(lk0)
        SL.surelock_step_host(ctx, tk, mk, lk, 1e-3, n_h, ai, klh, cfh, amh)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        lk.copy_(lk0)
        SL.surelock_step_host(ctx, tk, mk, lk, 1e-3, n_h, ai, klh, cfh, amh)
    torch.cuda.synchronize()
    e2e_ms = dist_util.max_over_ranks((time.perf_counter() - t0) * 1e3 / args.steps, dev)
    e2e = dict(value=dist_util.sum_over_ranks(int(n_h.item()), dev) / (e2e_ms * 1e-3), unit="tokens/s", ms_per_step=e2e_ms,
               h2d_bytes_per_step=R * 4 + R + R, d2h_bytes_per_step=R + 4 + 4 * R * 4)

    sweep = []
    if args.ratios:
        for r in [float(x) for x in args.ratios.split(",") if x]:
            Ms, mss, _, _ = timed(r, max(2, args.steps // 2), 3)
            ideal_ms = max(Ms * gemm_flops_per_row(cfg) / (pk["bf16_tflops_sustained"] * 1e12),
                           wbytes / (pk["hbm_gbs"] * 1e9)) * 1e3
            sweep.append(dict(ratio=r, M=Ms, ms_per_step=round(mss, 4),
                              tokens_per_s=round(dist_util.sum_over_ranks(Ms, dev) / (mss * 1e-3), 1),
                              gemm_ideal_ms=round(ideal_ms, 4), frac_of_gemm_ideal=round(ideal_ms / mss, 4)))

    # the paper's own run metrics on a short decoding run: the sampler loop with and without SureLock
    sampler_run = None
    if args.sampler_steps > 0 and rank == 0:
        from paper_2602_06412_b200 import sampler
        block_len = {"c3": 32, "c4": 64, "c5": 64, "tiny": 64}[args.workload]
        runs = {}
        tk, mk = tokens.to(dev), mask.to(dev)
        sampler.run(ctx, tk, mk, n_prompt, block_len, 2, 1e-3)               # untimed: first-use costs of the loop's torch ops
        for mode in ("surelock", "baseline", "selection", "hybrid"):
            tk, mk = tokens.to(dev), mask.to(dev)
            r = sampler.run(ctx, tk, mk, n_prompt, block_len, args.sampler_steps, 1e-3,
                            surelock=mode in ("surelock", "hybrid"),
                            select_fraction=0.8 if mode in ("selection", "hybrid") else None)
            runs[mode] = r
        base_tps = max(runs["baseline"]["e2e_tps"], 1e-9)
        sampler_run = dict(
            steps=args.sampler_steps, block_len=block_len, kl_eps=1e-3, confidence_gate="off",
            r_bar=round(runs["surelock"]["r_bar"], 4), flops_ratio=round(runs["surelock"]["flops_ratio"], 4),
            f_base_per_position=runs["baseline"]["f_base_per_position"],
            f_prop_per_position=runs["surelock"]["f_prop_per_position"],
            e2e_tps_surelock=round(runs["surelock"]["e2e_tps"], 2), e2e_tps_baseline=round(runs["baseline"]["e2e_tps"], 2),
            tps_ratio=round(runs["surelock"]["e2e_tps"] / base_tps, 3),
            # Experiment 5: selection surrogate (0.8 of the positions) alone and combined with SureLock
            selection=dict(fraction=0.8, tps_ratio=round(runs["selection"]["e2e_tps"] / base_tps, 3),
                           flops_ratio=round(runs["selection"]["r_bar"], 4)),
            hybrid=dict(fraction=0.8, tps_ratio=round(runs["hybrid"]["e2e_tps"] / base_tps, 3),
                        flops_ratio=round(runs["hybrid"]["r_bar"], 4)),
            M_trace=runs["surelock"]["M_trace"],
            ms_per_step_surelock=[round(x, 3) for x in runs["surelock"]["ms_per_step"]],
            ms_per_step_baseline_median=round(float(np.median(runs["baseline"]["ms_per_step"])), 3),
            note="random-init weights: the lock trajectory is synthetic (posteriors barely move, so unmasked rows lock "
                 "at their second step); the paper reports 0.54x FLOPs and 1.30x TPS for SureLock, 0.64x / 1.18x for "
                 "selection at 0.8 and 0.28x / 1.73x for the combination (LLaDA-8B-Instruct on its GPU)")
        SL.surelock_reset(ctx)

    status = SL.surelock_status_poll(ctx)
    line = {
        "metric": "active_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if dtype == torch.bfloat16 else "f32", "data": "synthetic",
        "config": workload_config(args, cfgname, cfg, B, N, pattern, M),
        "e2e": e2e, "gpu_launches": launches, "clocks": clocks, "roofline": roof, "kernels": kernels, "sweep": sweep,
        "sampler_run": sampler_run,
        "device_status": status,
    }
    if rank == 0 and not args.no_cpu_baseline:
        v, secs, threads, desc = oracle_sample(cfg, B, N)
        line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc,
                                "seconds": round(secs, 2)}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
