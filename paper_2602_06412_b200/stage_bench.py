"""Time ONE stage of the SureLock step alone, through the C ABI, against its roofline.

    python -m paper_2602_06412_b200.stage_bench --stage gemm --M 4096 --n_out 12288 --K 4096
    python -m paper_2602_06412_b200.stage_bench --stage attention --B 8 --N 1536 --ratio 0.5
    python -m paper_2602_06412_b200.stage_bench --stage softmax_kl --rows 820
    python -m paper_2602_06412_b200.stage_bench --stage kv_scatter --rows 6144
    python -m paper_2602_06412_b200.stage_bench --stage compact --flags 67108864

Prints one JSON line: median and minimum device time (CUDA events on the launching stream, after warm-up), the
algorithmic bytes / FLOPs of the launch, and the achieved fraction of the measured HBM or bf16 peak.  A buffer
larger than L2 is written between iterations unless --warm-l2 is given.  Small, self-contained cases of this
module are also what the ncu captures under profiles/ run.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

from . import binding as SL
from . import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return d["hbm_gbs"], d["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def _time(fn, iters, warmup, flush):
    scratch = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if flush else None
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        if scratch is not None:
            scratch.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    ts.sort()
    return ts[len(ts) // 2], ts[0]


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--stage", required=True, choices=["gemm", "attention", "softmax_kl", "kv_scatter", "compact"])
    ap.add_argument("--M", type=int, default=4096)
    ap.add_argument("--n_out", type=int, default=12288)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--impl", type=int, default=0)
    ap.add_argument("--epilogue", type=int, default=0, help="gemm: 0 store, 1 += into the fp32 residual stream, 2 SwiGLU")
    ap.add_argument("--B", type=int, default=8)
    ap.add_argument("--N", type=int, default=1536)
    ap.add_argument("--H", type=int, default=32)
    ap.add_argument("--dh", type=int, default=128)
    ap.add_argument("--ratio", type=float, default=0.5)
    ap.add_argument("--rows", type=int, default=820)
    ap.add_argument("--V", type=int, default=126464)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--flags", type=int, default=1 << 26)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--warm-l2", action="store_true")
    a = ap.parse_args(argv)
    SL.lib()
    dev = "cuda"
    hbm, tf, kind = _peaks()
    g = torch.Generator(device=dev).manual_seed(1)
    rnd = lambda *s: torch.randn(s, device=dev, generator=g)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    res = dict(stage=a.stage, peak_kind=kind)

    if a.stage == "gemm":
        A = rnd(a.M, a.K).to(torch.bfloat16)
        W = (rnd(a.n_out, a.K) * 0.02).to(torch.bfloat16)
        Cout = torch.empty((a.M, a.n_out), dtype=torch.bfloat16, device=dev)
        n = torch.tensor([a.M], dtype=torch.int32, device=dev)
        wsp = torch.zeros(SL.surelock_gemm_workspace_bytes(), dtype=torch.uint8, device=dev)
        flops = 2.0 * a.M * a.n_out * a.K
        byts = 2.0 * (a.M * a.K + a.n_out * a.K + a.M * a.n_out)
        if a.epilogue == 1:                                   # fp32 stream read and written
            Cout = torch.zeros((a.M, a.n_out), dtype=torch.float32, device=dev)
            fn = lambda: SL.surelock_gemm_fused(A, W, None, Cout, n, 1, impl=a.impl, dev_status=status, workspace=wsp)
            byts = 2.0 * (a.M * a.K + a.n_out * a.K) + 8.0 * a.M * a.n_out
        elif a.epilogue == 2:                                 # gate and up matrices
            W2 = (rnd(a.n_out, a.K) * 0.02).to(torch.bfloat16)
            fn = lambda: SL.surelock_gemm_fused(A, W, W2, Cout, n, 2, impl=a.impl, dev_status=status, workspace=wsp)
            flops, byts = 2 * flops, byts + 2.0 * a.n_out * a.K
        else:
            fn = lambda: SL.surelock_gemm(A, W, Cout, n, impl=a.impl, dev_status=status, workspace=wsp)
        res.update(shape=[a.M, a.n_out, a.K], epilogue=a.epilogue, flops=flops, bytes=byts)
    elif a.stage == "attention":
        B, N, H, dh = a.B, a.N, a.H, a.dh
        na = [max(1, int(N * a.ratio))] * B
        lock = inputs.random_lock(B, N, na, 3).to(dev)
        M = sum(na)
        idx = torch.nonzero(lock.reshape(-1) == 0).flatten().to(torch.int32)
        offs = torch.tensor([0] + list(torch.tensor(na).cumsum(0)), dtype=torch.int32, device=dev)
        q = rnd(M, H, dh).to(torch.bfloat16)
        Kc = rnd(B * N, H, dh).to(torch.bfloat16)
        Vc = rnd(B * N, H, dh).to(torch.bfloat16)
        o = torch.empty_like(q)
        n = torch.tensor([M], dtype=torch.int32, device=dev)
        fn = lambda: SL.surelock_attention(q, Kc, Vc, idx, offs, n, B, N, o, impl=a.impl, dev_status=status)
        flops = 4.0 * M * N * H * dh
        byts = 2.0 * (2 * B * N * H * dh + 2 * M * H * dh)
        res.update(shape=dict(B=B, N=N, H=H, dh=dh, M=M), flops=flops, bytes=byts)
    elif a.stage == "softmax_kl":
        rows, V = a.rows, a.V
        cur, prev, mask = inputs.kl_logit_pairs(rows, V, 7, device=dev)
        kl = torch.empty(rows, device=dev)
        conf = torch.empty(rows, device=dev)
        am = torch.empty(rows, dtype=torch.int32, device=dev)
        lse = torch.empty(rows, device=dev)
        plse = torch.empty(rows, device=dev)
        lock = torch.zeros(rows, dtype=torch.uint8, device=dev)
        n = torch.tensor([rows], dtype=torch.int32, device=dev)
        ones = torch.ones(rows, dtype=torch.uint8, device=dev)
        SL.surelock_softmax_kl_sure(prev, None, None, None, None, n, ones, lock, 0.0, kl, conf, am, plse)   # lse of the previous rows
        fn = lambda: SL.surelock_softmax_kl_sure(cur, prev, None, plse, None, n, mask, lock, 1e-3, kl, conf, am, lse)
        byts = 2.0 * rows * V * 2
        res.update(shape=dict(rows=rows, V=V), bytes=byts, flops=0.0)
    elif a.stage == "kv_scatter":
        rows, d = a.rows, a.d
        cap = 2 * rows
        k, v = rnd(rows, d).to(torch.bfloat16), rnd(rows, d).to(torch.bfloat16)
        kc = torch.zeros((cap, d), dtype=torch.bfloat16, device=dev)
        vc = torch.zeros_like(kc)
        idx = torch.randperm(cap, device=dev, generator=g)[:rows].sort().values.to(torch.int32)
        n = torch.tensor([rows], dtype=torch.int32, device=dev)
        fn = lambda: SL.surelock_kv_scatter(k, v, idx, n, kc, vc)
        byts = 2.0 * 2 * rows * d * 2          # K and V, read + write
        res.update(shape=dict(rows=rows, d=d), bytes=byts, flops=0.0)
    else:
        total = a.flags
        lock = (torch.rand(total, device=dev, generator=g) < 0.5).to(torch.uint8)
        idx = torch.empty(total, dtype=torch.int32, device=dev)
        offs = torch.empty(2, dtype=torch.int32, device=dev)
        n = torch.empty(1, dtype=torch.int32, device=dev)
        rop = torch.empty(total, dtype=torch.int32, device=dev)
        scratch = torch.empty(SL.surelock_compact_scratch_bytes(total), dtype=torch.uint8, device=dev)
        fn = lambda: SL.surelock_compact(lock, 1, total, idx, offs, n, rop, scratch, status)
        fn()
        torch.cuda.synchronize()
        byts = total * 1.0 + 4.0 * int(n.item()) + 4.0 * total     # flags in, indices out, row_of_pos out
        res.update(shape=dict(flags=total, active=int(n.item())), bytes=byts, flops=0.0)

    med, best = _time(fn, a.iters, a.warmup, not a.warm_l2)
    assert status.item() == 0, "device status %d" % status.item()
    res.update(ms_median=med, ms_min=best, l2="warm" if a.warm_l2 else "flushed between iterations")
    gbs = res["bytes"] / (med * 1e-3) / 1e9
    res.update(gbs=gbs, frac_hbm=gbs / hbm, hbm_peak=hbm)
    if res["flops"]:
        t = res["flops"] / (med * 1e-3) / 1e12
        res.update(tflops=t, frac_tensor=t / tf, tensor_peak=tf)
    print(json.dumps(res), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
