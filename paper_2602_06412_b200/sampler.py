"""Decoding harness around the SureLock step: the sampler loop of Algorithm 1 with the unmasking policy on the device.

The library call `surelock_step` is Algorithm 1 lines 6-15 and 18-24, `surelock_update_mask` is line 16
(`UpdateMASK`); this module plays line 5 (the loop over diffusion steps): semi-autoregressive blocks, and in every step
each sequence reveals the `k` masked positions of its current block whose posterior is most confident, with their
argmax tokens (temperature 0, "low-confidence remasking": the rest stay masked).  Both calls are kernels of the
library working on device buffers, so the loop never waits for the GPU; per-step times are CUDA events read at the end.

It also computes what the paper reports from such a run: the per-step active-row trace M_t, the micro-averaged active
ratio r_bar, the algorithmic-FLOP ratio F_prop / F_base (Sec. 2.3), E2E-TPS and StepTPS (unmasked tokens per
wall-clock second, whole run and per step).  `surelock=False` is the paper's baseline: the same sampler recomputing all
positions every step (the lock mask is cleared after each step).
"""
from __future__ import annotations

from typing import Dict

import torch

from . import binding as SL
from . import inputs


def algorithmic_flops_per_step(cfg: Dict, B: int, N: int) -> int:
    """F^t_base of Sec. 2.3 (GEMMs only: QK^T + AV, Q, Out, K/V and FFN projections) for one full step of a batch."""
    L, d, H, dh, F = cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["head_dim"], cfg["d_ff"]
    return L * (4 * B * H * N * N * dh + 2 * B * N * d * d + 2 * B * N * d * d + 4 * B * N * d * H * dh + 6 * B * N * d * F)


def selection_skip_mask(lock: torch.Tensor, mask_state: torch.Tensor, fraction: float, step: int, seed: int):
    """Surrogate of a selection-based method (Experiment 5): compute only a fixed `fraction` of the positions that are
    not locked.  Which ones is the selection method's business; this surrogate ranks them by seeded scores
    (`inputs.selection_scores`), per sequence, and never skips a masked position (the sampler needs its posterior):
    of the eligible positions (unlocked and unmasked) the floor((1 - fraction) * unlocked) with the lowest scores are
    skipped, fewer when there are not that many.  Returns uint8 [B][N], 1 = skip this step.  This is harness code
    (torch operations on the lock mask, outside the library): the step itself is unchanged."""
    B, N = lock.shape
    score = inputs.selection_scores(B, N, step, seed, device=lock.device)
    eligible = (lock == 0) & (mask_state == 0)                       # may be skipped
    n_unlocked = (lock == 0).sum(dim=1, keepdim=True)
    n_skip = torch.minimum(torch.floor(n_unlocked * (1.0 - fraction)).long(), eligible.sum(dim=1, keepdim=True))
    score = torch.where(eligible, score, torch.full_like(score, 2.0))
    rank = score.argsort(dim=1).argsort(dim=1)                       # 0 = first to be skipped
    return ((rank < n_skip) & eligible).to(torch.uint8)


def run(ctx: SL.Ctx, tokens: torch.Tensor, mask_state: torch.Tensor, n_prompt: int, block_len: int, steps: int,
        kl_eps: float, surelock: bool = True, unmask_per_step: int = 1, select_fraction: float = None,
        select_seed: int = 0, observer=None, unlock: Dict = None) -> Dict:
    """Run `steps` diffusion steps on device tensors tokens int32 [B][N], mask_state uint8 [B][N] (both updated in
    place).  Generation positions n_prompt.. are decoded block by block (`block_len` positions, `steps_per_block` =
    ceil(block_len / unmask_per_step) steps each).  `select_fraction` (Experiment 5, e.g. 0.8) adds the selection
    surrogate: every step only that fraction of the not-yet-locked positions is computed; with `surelock` this is the
    paper's combination, without it the selection baseline.  A skipped row keeps its cached K/V; it has no posterior in
    that step, so it cannot lock in the step in which it returns (D needs the previous step's posterior).
    `unlock` (App. "Optional Unlocking"): a dict of the parameters of `surelock_set_unlocking` (period, eps_unlock,
    d_interval, d_cool, rho, m_percent) switches un-locking on for this run: after every step's unmasking the probe is
    called (it works every `period`-th step) and may return locked positions to the active set; the number of un-locked
    positions per step is in the result.
    `observer`, when given, is called after every step, before the unmasking of line 16, as
    observer(t, out, lock_in, lock_out, tokens, mask_state) with lock_in a copy of the lock mask the step was given
    (skip mask included) and lock_out the mask after the step; it is for tests that look at a step from outside and
    makes the loop wait for the GPU.
    Returns the trace and the paper's metrics."""
    B, N = tokens.shape
    dev = tokens.device
    R = B * N
    mask_token = ctx.cfg["vocab"] - 1
    steps_per_block = -(-block_len // unmask_per_step)
    lock = torch.zeros((B, N), dtype=torch.uint8, device=dev)
    m_trace = torch.zeros(steps, dtype=torch.int32, device=dev)
    unmasked_trace = torch.zeros(steps, dtype=torch.int32, device=dev)
    n_rev = torch.zeros(B, dtype=torch.int32, device=dev)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    if unlock is not None:
        SL.surelock_set_unlocking(ctx, **unlock)                            # (resets the ctx)
        unlocked_trace = torch.zeros(steps, dtype=torch.int32, device=dev)
    SL.surelock_reset(ctx)
    ev[0].record()
    for t in range(steps):
        if select_fraction is None:
            lock_in = lock.clone() if observer is not None else None
            out = SL.surelock_step(ctx, tokens, mask_state, lock, kl_eps)
        else:
            skip = selection_skip_mask(lock, mask_state, select_fraction, t, select_seed)
            step_lock = lock | skip                                          # skipped rows are simply not active
            lock_in = step_lock.clone() if observer is not None else None
            out = SL.surelock_step(ctx, tokens, mask_state, step_lock, kl_eps)
            lock |= step_lock & (skip ^ 1)                                   # new locks come from computed rows only
        if observer is not None:
            observer(t, out, lock_in, lock, tokens, mask_state)
        if not surelock:
            lock.zero_()                                                     # baseline sampler: nothing stays locked
        m_trace[t:t + 1] = out.n_active
        blk = min(t // steps_per_block, max((N - n_prompt + block_len - 1) // block_len - 1, 0))
        lo = n_prompt + blk * block_len
        hi = min(lo + block_len, N)
        SL.surelock_update_mask(out.conf, out.argmax, out.active_idx, out.row_offsets, B, N, lo, hi, unmask_per_step,
                                mask_token, tokens, mask_state, n_rev)
        unmasked_trace[t:t + 1] = n_rev.sum(dtype=torch.int32)
        if unlock is not None and surelock:
            po = SL.surelock_probe_unlock(ctx, tokens, lock)
            if po.probed:
                unlocked_trace[t:t + 1] = po.n_unlocked
        ev[t + 1].record()
    torch.cuda.synchronize()
    ms = [ev[t].elapsed_time(ev[t + 1]) for t in range(steps)]
    extra = {}
    if unlock is not None:
        extra["unlocked_per_step"] = unlocked_trace.cpu().tolist()
        SL.surelock_set_unlocking(ctx, off=True)
    M = m_trace.cpu().tolist()
    um = unmasked_trace.cpu().tolist()
    total_s = sum(ms) * 1e-3
    f_base = algorithmic_flops_per_step(ctx.cfg, B, N)
    r_bar = sum(M) / float(steps * R)
    return dict(steps=steps, M_trace=M, ms_per_step=ms, unmasked_per_step=um, r_bar=r_bar,
                flops_ratio=r_bar,                                           # F_prop = (M / (B N)) F_base, step by step
                f_base_per_position=steps * f_base / R, f_prop_per_position=sum(M) * f_base / (R * R),
                e2e_tps=sum(um) / total_s if total_s > 0 else 0.0,
                step_tps=[u / (m * 1e-3) if m > 0 else 0.0 for u, m in zip(um, ms)],
                total_ms=sum(ms), locked_at_end=int(lock.sum().item()), masked_at_end=int(mask_state.sum().item()), **extra)
