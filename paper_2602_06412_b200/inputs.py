"""Seeded synthetic inputs shared by the CUDA path's tests, the CPU oracle's tests and the benchmark.

This module holds NO arithmetic of the method: it only draws random weights,
tokens, masks, lock patterns and logit pairs with the shapes and value
distributions of the workloads (LLaDA-8B-shaped transformer, N(0, 0.02) weights,
norm gains of one, prompt + masked generation region).  Both sides of a parity
test receive the same bytes produced here.
"""
from __future__ import annotations

import math
from typing import Dict, List

import torch

# name -> shape; "llada8b" is the LLaDA-8B shape (32 layers, d=4096, 32x128 heads, FFN 12288, vocab 126464)
MODEL_SHAPES: Dict[str, Dict] = {
    "tiny": dict(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ff=1024, vocab=2048,
                 rms_eps=1e-5, rope_theta=10000.0),
    "llada8b": dict(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ff=12288, vocab=126464,
                    rms_eps=1e-5, rope_theta=500000.0),
}


def model_shape(name: str, **overrides) -> Dict:
    cfg = dict(MODEL_SHAPES[name])
    cfg.update(overrides)
    return cfg


def _gen(seed: int, device="cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal(shape, std, seed, dtype, device):
    # drawn in fp32, then rounded to the storage dtype: both sides of a parity test widen the ROUNDED values
    t = torch.empty(shape, dtype=torch.float32, device=device)
    t.normal_(0.0, std, generator=_gen(seed, device))
    return t.to(dtype)


def make_layer_weights(cfg: Dict, layer: int, seed: int, dtype=torch.bfloat16, device="cpu",
                       std: float = 0.02) -> Dict:
    d, F = cfg["d_model"], cfg["d_ff"]
    hd = cfg["n_heads"] * cfg["head_dim"]
    s = seed * 1000003 + layer * 101
    return dict(
        attn_norm_g=torch.ones(d, dtype=dtype, device=device),
        wq=_normal((hd, d), std, s + 1, dtype, device),
        wk=_normal((hd, d), std, s + 2, dtype, device),
        wv=_normal((hd, d), std, s + 3, dtype, device),
        wo=_normal((d, hd), std, s + 4, dtype, device),
        ffn_norm_g=torch.ones(d, dtype=dtype, device=device),
        w_gate=_normal((F, d), std, s + 5, dtype, device),
        w_up=_normal((F, d), std, s + 6, dtype, device),
        w_down=_normal((d, F), std, s + 7, dtype, device),
    )


def make_weights(cfg: Dict, seed: int, dtype=torch.bfloat16, device="cpu", std: float = 0.02) -> Dict:
    """Random-init weights N(0, std^2) (0.02 in every workload), RMSNorm gains 1, matrices stored [out][in]."""
    d, V = cfg["d_model"], cfg["vocab"]
    w = dict(
        tok_emb=_normal((V, d), std, seed * 1000003 + 11, dtype, device),
        lm_head=_normal((V, d), std, seed * 1000003 + 13, dtype, device),
        final_norm_g=torch.ones(d, dtype=dtype, device=device),
        layers=[make_layer_weights(cfg, l, seed, dtype, device, std) for l in range(cfg["n_layers"])],
    )
    return w


def weights_to_numpy(w: Dict) -> Dict:
    """Widen (exactly) to float32 numpy arrays for the CPU side; bf16/fp32 values are preserved bit for bit."""
    def cv(t):
        return t.detach().to("cpu", torch.float32).numpy()
    out = {k: cv(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: cv(v) for k, v in lw.items()} for lw in w["layers"]]
    return out


def make_tokens(B: int, N: int, n_prompt: int, vocab: int, seed: int):
    """Prompt tokens uniform over [0, vocab-2]; the remaining positions hold the mask token vocab-1.

    Returns (tokens int32 [B][N], mask_state uint8 [B][N] with 1 = masked); each sequence has its own stream.
    """
    tokens = torch.full((B, N), vocab - 1, dtype=torch.int32)
    mask_state = torch.ones((B, N), dtype=torch.uint8)
    for b in range(B):
        g = _gen(seed * 7919 + b)
        tokens[b, :n_prompt] = torch.randint(0, vocab - 1, (n_prompt,), generator=g, dtype=torch.int32)
        mask_state[b, :n_prompt] = 0
    return tokens, mask_state


def random_lock(B: int, N: int, n_active: List[int], seed: int) -> torch.Tensor:
    """lock mask uint8 [B][N]: sequence b keeps a seeded uniform random subset of n_active[b] positions unlocked."""
    lock = torch.ones((B, N), dtype=torch.uint8)
    for b in range(B):
        perm = torch.randperm(N, generator=_gen(seed * 104729 + b))
        lock[b, perm[: n_active[b]]] = 0
    return lock


def contiguous_plus_random_lock(B: int, N: int, n_active: List[int], seed: int) -> torch.Tensor:
    """Long-context lock pattern: of the N - n_active[b] locked positions, 3/4 form a contiguous prefix and
    the rest are a seeded uniform sample of the remaining positions (own stream per sequence)."""
    lock = torch.zeros((B, N), dtype=torch.uint8)
    for b in range(B):
        n_lock = N - n_active[b]
        n_pre = (3 * n_lock) // 4
        lock[b, :n_pre] = 1
        rest = torch.randperm(N - n_pre, generator=_gen(seed * 15485863 + b))[: n_lock - n_pre] + n_pre
        lock[b, rest] = 1
    return lock


def bernoulli_lock_schedule(lock: torch.Tensor, lockable: torch.Tensor, p: float, seed: int) -> torch.Tensor:
    """Forced schedule: additionally lock each currently unlocked, lockable position with probability p."""
    u = torch.rand(lock.shape, generator=_gen(seed))
    add = (u < p) & (lock == 0) & lockable.bool()
    return (lock.bool() | add).to(torch.uint8)


def hidden_states(rows: int, d: int, seed: int, dtype=torch.bfloat16, device="cpu") -> torch.Tensor:
    """Random hidden states N(0, 1) for the single-layer microbenchmark."""
    return _normal((rows, d), 1.0, seed * 31 + 5, dtype, device)


def kl_logit_pairs(rows: int, vocab: int, seed: int, dtype=torch.bfloat16, device="cpu"):
    """Current / previous logit rows for the sure-test kernel run alone.

    cur ~ N(0, 3^2); prev = cur + sigma_r * N(0,1) with sigma_r log-uniform in [1e-3, 0.3] per row, so the
    step-wise KL spans the paper's threshold range (5e-8 ... 5e-2); every 20th row has prev == cur (KL = 0);
    every 4th row is "peaked" (+15 on one seeded logit in both), like a confident unmasked position.
    Returns (cur, prev, mask_state uint8 [rows], seeded 50/50).
    """
    g = _gen(seed * 613 + 1, device)
    cur = torch.empty((rows, vocab), dtype=torch.float32, device=device).normal_(0.0, 3.0, generator=g)
    r = torch.arange(rows, device=device)
    peak_col = torch.randint(0, vocab, (rows,), generator=g, device=device)
    peaked = (r % 4) == 1
    cur[r[peaked], peak_col[peaked]] += 15.0
    lo, hi = math.log(1e-3), math.log(0.3)
    sig = torch.exp(torch.rand(rows, generator=g, device=device) * (hi - lo) + lo)
    noise = torch.empty_like(cur).normal_(0.0, 1.0, generator=g)
    prev = cur + sig[:, None] * noise
    same = (r % 20) == 7
    cur_r = cur.to(dtype)
    prev_r = prev.to(dtype)
    prev_r[same] = cur_r[same]
    mask_state = (torch.rand(rows, generator=g, device=device) < 0.5).to(torch.uint8)
    return cur_r, prev_r, mask_state


def selection_scores(B: int, N: int, step: int, seed: int, device="cpu") -> torch.Tensor:
    """Seeded uniform scores [B][N] float32 for the selection surrogate of Experiment 5 (which positions a selection
    method would skip in this step is that method's business; the surrogate ranks positions by these scores).  Drawn
    on the CPU so that every consumer sees the same numbers, then moved to `device`."""
    return torch.rand((B, N), generator=_gen(seed * 1000003 + step), dtype=torch.float32).to(device)
