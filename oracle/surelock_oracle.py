"""SureLock locked forward and sure test: the CPU oracle.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain fp64 statement of what
one SureLock decoding step computes.  Only the test-suite, the smoke check and
the benchmark's CPU-baseline leg may import it; the CUDA product path never does,
and this module imports nothing from the CUDA package (numpy only).

Every function cites the passage of the paper it follows
("Stopping Computation for Converged Tokens in Masked Diffusion-LM Decoding").
Arithmetic is float64 throughout; inputs that the GPU receives rounded to bf16 or
fp32 are handed in already rounded and are widened here.  A matrix product is a
single library call (numpy ``@`` / ``einsum``); nothing is blocked, fused or
reordered beyond what the paper's Algorithm 1 states.

Readings taken where the paper leaves a choice open (each also listed in the
design notes of the repository):
  * the active set is "not locked" (Algorithm 1, line 6), not "unmasked and not
    locked" (Sec. 2.1 prose): masked positions must be computed to be predicted;
  * block structure (the paper says only LN / Proj / Attn / FFN): pre-norm
    residual block, RMSNorm, no biases, rotary embedding in rotate-half pairing
    applied with the ORIGINAL position index, keys cached after the rotation,
    softmax scale 1/sqrt(d_h), no attention mask, SwiGLU FFN with three matrices
    (the paper's 6*d*d_ff FLOP term), untied output projection;
  * KL(p_t || p_{t-1}) in nats from log-softmax; the test is D <= eps; a row
    without a previous posterior has D = +inf (Algorithm 1, line 19);
  * the lock test reads the mask state the forward pass saw (the state passed
    to this step), so a row can lock only after a step that was fed its token;
    Algorithm 1 read literally updates the masked set (line 16) before the test
    (line 20): step(..., unmask=...) plays that order;
  * p_{t-1} of a row that was NOT computed in step t-1 (it cannot happen under
    Algorithm 1's monotone locks; un-locking and selection methods make it
    happen): OracleState(prev_policy="previous_step") gives such a row D = +inf
    (Algorithm 1 line 19 compares with the posterior of step t-1, which the row
    does not have); prev_policy="keep_last" compares with the last posterior the
    row ever had (Sec. 2.1: a locked row keeps p_t <- p_{t*});
  * the optional confidence-percentile gate (Algorithm 1, line 21) is off unless asked for; when on, the
    percentile is taken per sequence over the locking candidates Z_t (Algorithm 1) rather than over all active
    rows (Sec. 2.2 prose), with linear interpolation between order statistics, and a row passes when
    u <= theta_m.

Parity pins (tests that run without a GPU) tie this file to closed forms, printed
values of the paper's Table 2, library routines of a different library (torch
fp64), and a pure-Python brute force.  Nothing here is unpinned except sampler
trajectories of trained models, which need the paper's weights and datasets.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import numpy as np

F64 = np.float64


@dataclasses.dataclass
class ModelCfg:
    """Shape of the masked-diffusion transformer (paper Sec. 2.3 symbols L, d, H, d_h, d_ff)."""
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0


# --------------------------------------------------------------------------
# Algorithm 1, line 6: active / locked split
# --------------------------------------------------------------------------
def active_set(lock: np.ndarray):
    """A_t = {i : lock_i = 0} per sequence, ascending (Algorithm 1, line 6).

    lock: [B][N] of 0/1.  Returns (active_idx, row_offsets): flat indices b*N+i of
    the unlocked positions in ascending order, and row_offsets[b] = number of
    active rows of sequences 0..b-1 (length B+1, last entry = M).
    """
    lock = np.asarray(lock)
    B, N = lock.shape
    idx: List[int] = []
    offs = [0]
    for b in range(B):
        for i in range(N):
            if lock[b, i] == 0:
                idx.append(b * N + i)
        offs.append(len(idx))
    return np.asarray(idx, dtype=np.int32), np.asarray(offs, dtype=np.int32)


# --------------------------------------------------------------------------
# Row-wise building blocks of the transformer block (Algorithm 1, lines 10-12)
# --------------------------------------------------------------------------
def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """"LN" of Algorithm 1 line 10, read as RMSNorm: x / sqrt(mean(x^2) + eps) * g."""
    x = np.asarray(x, F64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(g, F64)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary position embedding, rotate-half pairing (j, j + d_h/2).

    x: [m][H][d_h]; pos: [m] ORIGINAL sequence positions i (not packed rows).
    Pair j is rotated by the angle pos * theta**(-2j/d_h).
    """
    x = np.asarray(x, F64)
    m, H, dh = x.shape
    half = dh // 2
    j = np.arange(half, dtype=F64)
    inv_freq = np.asarray(theta, F64) ** (-2.0 * j / dh)          # [half]
    ang = np.asarray(pos, F64)[:, None] * inv_freq[None, :]       # [m][half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    out = np.empty_like(x)
    out[..., :half] = lo * c - hi * s
    out[..., half:] = hi * c + lo * s
    return out


def silu(x: np.ndarray) -> np.ndarray:
    x = np.asarray(x, F64)
    return x / (1.0 + np.exp(-x))


def attention_rows(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Attn(Q[A_t], K^all, V^all) of Algorithm 1 line 12 for ONE sequence.

    q: [m][H][d_h] queries of the active rows; K, V: [N][H][d_h], every position
    of the sequence (fresh rows for active positions, frozen rows for locked
    ones).  Bidirectional: every query sees all N keys.  Returns [m][H*d_h].
    """
    q = np.asarray(q, F64)
    K = np.asarray(K, F64)
    V = np.asarray(V, F64)
    m, H, dh = q.shape
    s = np.einsum("mhd,nhd->hmn", q, K) / np.sqrt(F64(dh))
    s = s - s.max(axis=-1, keepdims=True)
    a = np.exp(s)
    a = a / a.sum(axis=-1, keepdims=True)
    o = np.einsum("hmn,nhd->mhd", a, V)
    return o.reshape(m, H * dh)


def log_softmax(z: np.ndarray) -> np.ndarray:
    """log p = z - logsumexp(z) along the vocabulary (Algorithm 1, line 15)."""
    z = np.asarray(z, F64)
    zmax = z.max(axis=-1, keepdims=True)
    lse = zmax + np.log(np.exp(z - zmax).sum(axis=-1, keepdims=True))
    return z - lse


def kl_rows(logp: np.ndarray, logp_prev: np.ndarray) -> np.ndarray:
    """D = KL(p_t || p_{t-1}) = sum_v p_t(v) (log p_t(v) - log p_{t-1}(v)), nats (Sec. 2.2)."""
    logp = np.asarray(logp, F64)
    logp_prev = np.asarray(logp_prev, F64)
    return np.sum(np.exp(logp) * (logp - logp_prev), axis=-1)


def kl_from_logits(z: np.ndarray, z_prev: np.ndarray) -> np.ndarray:
    """Step-wise KL of the posteriors given raw (temperature-1) logits of both steps."""
    return kl_rows(log_softmax(z), log_softmax(z_prev))


def posterior_stats(z: np.ndarray):
    """(conf, argmax) with conf = max_v p(v) = 1 - u (Algorithm 1 line 18); lowest index on ties."""
    logp = log_softmax(z)
    am = np.argmax(logp, axis=-1)
    conf = np.exp(np.take_along_axis(logp, am[..., None], axis=-1))[..., 0]
    return conf, am.astype(np.int32)


def sure_test(D: np.ndarray, masked: np.ndarray, kl_eps: float) -> np.ndarray:
    """F_t = {i in A_t, unmasked : D_i <= eps} (Algorithm 1, lines 20 and 23, gate off). NaN never locks."""
    D = np.asarray(D, F64)
    return (np.asarray(masked) == 0) & (D <= kl_eps)


def percentile_linear(values: Sequence[float], m: float) -> float:
    """Empirical m-th percentile (0 <= m <= 100) with linear interpolation between order statistics:
    x sorted ascending, h = (n-1) m / 100, result x[floor h] + (h - floor h)(x[ceil h] - x[floor h]).
    An empty set has no percentile: returns -inf (so that nothing passes a "<= theta" test)."""
    x = sorted(float(v) for v in values)
    n = len(x)
    if n == 0:
        return -np.inf
    h = (n - 1) * (float(m) / 100.0)
    lo = int(np.floor(h))
    hi = min(lo + 1, n - 1)
    return x[lo] + (h - lo) * (x[hi] - x[lo])


def confidence_gate(conf: np.ndarray, candidate: np.ndarray, seq_of_row: np.ndarray, n_seq: int, m: float):
    """Optional confidence gate (Algorithm 1 lines 18, 21 and 23; Sec. 2.2 "Optional: Confidence gate").

    u_i = 1 - max_v p_i(v) = 1 - conf_i.  Per sequence, theta_m is the m-th percentile of u over the locking
    candidates Z_t (active and unmasked rows of that sequence); a candidate passes when u_i <= theta_m, i.e. it is
    among the top-m % most confident candidates.  Returns (passes [rows] bool, theta [n_seq]).
    """
    u = 1.0 - np.asarray(conf, F64)
    candidate = np.asarray(candidate, bool)
    seq_of_row = np.asarray(seq_of_row)
    theta = np.full(n_seq, -np.inf, F64)
    passes = np.zeros(len(u), bool)
    for b in range(n_seq):
        rows = np.flatnonzero((seq_of_row == b) & candidate)
        theta[b] = percentile_linear(u[rows], m)
        passes[rows] = u[rows] <= theta[b]
    return passes, theta


# --------------------------------------------------------------------------
# Unmasking policy (Algorithm 1 line 16)
# --------------------------------------------------------------------------
def update_mask(tokens: np.ndarray, mask_state: np.ndarray, conf: np.ndarray, argmax: np.ndarray,
                active_idx: np.ndarray, lo: int, hi: int, k: int, mask_token: int):
    """UpdateMASK (Algorithm 1 line 16), the confidence-ordered policy the paper describes for masked-diffusion
    samplers (App. "semantically distant options": per step a fixed number of masked positions with the highest
    posterior probability become concrete tokens) restricted to one semi-autoregressive block (Sec. 4 set-up).

    Per sequence: among the positions lo <= n < hi that are still masked, the k with the largest conf = max_v p(v)
    (ties: lowest position) take their argmax token and become unmasked; everything else is unchanged.  A position
    whose argmax is the mask token itself takes token 0 (a sampler never emits the mask token).  The Algorithm leaves
    the policy open; this reading is the harness's, not part of the method.

    tokens int [B][N], mask_state uint8 [B][N] (1 = masked), conf / argmax per packed active row, active_idx the
    flat position b * N + n of each packed row.  Returns (new tokens, new mask_state, revealed per sequence).
    """
    tokens = np.array(tokens, dtype=np.int64)
    mask_state = np.array(mask_state, dtype=np.uint8)
    B, N = tokens.shape
    conf = np.asarray(conf, F64)
    revealed = np.zeros(B, np.int64)
    for b in range(B):
        cand = []                                      # (position, row) of masked block positions that were computed
        for r, flat in enumerate(np.asarray(active_idx)):
            bb, n = divmod(int(flat), N)
            if bb == b and lo <= n < hi and mask_state[b, n] == 1:
                cand.append((n, r))
        for _ in range(k):
            if not cand:
                break
            best = max(cand, key=lambda nr: (conf[nr[1]], -nr[0]))      # highest conf, then lowest position
            n, r = best
            tok = int(argmax[r])
            tokens[b, n] = 0 if tok == mask_token else tok
            mask_state[b, n] = 0
            revealed[b] += 1
            cand.remove(best)
    return tokens, mask_state, revealed


def selection_skip(lock: np.ndarray, mask_state: np.ndarray, scores: np.ndarray, fraction: float) -> np.ndarray:
    """The selection surrogate of Experiment 5 ("computes only on a fixed fraction k of active tokens at each step").
    Which positions a selection method drops is not the paper's subject; the surrogate's rule, given per-position
    scores as input: per sequence, with U = number of unlocked positions, skip the floor((1 - k) U) eligible positions
    (unlocked and unmasked: a masked position is always computed, the sampler needs its posterior) that have the
    lowest scores, ties to the lower position; fewer if there are not that many eligible ones.
    Returns uint8 [B][N], 1 = not computed in this step."""
    lock = np.asarray(lock)
    B, N = lock.shape
    skip = np.zeros((B, N), np.uint8)
    for b in range(B):
        unlocked = [i for i in range(N) if lock[b, i] == 0]
        eligible = [i for i in unlocked if mask_state[b, i] == 0]
        n_skip = min(int(np.floor(np.float32(len(unlocked)) * np.float32(1.0 - fraction))), len(eligible))
        for i in sorted(eligible, key=lambda i: (scores[b, i], i))[:n_skip]:
            skip[b, i] = 1
    return skip


# --------------------------------------------------------------------------
# Algorithmic FLOPs (Sec. 2.3)
# --------------------------------------------------------------------------
def flops_base_step(cfg: ModelCfg, B: int, N: int, n_kv_heads: Optional[int] = None) -> int:
    """F^t_base of Sec. 2.3: GEMM-only FLOPs of one full-recompute step of a batch."""
    L, d, H, dh, dff = cfg.n_layers, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.d_ff
    Hkv = H if n_kv_heads is None else n_kv_heads
    return L * (4 * B * H * N * N * dh + 2 * B * N * d * d + 2 * B * N * d * d
                + 4 * B * N * d * Hkv * dh + 6 * B * N * d * dff)


def flops_prop_step(cfg: ModelCfg, B: int, N: int, M: int) -> float:
    """F^t_prop = (M / (B N)) F^t_base (Sec. 2.3, SureLock paragraph)."""
    return flops_base_step(cfg, B, N) * (M / (B * N))


# --------------------------------------------------------------------------
# One transformer block on the active rows (Algorithm 1, lines 10-13)
# --------------------------------------------------------------------------
def qkv_rows(cfg: ModelCfg, lw: Dict[str, np.ndarray], x: np.ndarray, pos: np.ndarray):
    """Proj_{Q,K,V}(LN(x[A_t])) with the rotation applied to q and k (line 10).

    x: [m][d] block input of active rows; pos: [m] their sequence positions.
    Weight matrices are stored [out][in].  Returns q, k, v as [m][H][d_h].
    """
    H, dh = cfg.n_heads, cfg.head_dim
    h = rmsnorm(x, lw["attn_norm_g"], cfg.rms_eps)
    m = h.shape[0]
    q = (h @ np.asarray(lw["wq"], F64).T).reshape(m, H, dh)
    k = (h @ np.asarray(lw["wk"], F64).T).reshape(m, H, dh)
    v = (h @ np.asarray(lw["wv"], F64).T).reshape(m, H, dh)
    return rope(q, pos, cfg.rope_theta), rope(k, pos, cfg.rope_theta), v


def ffn_rows(cfg: ModelCfg, lw: Dict[str, np.ndarray], x: np.ndarray) -> np.ndarray:
    """x + W_d( silu(W_g h) * (W_u h) ), h = RMSNorm(x): the FFN sub-block on active rows (line 12)."""
    h = rmsnorm(x, lw["ffn_norm_g"], cfg.rms_eps)
    a = silu(h @ np.asarray(lw["w_gate"], F64).T) * (h @ np.asarray(lw["w_up"], F64).T)
    return np.asarray(x, F64) + a @ np.asarray(lw["w_down"], F64).T


def layer_rows(cfg: ModelCfg, lw: Dict[str, np.ndarray], x: np.ndarray, pos: np.ndarray,
               Kc: np.ndarray, Vc: np.ndarray) -> np.ndarray:
    """One block for the active rows of ONE sequence (Algorithm 1, lines 10-13).

    x: [m][d]; pos: [m] ascending positions of those rows; Kc, Vc: [N][H][d_h]
    this layer's cache of the sequence, updated IN PLACE at the active positions
    (line 11: fresh K/V for A_t, cached K/V for L_t) before attention reads all N
    rows.  Locked rows are not touched (line 13: they pass through).
    """
    x = np.asarray(x, F64)
    q, k, v = qkv_rows(cfg, lw, x, pos)
    Kc[pos] = k
    Vc[pos] = v
    o = attention_rows(q, Kc, Vc)
    x = x + o @ np.asarray(lw["wo"], F64).T
    return ffn_rows(cfg, lw, x)


def layer_flops(cfg: ModelCfg, m: int, N: int) -> int:
    """GEMM FLOPs layer_rows() performs for m active rows against N keys (same terms as Sec. 2.3)."""
    d, H, dh, dff = cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.d_ff
    return 4 * H * m * N * dh + 2 * m * d * d + 2 * m * d * d + 4 * m * d * H * dh + 6 * m * d * dff


# --------------------------------------------------------------------------
# Sampler-visible state and one full step (Algorithm 1, lines 6-24)
# --------------------------------------------------------------------------
class OracleState:
    """lock-independent state of Algorithm 1 lines 1-2: per-layer K/V caches and p_{t-1}.

    K, V: [L][B][N][H][d_h] float64.  prev_logp: [B][N][V] float64 with
    prev_valid [B][N]; an invalid row stands for "p_{t-1} = None".

    prev_policy decides what p_{t-1} is for a row that was not computed in the step just before (see the module
    header): "previous_step" -> it has none (D = +inf), "keep_last" -> the last posterior it ever had.  Under
    Algorithm 1 itself (locks only grow, every unlocked row is computed every step) the two never differ.
    """

    def __init__(self, cfg: ModelCfg, B: int, N: int, prev_policy: str = "previous_step"):
        if prev_policy not in ("previous_step", "keep_last"):
            raise ValueError(prev_policy)
        self.prev_policy = prev_policy
        self.cfg, self.B, self.N = cfg, B, N
        shp = (cfg.n_layers, B, N, cfg.n_heads, cfg.head_dim)
        self.K = np.zeros(shp, F64)
        self.V = np.zeros(shp, F64)
        self.prev_logp = np.zeros((B, N, cfg.vocab), F64)
        self.prev_valid = np.zeros((B, N), bool)
        self.flops = 0

    def reset(self):
        self.prev_valid[:] = False
        self.flops = 0


def step(state: OracleState, weights: Dict, tokens: np.ndarray, mask_state: np.ndarray,
         lock: np.ndarray, kl_eps: float, logits_round=None, conf_gate_m: Optional[float] = None,
         unmask=None, skip: Optional[np.ndarray] = None, kl_eps_rows: Optional[np.ndarray] = None,
         may_lock: Optional[np.ndarray] = None):
    """One SureLock step (Algorithm 1, lines 6-15 and 18-24; line 16 belongs to the caller).

    unmask: None (default) = the lock test of lines 20-23 reads the mask state that was passed in, i.e. the state
    the forward pass saw.  A callable plays Algorithm 1 in its LITERAL order: it is line 16, called after the
    posteriors of line 15 as unmask(tokens, mask_state, conf, argmax, active_idx) -> (tokens', mask_state'), and
    the candidates of line 20 are then taken from mask_state' (a position revealed in this step can lock in this
    step, with K/V that were computed from the mask token).  The result carries tokens' / mask_state'.

    skip: optional [B][N] of 0/1, the selection surrogate of Experiment 5: an unlocked position with skip = 1 is not
    computed in this step (it is not in the active set; its cached K/V and its lock bit stay as they are, it gets no
    posterior), so that only a fraction of the not-yet-locked positions is recomputed; new locks come from computed
    rows only.

    kl_eps_rows / may_lock: optional [B][N] arrays used by the un-locking extension (App. "Optional Unlocking"):
    a per-position threshold that replaces kl_eps (the stricter rho * eps of a position that was un-locked before)
    and a per-position permission (0 during the cool-down after an un-lock).

    weights: {"tok_emb": [V][d], "lm_head": [V][d], "final_norm_g": [d],
              "layers": [ {attn_norm_g, wq, wk, wv, wo, ffn_norm_g, w_gate, w_up, w_down} ]}.
    tokens [B][N] int; mask_state [B][N] (1 = masked); lock [B][N] (1 = locked),
    NOT modified.  logits_round: optional callable applied to the logits before
    the posterior is formed (lets a test reproduce the storage precision of the
    logits, e.g. rounding to bf16); None = no rounding.

    Returns dict: active_idx, row_offsets, hidden [M][d] (x^{(L+1)}), logits
    [M][V], kl [M], conf [M], argmax [M], new_lock [B][N], flops (GEMM FLOPs of
    the L blocks, the quantity Sec. 2.3 counts).
    """
    cfg, B, N = state.cfg, state.B, state.N
    tokens = np.asarray(tokens)
    not_computed = np.asarray(lock) != 0
    if skip is not None:
        not_computed = not_computed | (np.asarray(skip) != 0)
    idx, offs = active_set(not_computed.astype(np.uint8))
    M = len(idx)
    emb = np.asarray(weights["tok_emb"])
    hidden = np.zeros((M, cfg.d_model), F64)
    flops = 0
    for b in range(B):
        r0, r1 = int(offs[b]), int(offs[b + 1])
        if r1 == r0:
            continue
        pos = (idx[r0:r1] - b * N).astype(np.int64)
        x = np.asarray(emb[tokens[b, pos]], F64)                  # line 7
        for l, lw in enumerate(weights["layers"]):                # lines 9-14
            x = layer_rows(cfg, lw, x, pos, state.K[l, b], state.V[l, b])
            flops += layer_flops(cfg, r1 - r0, N)
        hidden[r0:r1] = x
    hn = rmsnorm(hidden, weights["final_norm_g"], cfg.rms_eps)
    logits = hn @ np.asarray(weights["lm_head"], F64).T           # line 15
    if logits_round is not None:
        logits = np.asarray(logits_round(logits), F64)
    logp = log_softmax(logits)
    conf, am = posterior_stats(logits)                            # line 18
    bb, ii = idx // N, idx % N
    D = np.full(M, np.inf, F64)                                   # line 19: KL(p_t || p_{t-1}) if t > 1 else inf
    # p_{t-1} is the posterior computed at step t-1.  Under Algorithm 1 the active set only shrinks, so every active row
    # has one from the second step on; a row that an extension (un-locking, a selection method) returns to the active
    # set after steps in which it was not computed has none, and gets inf like a first step.
    has_prev = state.prev_valid[bb, ii]
    if has_prev.any():
        D[has_prev] = kl_rows(logp[has_prev], state.prev_logp[bb[has_prev], ii[has_prev]])
    new_tokens, new_mask = tokens, np.asarray(mask_state)
    if unmask is not None:                                        # line 16 in its literal place, before line 20
        new_tokens, new_mask = unmask(tokens, np.asarray(mask_state), conf, am, idx)
        new_tokens, new_mask = np.asarray(new_tokens), np.asarray(new_mask)
    eps_rows = kl_eps if kl_eps_rows is None else np.asarray(kl_eps_rows, F64)[bb, ii]
    lockable = sure_test(D, new_mask[bb, ii], eps_rows)           # lines 20, 23
    if may_lock is not None:
        lockable = lockable & (np.asarray(may_lock)[bb, ii] != 0)
    theta = None
    if conf_gate_m is not None:                                   # line 21: u <= theta_m over the candidates Z_t
        gate, theta = confidence_gate(conf, new_mask[bb, ii] == 0, bb, B, conf_gate_m)
        lockable = lockable & gate
    new_lock = np.array(lock, dtype=np.uint8, copy=True)
    new_lock[bb[lockable], ii[lockable]] = 1                      # line 24
    state.prev_logp[bb, ii] = logp                                # rows that were not computed keep their last posterior
    if state.prev_policy == "previous_step":
        state.prev_valid[:] = False                               # "previous" means computed in the step just taken
    state.prev_valid[bb, ii] = True
    state.flops += flops
    return dict(active_idx=idx, row_offsets=offs, hidden=hidden, logits=logits, kl=D,
                conf=conf, argmax=am, new_lock=new_lock, flops=flops, theta=theta, logp=logp,
                tokens=new_tokens, mask_state=new_mask)


# --------------------------------------------------------------------------
# Optional un-locking (App. "Optional Unlocking")
# --------------------------------------------------------------------------
# The appendix leaves open what the "budgeted proxy" is, how theta_t treats a sequence without active rows, and says
# "if any holds" above an equation whose three conditions are joined by AND.  Readings taken here:
#   * the proxy recomputes the LOCKED rows as queries through the whole stack against the caches as they stand
#     (variable-length attention over all N cached keys / values) WITHOUT writing their K/V back: probe_rows();
#   * the rule is the printed equation: all three conditions must hold;
#   * theta_t is, per sequence, the m-th percentile (linear interpolation, as for the confidence gate) of
#     u = 1 - max_v p over the rows that were ACTIVE in step t; a sequence with no active row has no reference
#     uncertainty and un-locks nothing (theta = +inf);
#   * a position un-locked after step t is active from step t+1 on; "invalidate cached K/V" needs no action because
#     every active row's K/V is rewritten in every step; it may lock again from step t + D_cool + 1 on, and from then
#     on under the threshold rho * eps.
@dataclasses.dataclass
class UnlockParams:
    period: int            # P: the probe runs after every P-th step
    eps_unlock: float      # drift threshold on KL(p_hat_t || p_{t*})
    d_interval: int        # a position stays locked for more than this many steps before it may be un-locked
    d_cool: int            # steps after an un-lock during which the position cannot lock again
    rho: float             # re-lock threshold factor, rho <= 1
    m: float               # percentile (0..100) of the active rows' uncertainty that gives theta_t


class UnlockState:
    """What un-locking needs beyond Algorithm 1's state: per position the step t* at which it locked, the posterior
    p_{t*} it had then (as log-probabilities), the last step of its cool-down, and whether it was ever un-locked."""

    def __init__(self, B: int, N: int, V: int):
        self.t_star = np.full((B, N), -1, np.int64)
        self.frozen_logp = np.zeros((B, N, V), F64)
        self.cool_until = np.full((B, N), -1, np.int64)
        self.relock = np.zeros((B, N), bool)


def record_locks(ustate: UnlockState, t: int, lock_before: np.ndarray, step_out: Dict, N: int) -> None:
    """After step t: every position that this step locked gets t* = t and keeps its posterior of step t as p_{t*}."""
    idx = np.asarray(step_out["active_idx"])
    bb, ii = idx // N, idx % N
    newly = (np.asarray(step_out["new_lock"])[bb, ii] != 0) & (np.asarray(lock_before)[bb, ii] == 0)
    ustate.t_star[bb[newly], ii[newly]] = t
    ustate.frozen_logp[bb[newly], ii[newly]] = np.asarray(step_out["logp"])[newly]


def relock_thresholds(ustate: UnlockState, kl_eps: float, rho: float, t: int):
    """Per-position lock threshold and permission for step t: rho * eps for a position that was un-locked before,
    eps otherwise; no locking while t <= cool_until (the D_cool steps after the un-lock)."""
    eps_rows = np.where(ustate.relock, rho * kl_eps, kl_eps).astype(F64)
    may_lock = (t > ustate.cool_until).astype(np.uint8)
    return eps_rows, may_lock


def probe_rows(state: OracleState, weights: Dict, tokens: np.ndarray, lock: np.ndarray):
    """The proxy: posteriors p_hat_t of the LOCKED rows, recomputed against the caches as they stand.

    For every sequence the locked positions (ascending) go through every block like active rows do in step()
    (lines 7, 10, 12, 15), except that line 11 is not executed: their fresh k, v are discarded and attention reads
    all N cached rows, their own frozen entries included.  Nothing in `state` is modified.
    Returns (locked_idx flat ascending, logits [n][V], logp [n][V], conf [n]).
    """
    cfg, B, N = state.cfg, state.B, state.N
    tokens = np.asarray(tokens)
    idx, offs = active_set(1 - (np.asarray(lock) != 0).astype(np.uint8))      # positions with lock = 1
    n = len(idx)
    hidden = np.zeros((n, cfg.d_model), F64)
    emb = np.asarray(weights["tok_emb"])
    for b in range(B):
        r0, r1 = int(offs[b]), int(offs[b + 1])
        if r1 == r0:
            continue
        pos = (idx[r0:r1] - b * N).astype(np.int64)
        x = np.asarray(emb[tokens[b, pos]], F64)
        for l, lw in enumerate(weights["layers"]):
            q, _, _ = qkv_rows(cfg, lw, x, pos)
            o = attention_rows(q, state.K[l, b], state.V[l, b])
            x = ffn_rows(cfg, lw, x + o @ np.asarray(lw["wo"], F64).T)
        hidden[r0:r1] = x
    logits = rmsnorm(hidden, weights["final_norm_g"], cfg.rms_eps) @ np.asarray(weights["lm_head"], F64).T
    logp = log_softmax(logits)
    conf, _ = posterior_stats(logits)
    return idx, logits, logp, conf


def unlock_test(u_probe, D_probe, theta, t: int, t_star, p: UnlockParams) -> np.ndarray:
    """The un-lock rule: u~ > theta_t  AND  D~ > eps_unlock  AND  t - t* > D_interval (element-wise)."""
    return (np.asarray(u_probe, F64) > np.asarray(theta, F64)) & (np.asarray(D_probe, F64) > p.eps_unlock) & \
           ((t - np.asarray(t_star)) > p.d_interval)


def active_uncertainty_threshold(conf_active: np.ndarray, active_idx: np.ndarray, B: int, N: int, m: float):
    """theta_t per sequence: the m-th percentile of u = 1 - conf over the rows that were active in step t;
    +inf for a sequence without active rows."""
    u = 1.0 - np.asarray(conf_active, F64)
    seq = np.asarray(active_idx) // N
    theta = np.full(B, np.inf, F64)
    for b in range(B):
        rows = np.flatnonzero(seq == b)
        if len(rows):
            theta[b] = percentile_linear(u[rows], m)
    return theta


def probe_unlock(state: OracleState, ustate: UnlockState, weights: Dict, tokens: np.ndarray, lock: np.ndarray, t: int,
                 conf_active: np.ndarray, active_idx: np.ndarray, p: UnlockParams, logits_round=None):
    """The probe after step t (called when t is a multiple of P): proxy posteriors of the locked rows, drift against
    p_{t*}, the un-lock rule, and the state changes of an un-lock.  `lock` is the mask after step t's lock update;
    conf_active / active_idx are step t's outputs.  Returns dict(new_lock, locked_idx, u, drift, theta, unlocked)."""
    B, N = state.B, state.N
    idx, logits, logp, conf = probe_rows(state, weights, tokens, lock)
    if logits_round is not None:
        logits = np.asarray(logits_round(logits), F64)
        logp = log_softmax(logits)
        conf, _ = posterior_stats(logits)
    bb, ii = idx // N, idx % N
    drift = kl_rows(logp, ustate.frozen_logp[bb, ii])
    theta = active_uncertainty_threshold(conf_active, active_idx, B, N, p.m)
    u = 1.0 - conf
    fire = unlock_test(u, drift, theta[bb], t, ustate.t_star[bb, ii], p)
    new_lock = np.array(lock, dtype=np.uint8, copy=True)
    new_lock[bb[fire], ii[fire]] = 0
    ustate.cool_until[bb[fire], ii[fire]] = t + p.d_cool
    ustate.relock[bb[fire], ii[fire]] = True
    return dict(new_lock=new_lock, locked_idx=idx, u=u, drift=drift, theta=theta, unlocked=fire, logits=logits)
