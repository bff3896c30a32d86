"""Pins that tie the CPU oracle to things other than itself (no GPU needed).

Each test checks `oracle/surelock_oracle.py` against a value the paper prints, a
closed form, an invariant the paper states, a routine of a different library
(torch fp64, scipy), or a pure-Python brute force.
"""
import math
import os

import numpy as np
import pytest
import scipy.special
import torch
import torch.nn.functional as F

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import inputs
from tests import dense_reference as DR

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _cfg(**kw):
    c = inputs.model_shape("tiny", **kw)
    return c, O.ModelCfg(**c)


def _small(seed=3, L=2, d=64, H=2, dh=32, Fd=128, V=97, std=0.25):
    c, oc = _cfg(n_layers=L, d_model=d, n_heads=H, head_dim=dh, d_ff=Fd, vocab=V)
    w = inputs.make_weights(c, seed, dtype=torch.float32, std=std)
    return c, oc, w, inputs.weights_to_numpy(w)


def _w64(w):
    out = {k: v.double() for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: v.double() for k, v in lw.items()} for lw in w["layers"]]
    return out


# ------------------------------------------------------------------ FLOPs (Sec. 2.3, Tables 1-2)
def test_flops_table2_printed_values():
    oc = O.ModelCfg(**inputs.model_shape("llada8b"))
    rows = [l.split() for l in open(os.path.join(GOLD, "table2_fbase.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 8
    for n_gen, steps, printed in rows:
        Nb, B = 64 + int(n_gen), 4
        per_pos = int(steps) * O.flops_base_step(oc, B, Nb) / (B * Nb)
        # four printed digits; one row (1.7996e12 printed as 1.799e+12) is truncated rather than rounded
        assert abs(per_pos / float(printed) - 1.0) < 4e-4, (n_gen, steps, per_pos, printed)


def test_flops_closed_form_terms():
    # each term of the Sec. 2.3 formula, isolated by zeroing the others
    oc = O.ModelCfg(n_layers=3, d_model=10, n_heads=2, head_dim=5, d_ff=7, vocab=11)
    B, N = 2, 6
    assert O.flops_base_step(oc, B, N) == 3 * (4 * 2 * 2 * 36 * 5 + 2 * 2 * 6 * 100 * 2 + 4 * 2 * 6 * 10 * 10
                                                + 6 * 2 * 6 * 10 * 7)
    # fewer K/V heads only shrink the K,V projection term
    assert O.flops_base_step(oc, B, N) - O.flops_base_step(oc, B, N, n_kv_heads=1) == 3 * 4 * B * N * 10 * 5


def test_flops_ratio_is_active_ratio_table1():
    oc = O.ModelCfg(**inputs.model_shape("llada8b"))
    B, N = 4, 414
    for l in open(os.path.join(GOLD, "table1_ratio.txt")):
        if not l.strip() or l[0] == "#":
            continue
        n_gen, eps, rbar, fb, fp, ratio = l.split()
        assert abs(float(fp) / float(fb) - float(ratio)) < 1.5e-3
        assert abs(float(rbar) - float(ratio)) <= 1.001e-3          # paper: r_bar tracks the FLOP ratio
        M = round(float(rbar) * B * N)
        assert abs(O.flops_prop_step(oc, B, N, M) / O.flops_base_step(oc, B, N) - M / (B * N)) < 1e-15


def test_counted_flops_match_formula():
    c, oc, w, wn = _small()
    B, N = 2, 12
    tokens, mask = inputs.make_tokens(B, N, 6, c["vocab"], 1)
    st = O.OracleState(oc, B, N)
    lock0 = np.zeros((B, N), np.uint8)
    r = O.step(st, wn, tokens.numpy(), mask.numpy(), lock0, 1e-3)
    assert r["flops"] == O.flops_base_step(oc, B, N)
    lock = inputs.random_lock(B, N, [5, 9], 4).numpy()
    r = O.step(st, wn, tokens.numpy(), mask.numpy(), lock, 1e-3)
    # SureLock count: per-sequence m_b rows against N keys == (M_b / N) share of the per-sequence baseline
    assert r["flops"] == sum(O.flops_base_step(oc, 1, N) * m // N for m in (5, 9))
    assert abs(r["flops"] - O.flops_prop_step(oc, B, N, 14)) < 1e-6 * r["flops"]


# ------------------------------------------------------------------ building blocks vs library routines
def test_rmsnorm_silu_logsoftmax_vs_torch():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(7, 33)) * 3
    g = rng.normal(size=33)
    t = torch.from_numpy
    np.testing.assert_allclose(O.rmsnorm(x, g, 1e-5), F.rms_norm(t(x), (33,), t(g), 1e-5).numpy(), rtol=1e-13)
    np.testing.assert_allclose(O.silu(x), F.silu(t(x)).numpy(), rtol=1e-13)
    np.testing.assert_allclose(O.log_softmax(x), F.log_softmax(t(x), -1).numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(O.log_softmax(x), scipy.special.log_softmax(x, axis=-1), rtol=1e-12, atol=1e-13)


def test_attention_is_textbook_sdpa():
    rng = np.random.default_rng(1)
    m, N, H, dh = 5, 19, 3, 8
    q, K, V = rng.normal(size=(m, H, dh)), rng.normal(size=(N, H, dh)), rng.normal(size=(N, H, dh))
    t = lambda a: torch.from_numpy(a).transpose(0, 1)
    ref = F.scaled_dot_product_attention(t(q), t(K), t(V)).transpose(0, 1).reshape(m, H * dh).numpy()
    np.testing.assert_allclose(O.attention_rows(q, K, V), ref, rtol=1e-12, atol=1e-14)
    # a single key: attention returns that key's value whatever the query
    one = O.attention_rows(q, K[:1], V[:1])
    np.testing.assert_allclose(one, np.broadcast_to(V[:1].reshape(1, -1), one.shape), rtol=1e-14)


def test_rope_properties():
    rng = np.random.default_rng(2)
    H, dh, theta = 2, 16, 10000.0
    x = rng.normal(size=(4, H, dh))
    y = rng.normal(size=(4, H, dh))
    np.testing.assert_allclose(O.rope(x, np.zeros(4), theta), x, rtol=0, atol=0)          # position 0 = identity
    r = O.rope(x, np.array([3, 17, 100, 4095]), theta)
    np.testing.assert_allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)
    # inner product depends only on the position difference
    a = np.einsum("mhd,mhd->mh", O.rope(x, np.full(4, 40), theta), O.rope(y, np.full(4, 33), theta))
    b = np.einsum("mhd,mhd->mh", O.rope(x, np.full(4, 1007), theta), O.rope(y, np.full(4, 1000), theta))
    np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)
    # explicit 2x2 rotation of pair (j, j+dh/2) by pos * theta^(-2j/dh)
    pos, j = 5, 3
    ang = pos * theta ** (-2 * j / dh)
    v = O.rope(x[:1], np.array([pos]), theta)[0, 0]
    assert abs(v[j] - (x[0, 0, j] * math.cos(ang) - x[0, 0, j + 8] * math.sin(ang))) < 1e-14
    assert abs(v[j + 8] - (x[0, 0, j + 8] * math.cos(ang) + x[0, 0, j] * math.sin(ang))) < 1e-14
    # a different library's complex-multiplication form, positions 0..N-1
    xs = rng.normal(size=(9, H, dh))
    np.testing.assert_allclose(O.rope(xs, np.arange(9), theta),
                               DR._rope_complex(torch.from_numpy(xs), theta).numpy(), rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ KL (Sec. 2.2) closed forms and library
def test_kl_closed_forms_and_library():
    rng = np.random.default_rng(3)
    V = 211
    z = rng.normal(size=(6, V)) * 3
    zp = z + rng.normal(size=(6, V)) * 0.2
    kl = O.kl_from_logits(z, zp)
    assert np.all(kl >= 0)
    assert np.all(O.kl_from_logits(z, z) == 0.0)                                   # KL(p||p) = 0 exactly
    p, q = scipy.special.softmax(z, -1), scipy.special.softmax(zp, -1)
    np.testing.assert_allclose(kl, scipy.special.rel_entr(p, q).sum(-1), rtol=1e-10)
    np.testing.assert_allclose(kl, DR.kl_torch(torch.from_numpy(z), torch.from_numpy(zp)).numpy(), rtol=1e-10)
    # direction matters: KL(p_t || p_{t-1}), not the reverse
    assert not np.allclose(kl, O.kl_from_logits(zp, z), rtol=1e-3)
    # shift invariance in either row (raw-logit, temperature-1 criterion)
    np.testing.assert_allclose(O.kl_from_logits(z + 7.5, zp - 3.25), kl, rtol=1e-9)
    # Pinsker (used in the paper's proof): ||p - q||_1 <= sqrt(2 KL)
    assert np.all(np.abs(p - q).sum(-1) <= np.sqrt(2 * kl) + 1e-15)
    # against the uniform posterior: KL = log V - H(p)
    Hp = -(p * np.log(p)).sum(-1)
    np.testing.assert_allclose(O.kl_from_logits(z, np.zeros_like(z)), np.log(V) - Hp, rtol=1e-11)
    # two-level logits (a,0,...,0) vs (b,0,...,0): closed form
    a, b = 2.0, -1.0
    za, zb = np.zeros((1, V)), np.zeros((1, V))
    za[0, 0], zb[0, 0] = a, b
    Za, Zb = math.exp(a) + V - 1, math.exp(b) + V - 1
    closed = math.exp(a) / Za * (a - math.log(Za) - b + math.log(Zb)) + (V - 1) / Za * (math.log(Zb) - math.log(Za))
    assert abs(O.kl_from_logits(za, zb)[0] - closed) < 1e-14
    # small-perturbation asymptote KL ~ Var_p(delta)/2
    dl = rng.normal(size=(1, V)) * 1e-3
    var = (p[:1] * dl ** 2).sum() - ((p[:1] * dl).sum()) ** 2
    assert abs(O.kl_from_logits(z[:1], z[:1] - dl)[0] / (0.5 * var) - 1) < 5e-3


def test_posterior_stats_and_sure_test():
    z = np.array([[0.0, 2.0, 2.0, -1.0], [5.0, 0.0, 0.0, 0.0]])
    conf, am = O.posterior_stats(z)
    assert list(am) == [1, 0]                                                     # lowest index on ties
    np.testing.assert_allclose(conf, scipy.special.softmax(z, -1).max(-1), rtol=1e-14)
    D = np.array([1e-3, 1e-3, 0.9999e-3, 1.0001e-3, np.inf, np.nan, 0.0])
    masked = np.array([0, 1, 0, 0, 0, 0, 0])
    got = O.sure_test(D, masked, 1e-3)
    assert list(got) == [True, False, True, False, False, False, True]            # "<=", masked and NaN never lock


def test_active_set_definition():
    lock = np.array([[0, 1, 0, 0], [1, 1, 1, 1], [0, 0, 0, 1]], np.uint8)
    idx, offs = O.active_set(lock)
    assert list(idx) == [0, 2, 3, 8, 9, 10] and list(offs) == [0, 3, 3, 6]
    rng = np.random.default_rng(5)
    lock = (rng.random((3, 50)) < 0.6).astype(np.uint8)
    idx, offs = O.active_set(lock)
    assert list(idx) == list(np.flatnonzero(lock.reshape(-1) == 0))
    assert list(offs) == [0] + list(np.cumsum((lock == 0).sum(1)))


# ------------------------------------------------------------------ the locked forward against full recomputation
def test_no_locks_equals_dense_forward():
    c, oc, w, wn = _small()
    B, N = 2, 16
    tokens, mask = inputs.make_tokens(B, N, 8, c["vocab"], 2)
    st = O.OracleState(oc, B, N)
    r = O.step(st, wn, tokens.numpy(), mask.numpy(), np.zeros((B, N), np.uint8), 1e-3)
    assert list(r["active_idx"]) == list(range(B * N))
    for b in range(B):
        ref = DR.dense_forward(c, _w64(w), tokens[b]).numpy()
        got = r["logits"][b * N:(b + 1) * N]
        assert np.max(np.abs(got - ref)) <= 1e-11 * np.max(np.abs(ref))
    assert np.all(np.isinf(r["kl"])) and np.array_equal(r["new_lock"], np.zeros((B, N), np.uint8))  # D_1 = inf


def test_locked_forward_equals_dense_with_frozen_kv():
    c, oc, w, wn = _small(seed=5)
    B, N = 2, 14
    tokens, mask = inputs.make_tokens(B, N, 7, c["vocab"], 3)
    st = O.OracleState(oc, B, N)
    O.step(st, wn, tokens.numpy(), mask.numpy(), np.zeros((B, N), np.uint8), 0.0)
    K0, V0 = st.K.copy(), st.V.copy()
    # the sampler reveals tokens; then some rows are locked (frozen K/V stem from the OLD tokens)
    tok2 = tokens.clone()
    tok2[:, 7:10] = torch.tensor([[3, 4, 5], [9, 8, 7]], dtype=torch.int32)
    lock = inputs.random_lock(B, N, [6, 9], 7).numpy()
    r = O.step(st, wn, tok2.numpy(), mask.numpy(), lock, 0.0)
    for b in range(B):
        locked = torch.from_numpy(np.flatnonzero(lock[b]))
        ov = {l: (locked, torch.from_numpy(K0[l, b][locked]), torch.from_numpy(V0[l, b][locked]))
              for l in range(c["n_layers"])}
        ref = DR.dense_forward(c, _w64(w), tok2[b], kv_override=ov).numpy()
        act = np.flatnonzero(lock[b] == 0)
        got = r["logits"][r["row_offsets"][b]:r["row_offsets"][b + 1]]
        assert np.max(np.abs(got - ref[act])) <= 1e-11 * np.max(np.abs(ref))
        # frozen rows are bit-identical, active rows were rewritten with this step's K/V
        assert np.array_equal(st.K[:, b][:, lock[b] == 1], K0[:, b][:, lock[b] == 1])
        assert np.array_equal(st.V[:, b][:, lock[b] == 1], V0[:, b][:, lock[b] == 1])
        changed = np.flatnonzero(np.any(st.K[0, b] != K0[0, b], axis=(1, 2)))
        assert set(changed) <= set(act)
    # and the result differs from naive full recomputation (the method is an approximation, not a shortcut)
    full = DR.dense_forward(c, _w64(w), tok2[0]).numpy()
    act0 = np.flatnonzero(lock[0] == 0)
    assert np.max(np.abs(r["logits"][:len(act0)] - full[act0])) > 1e-6


def test_stationary_sequence_locks_losslessly():
    c, oc, w, wn = _small(seed=6)
    B, N = 1, 12
    tokens, mask = inputs.make_tokens(B, N, 8, c["vocab"], 4)
    st = O.OracleState(oc, B, N)
    lock = np.zeros((B, N), np.uint8)
    r1 = O.step(st, wn, tokens.numpy(), mask.numpy(), lock, 1e-3)
    assert not r1["new_lock"].any()
    r2 = O.step(st, wn, tokens.numpy(), mask.numpy(), r1["new_lock"], 1e-3)
    assert np.all(r2["kl"] == 0.0)
    np.testing.assert_array_equal(r2["logits"], r1["logits"])
    assert np.array_equal(r2["new_lock"], (mask.numpy() == 0).astype(np.uint8))   # every unmasked row locks, no masked row does
    r3 = O.step(st, wn, tokens.numpy(), mask.numpy(), r2["new_lock"], 1e-3)
    assert list(r3["active_idx"]) == list(range(8, 12))
    np.testing.assert_allclose(r3["logits"], r2["logits"][8:], rtol=1e-12, atol=1e-13)
    assert np.all(np.abs(r3["kl"]) < 1e-12)                                      # fp64 rounding order only
    assert np.all(r3["new_lock"] >= r2["new_lock"])                               # monotone


def test_rows_are_independent_given_the_cache():
    # per-row stages do not depend on which other rows are packed beside them
    c, oc, w, wn = _small(seed=8, L=1)
    rng = np.random.default_rng(4)
    N, H, dh, d = 10, c["n_heads"], c["head_dim"], c["d_model"]
    Kc, Vc = rng.normal(size=(N, H, dh)), rng.normal(size=(N, H, dh))
    x = rng.normal(size=(4, d))
    pos = np.array([1, 4, 5, 9])
    lw = wn["layers"][0]
    full = O.layer_rows(oc, lw, x, pos, Kc.copy(), Vc.copy())
    K2, V2 = Kc.copy(), Vc.copy()
    _, k, v = O.qkv_rows(oc, lw, x, pos)
    K2[pos], V2[pos] = k, v                                                       # all fresh K/V first (line 11)
    for r in (2, 0, 3, 1):
        one = O.layer_rows(oc, lw, x[r:r + 1], pos[r:r + 1], K2.copy(), V2.copy())
        np.testing.assert_allclose(one[0], full[r], rtol=1e-12, atol=1e-13)


def test_active_row_uses_original_position_for_rope():
    c, oc, w, wn = _small(seed=9, L=1)
    N = 9
    tokens, _ = inputs.make_tokens(1, N, N, c["vocab"], 5)
    _, kvs, _ = DR.dense_forward(c, _w64(w), tokens[0], return_kv=True)
    x = wn["tok_emb"][tokens[0].numpy()]
    pos = np.array([4, 7, 8])                                                     # a locked prefix does not renumber rows
    _, k, v = O.qkv_rows(oc, wn["layers"][0], x[pos], pos)
    np.testing.assert_allclose(k, kvs[0][0][pos].numpy(), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(v, kvs[0][1][pos].numpy(), rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------ brute force on a tiny case, pure-Python loops
def _brute_step(cfg, w, tokens, lock, Kc, Vc):
    """One sequence, scalar loops only (math module).  Kc/Vc: nested lists [L][N][H][dh], updated in place."""
    d, H, dh, Fd, V, L = (cfg[k] for k in ("d_model", "n_heads", "head_dim", "d_ff", "vocab", "n_layers"))
    N = len(tokens)
    act = [i for i in range(N) if not lock[i]]

    def norm(x, g):
        ms = sum(t * t for t in x) / len(x)
        return [t / math.sqrt(ms + cfg["rms_eps"]) * gg for t, gg in zip(x, g)]

    def matvec(Wm, x):
        return [sum(Wm[o][i] * x[i] for i in range(len(x))) for o in range(len(Wm))]

    def rot(vec, pos):
        out = list(vec)
        for h in range(H):
            for j in range(dh // 2):
                a = pos * cfg["rope_theta"] ** (-2.0 * j / dh)
                x0, x1 = vec[h * dh + j], vec[h * dh + j + dh // 2]
                out[h * dh + j] = x0 * math.cos(a) - x1 * math.sin(a)
                out[h * dh + j + dh // 2] = x1 * math.cos(a) + x0 * math.sin(a)
        return out

    xs = {i: [float(t) for t in w["tok_emb"][tokens[i]]] for i in act}
    for l in range(L):
        lw = w["layers"][l]
        qs = {}
        for i in act:
            h = norm(xs[i], lw["attn_norm_g"])
            qs[i] = rot(matvec(lw["wq"], h), i)
            k = rot(matvec(lw["wk"], h), i)
            v = matvec(lw["wv"], h)
            for hh in range(H):
                Kc[l][i][hh] = k[hh * dh:(hh + 1) * dh]
                Vc[l][i][hh] = v[hh * dh:(hh + 1) * dh]
        for i in act:
            o = []
            for hh in range(H):
                s = [sum(qs[i][hh * dh + t] * Kc[l][j][hh][t] for t in range(dh)) / math.sqrt(dh) for j in range(N)]
                mx = max(s)
                e = [math.exp(t - mx) for t in s]
                Z = sum(e)
                o += [sum(e[j] / Z * Vc[l][j][hh][t] for j in range(N)) for t in range(dh)]
            xs[i] = [a + b for a, b in zip(xs[i], matvec(lw["wo"], o))]
            h2 = norm(xs[i], lw["ffn_norm_g"])
            g, u = matvec(lw["w_gate"], h2), matvec(lw["w_up"], h2)
            a_ = [gg / (1 + math.exp(-gg)) * uu for gg, uu in zip(g, u)]
            xs[i] = [a + b for a, b in zip(xs[i], matvec(lw["w_down"], a_))]
    logits = {i: matvec(w["lm_head"], norm(xs[i], w["final_norm_g"])) for i in act}
    return act, logits


def test_brute_force_tiny():
    c, oc = _cfg(n_layers=1, d_model=8, n_heads=2, head_dim=4, d_ff=16, vocab=5)
    w = inputs.make_weights(c, 12, dtype=torch.float32, std=0.5)
    wn = inputs.weights_to_numpy(w)
    wl = {k: v.tolist() for k, v in wn.items() if k != "layers"}
    wl["layers"] = [{k: v.tolist() for k, v in lw.items()} for lw in wn["layers"]]
    N = 4
    tokens = np.array([[1, 3, 4, 4]], np.int32)
    mask = np.array([[0, 0, 1, 1]], np.uint8)
    st = O.OracleState(oc, 1, N)
    Kc = [[[[0.0] * 4 for _ in range(2)] for _ in range(N)]]
    Vc = [[[[0.0] * 4 for _ in range(2)] for _ in range(N)]]
    lock = np.zeros((1, N), np.uint8)
    r1 = O.step(st, wn, tokens, mask, lock, 1e-3)
    act, lg1 = _brute_step(c, wl, tokens[0].tolist(), lock[0].tolist(), Kc, Vc)
    np.testing.assert_allclose(r1["logits"], np.array([lg1[i] for i in act]), rtol=1e-11, atol=1e-13)
    # second step: token 2 revealed, position 0 locked by hand -> only rows 1..3 recomputed, K/V of 0 frozen
    tokens2 = np.array([[1, 3, 2, 4]], np.int32)
    lock2 = np.array([[1, 0, 0, 0]], np.uint8)
    r2 = O.step(st, wn, tokens2, mask, lock2, 1e-3)
    act2, lg2 = _brute_step(c, wl, tokens2[0].tolist(), lock2[0].tolist(), Kc, Vc)
    assert act2 == [1, 2, 3] and list(r2["active_idx"]) == act2
    got = np.array([lg2[i] for i in act2])
    np.testing.assert_allclose(r2["logits"], got, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(st.K[0, 0], np.array(Kc[0]), rtol=1e-12, atol=1e-14)
    # KL of step 2 against step 1 by scalar loops
    for r, i in enumerate(act2):
        def lsm(z):
            m = max(z)
            lse = m + math.log(sum(math.exp(t - m) for t in z))
            return [t - lse for t in z]
        a, b = lsm(lg2[i]), lsm(lg1[i])
        kl = sum(math.exp(x) * (x - y) for x, y in zip(a, b))
        assert abs(r2["kl"][r] - kl) < 1e-13
        assert bool(r2["new_lock"][0, i]) == (mask[0, i] == 0 and kl <= 1e-3)
    assert r2["new_lock"][0, 0] == 1


# ------------------------------------------------------------------ optional confidence gate (Algorithm 1 line 21)
def test_percentile_and_confidence_gate():
    rng = np.random.default_rng(11)
    for n in (1, 2, 5, 40, 101):
        x = rng.random(n)
        for m in (0, 10, 20, 40, 50, 99.5, 100):
            assert abs(O.percentile_linear(x, m) - np.percentile(x, m)) < 1e-15     # numpy's default (linear) rule
    assert O.percentile_linear([], 20) == -np.inf
    assert O.percentile_linear([3.0, 1.0, 2.0], 0) == 1.0 and O.percentile_linear([3.0, 1.0, 2.0], 100) == 3.0
    assert O.percentile_linear([0.0, 10.0], 25) == 2.5                              # interpolation by hand
    # gate: per sequence, over candidates only
    conf = np.array([0.9, 0.5, 0.99, 0.2, 0.7, 0.6, 0.95])
    cand = np.array([1, 1, 1, 0, 1, 1, 1], bool)
    seq = np.array([0, 0, 0, 0, 1, 1, 1])
    passes, theta = O.confidence_gate(conf, cand, seq, 3, 50)
    # sequence 0: u = .1, .5, .01 -> median .1 -> rows with u <= .1; the non-candidate (u = .8) never passes
    assert abs(theta[0] - 0.1) < 1e-15 and list(passes[:4]) == [True, False, True, False]
    # sequence 1: u = .3, .4, .05 -> median .3
    assert abs(theta[1] - 0.3) < 1e-15 and list(passes[4:]) == [True, False, True]
    assert theta[2] == -np.inf                                                      # no candidates: nothing passes
    p100, _ = O.confidence_gate(conf, cand, seq, 3, 100)
    assert list(p100) == list(cand)                                                 # m = 100 passes every candidate
    p0, _ = O.confidence_gate(conf, cand, seq, 3, 0)
    assert list(p0) == [False, False, True, False, False, False, True]              # m = 0: only the most confident


def test_step_with_confidence_gate_locks_a_subset():
    c, oc, w, wn = _small(seed=13)
    B, N = 2, 16
    tokens, mask = inputs.make_tokens(B, N, 10, c["vocab"], 6)
    lock0 = np.zeros((B, N), np.uint8)
    a, b = O.OracleState(oc, B, N), O.OracleState(oc, B, N)
    for st in (a, b):
        O.step(st, wn, tokens.numpy(), mask.numpy(), lock0, 1e-3)
    plain = O.step(a, wn, tokens.numpy(), mask.numpy(), lock0, 1e-3)                # stationary: every unmasked row locks
    gated = O.step(b, wn, tokens.numpy(), mask.numpy(), lock0, 1e-3, conf_gate_m=20)
    assert plain["new_lock"].sum() == 20
    assert np.all(gated["new_lock"] <= plain["new_lock"])                          # the gate only removes locks
    # 10 candidates per sequence, 20th percentile: h = 1.8 -> the two most confident rows pass
    assert list(gated["new_lock"].sum(1)) == [2, 2]
    for bb in range(B):
        u = 1 - gated["conf"][bb * N: bb * N + 10]
        assert set(np.flatnonzero(gated["new_lock"][bb])) == set(np.argsort(u)[:2])
    np.testing.assert_array_equal(gated["logits"], plain["logits"])                 # the gate changes decisions only


def test_update_mask_reveals_the_most_confident_masked_block_positions():
    """UpdateMASK (Algorithm 1 line 16) against a different library's routine (torch.topk on a stable ordering) and
    against the properties that define the policy: per sequence exactly min(k, masked-and-computed block positions)
    reveals, every revealed confidence >= every confidence left masked in the block, ties to the lowest position,
    nothing outside the block or already unmasked changes, the mask token is never written."""
    rng = np.random.default_rng(5)
    B, N, V = 3, 40, 11
    mask_tok = V - 1
    for trial in range(20):
        lo, hi, k = int(rng.integers(0, 20)), int(rng.integers(20, 41)), int(rng.integers(1, 6))
        tokens = rng.integers(0, V - 1, (B, N))
        mask = (rng.random((B, N)) < 0.5).astype(np.uint8)
        tokens[mask == 1] = mask_tok
        lock = (rng.random((B, N)) < 0.3) & (mask == 0)               # masked positions are never locked
        idx, _ = O.active_set(lock.astype(np.uint8))
        conf = np.round(rng.random(len(idx)), 1)                      # coarse values: many ties
        am = rng.integers(0, V, len(idx))                             # may propose the mask token
        t2, m2, rev = O.update_mask(tokens, mask, conf, am, idx, lo, hi, k, mask_tok)
        conf_pos = np.full(B * N, -1.0)
        conf_pos[idx] = conf
        am_pos = np.zeros(B * N, np.int64)
        am_pos[idx] = am
        for b in range(B):
            blk = np.arange(lo, hi)
            cand = blk[mask[b, blk] == 1]
            n_rev = min(k, len(cand))
            assert rev[b] == n_rev
            # torch.topk on (conf, -position) via a stable sort key
            key = torch.tensor(conf_pos[b * N + cand]) * 1000 - torch.tensor(cand, dtype=torch.float64) * 1e-3
            chosen = set(cand[torch.topk(key, n_rev).indices.numpy()].tolist()) if n_rev else set()
            changed = set(np.flatnonzero(m2[b] != mask[b]).tolist())
            assert changed == chosen
            for n in chosen:
                want = am_pos[b * N + n]
                assert t2[b, n] == (0 if want == mask_tok else want) and t2[b, n] != mask_tok and m2[b, n] == 0
            untouched = np.setdiff1d(np.arange(N), list(chosen))
            assert np.array_equal(t2[b, untouched], tokens[b, untouched])
            left = [n for n in cand if n not in chosen]
            if chosen and left:
                assert min(conf_pos[b * N + n] for n in chosen) >= max(conf_pos[b * N + n] for n in left)
    # worked example: block [2, 6), k = 2, confidences 0.9 (pos 2), 0.9 (pos 4), 0.95 (pos 5); position 3 is unmasked
    tokens = np.array([[7, 7, 9, 1, 9, 9, 9]])
    mask = np.array([[0, 0, 1, 0, 1, 1, 1]], np.uint8)
    idx = np.arange(7)
    conf = np.array([0.1, 0.1, 0.9, 0.99, 0.9, 0.95, 0.999])
    am = np.array([0, 0, 3, 3, 4, 9, 6])
    t2, m2, rev = O.update_mask(tokens, mask, conf, am, idx, 2, 6, 2, 9)
    assert t2.tolist() == [[7, 7, 3, 1, 9, 0, 9]] and m2.tolist() == [[0, 0, 0, 0, 1, 0, 1]] and rev.tolist() == [2]


def test_kl_is_stepwise_a_returning_row_starts_over():
    """Algorithm 1 line 19: D_t = KL(p_t || p_{t-1}) if t > 1 else inf.  Pinned by hand on a tiny model: the rows of a
    second step have D equal to the KL between the two steps' softmaxes (scipy), and a row that sat out one step has
    D = inf in the step in which it returns, whatever posterior it had before."""
    c, oc, w, wn = _small(seed=8)
    B, N = 1, 10
    tokens, mask = inputs.make_tokens(B, N, 4, c["vocab"], 8)
    st = O.OracleState(oc, B, N)
    lock = np.zeros((B, N), np.uint8)
    r1 = O.step(st, wn, tokens.numpy(), mask.numpy(), lock, 1e-3)
    assert np.isinf(r1["kl"]).all()
    tok2 = tokens.numpy().copy()
    tok2[0, 5] = 3
    m2 = mask.numpy().copy()
    m2[0, 5] = 0
    lock2 = lock.copy()
    lock2[0, 2] = 1                                                   # position 2 sits this step out
    r2 = O.step(st, wn, tok2, m2, lock2, 0.0)
    p1 = scipy.special.softmax(r1["logits"], axis=1)
    p2 = scipy.special.softmax(r2["logits"], axis=1)
    rows1 = r2["active_idx"]                                          # step-1 rows were all positions in order
    want = np.array([scipy.special.rel_entr(p2[i], p1[pos]).sum() for i, pos in enumerate(rows1)])
    np.testing.assert_allclose(r2["kl"], want, rtol=1e-9, atol=1e-15)
    r3 = O.step(st, wn, tok2, m2, lock, 1e-3)                         # position 2 is back
    back = int(np.flatnonzero(r3["active_idx"] == 2)[0])
    assert np.isinf(r3["kl"][back]) and np.isfinite(np.delete(r3["kl"], back)).all()
    assert r3["new_lock"][0, 2] == 0
