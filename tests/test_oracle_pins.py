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


def test_keep_last_policy_compares_a_returning_row_with_its_last_posterior():
    """The other reading of p_{t-1} for a row that sat out a step (Sec. 2.1: a locked row keeps p_{t*}): with
    prev_policy="keep_last" the returning row's D is the KL between its new posterior and the one it had two steps
    ago, by hand with scipy; every row that never sat out gets the same D under both policies."""
    c, oc, w, wn = _small(seed=8)
    B, N = 1, 10
    tokens, mask = inputs.make_tokens(B, N, 4, c["vocab"], 8)
    tok2 = tokens.numpy().copy()
    tok2[0, 5] = 3
    m2 = mask.numpy().copy()
    m2[0, 5] = 0
    lock0 = np.zeros((B, N), np.uint8)
    lock2 = lock0.copy()
    lock2[0, 2] = 1
    out = {}
    for pol in ("previous_step", "keep_last"):
        st = O.OracleState(oc, B, N, prev_policy=pol)
        r1 = O.step(st, wn, tokens.numpy(), mask.numpy(), lock0, 1e-3)
        O.step(st, wn, tok2, m2, lock2, 0.0)
        out[pol] = (r1, O.step(st, wn, tok2, m2, lock0, 1e-3))
    r1, r3 = out["keep_last"]
    p1 = scipy.special.softmax(r1["logits"][2])
    p3 = scipy.special.softmax(r3["logits"][2])
    np.testing.assert_allclose(r3["kl"][2], scipy.special.rel_entr(p3, p1).sum(), rtol=1e-9)
    assert np.isinf(out["previous_step"][1]["kl"][2])
    others = np.arange(N) != 2
    np.testing.assert_array_equal(r3["kl"][others], out["previous_step"][1]["kl"][others])
    np.testing.assert_array_equal(r3["logits"], out["previous_step"][1]["logits"])   # the forward itself is the same
    with pytest.raises(ValueError):
        O.OracleState(oc, B, N, prev_policy="something else")


def test_literal_algorithm_order_lets_a_position_lock_in_the_step_that_reveals_it():
    """Algorithm 1 line 16 (UpdateMASK) stands before line 20 (candidates = active and unmasked).  Read literally, a
    position revealed in step t is a candidate in step t.  On a stationary sequence (D = 0 for every row in step 2):
    the default reading locks exactly the rows that were fed as tokens; the literal order also locks the position
    that step 2 reveals, and its cached K/V are then those of the MASK token it was fed as."""
    c, oc, w, wn = _small(seed=6)
    B, N = 1, 12
    tokens, mask = inputs.make_tokens(B, N, 8, c["vocab"], 4)
    tk, mk = tokens.numpy(), mask.numpy()
    mask_tok = c["vocab"] - 1
    calls = []

    def reveal_position_9(tok, msk, conf, am, idx):
        calls.append((conf.copy(), am.copy(), idx.copy()))
        tok, msk = tok.copy(), msk.copy()
        tok[0, 9], msk[0, 9] = 5, 0
        return tok, msk

    res = {}
    for name, fn in (("default", None), ("literal", reveal_position_9)):
        st = O.OracleState(oc, B, N)
        O.step(st, wn, tk, mk, np.zeros((B, N), np.uint8), 1e-3)
        res[name] = (O.step(st, wn, tk, mk, np.zeros((B, N), np.uint8), 1e-3, unmask=fn), st)
    rd, rl = res["default"][0], res["literal"][0]
    assert np.all(rd["kl"] == 0.0) and np.all(rl["kl"] == 0.0)
    assert rd["new_lock"].tolist() == [[1] * 8 + [0] * 4]
    assert rl["new_lock"].tolist() == [[1] * 8 + [0, 1, 0, 0]]
    assert rl["tokens"][0, 9] == 5 and rl["mask_state"][0, 9] == 0 and rd["mask_state"][0, 9] == 1
    assert len(calls) == 1 and list(calls[0][2]) == list(range(N))
    np.testing.assert_array_equal(calls[0][0], rl["conf"])                        # line 16 sees this step's posteriors
    # the forward ran before the reveal: the K/V that position 9 is locked with are those of the mask token
    st = res["literal"][1]
    assert tk[0, 9] == mask_tok
    x = np.asarray(wn["tok_emb"], np.float64)[[mask_tok]]
    _, k, v = O.qkv_rows(oc, wn["layers"][0], x, np.array([9]))
    np.testing.assert_allclose(st.K[0, 0, 9], k[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(st.V[0, 0, 9], v[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(rd["logits"], rl["logits"])


def test_selection_skip_rows_are_not_computed_and_cannot_lock():
    """Experiment 5's selection surrogate as a skip mask: a skipped unlocked position is not in the active set, keeps
    its K/V and its lock bit, gets no posterior; the step equals a step in which those positions are locked, and the
    lock update touches computed rows only.  With the previous-step reading a skipped row has D = inf when it returns,
    with keep-last it compares with its older posterior."""
    c, oc, w, wn = _small(seed=9)
    B, N = 2, 10
    tokens, mask = inputs.make_tokens(B, N, 6, c["vocab"], 9)
    tk, mk = tokens.numpy(), mask.numpy()
    lock = np.zeros((B, N), np.uint8)
    lock[0, 1] = 1
    skip = np.zeros((B, N), np.uint8)
    skip[0, 3] = skip[1, 0] = skip[1, 4] = 1
    a = O.OracleState(oc, B, N)
    b = O.OracleState(oc, B, N)
    for st in (a, b):
        O.step(st, wn, tk, mk, np.zeros((B, N), np.uint8), 1e-3)
    K0 = a.K.copy()
    ra = O.step(a, wn, tk, mk, lock, 1e-3, skip=skip)
    rb = O.step(b, wn, tk, mk, lock | skip, 1e-3)
    want_idx = [i for i in range(B * N) if i not in (1, 3, 10, 14)]
    assert list(ra["active_idx"]) == want_idx and ra["row_offsets"].tolist() == [0, 8, 16]
    np.testing.assert_array_equal(ra["logits"], rb["logits"])
    np.testing.assert_array_equal(a.K[:, 0, 3], K0[:, 0, 3])                      # a skipped row's K/V stay
    # stationary tokens: D = 0 for every computed row, so every computed unmasked row locks; skipped ones do not
    want_lock = ((mk == 0) & (skip == 0)).astype(np.uint8) | lock
    assert np.array_equal(ra["new_lock"], want_lock)
    assert ra["new_lock"][0, 3] == 0 and ra["new_lock"][1, 0] == 0 and ra["new_lock"][1, 4] == 0
    assert np.array_equal(rb["new_lock"], want_lock | skip)                       # the locked-instead run keeps skip bits
    r3 = O.step(a, wn, tk, mk, ra["new_lock"], 1e-3)                              # the skipped rows return
    back = [int(np.flatnonzero(r3["active_idx"] == p)[0]) for p in (3, 10, 14)]
    assert np.isinf(r3["kl"][back]).all() and not r3["new_lock"][0, 3]
    kl = O.OracleState(oc, B, N, prev_policy="keep_last")
    O.step(kl, wn, tk, mk, np.zeros((B, N), np.uint8), 1e-3)
    r2k = O.step(kl, wn, tk, mk, lock, 1e-3, skip=skip)
    r3k = O.step(kl, wn, tk, mk, r2k["new_lock"], 1e-3)
    assert np.all(np.abs(r3k["kl"][back]) < 1e-12) and r3k["new_lock"][0, 3] == 1


# ------------------------------------------------------------------ optional un-locking (App. "Optional Unlocking")
def test_unlock_rule_truth_table():
    """The printed rule: u~ > theta AND D~ > eps_unlock AND t - t* > D_interval; strict inequalities."""
    p = O.UnlockParams(period=4, eps_unlock=0.01, d_interval=3, d_cool=2, rho=0.5, m=20.0)
    u = np.array([0.5, 0.5, 0.5, 0.5, 0.2, 0.5, 0.5, 0.3])
    D = np.array([0.02, 0.02, 0.02, 0.01, 0.02, 0.005, 0.02, 0.02])
    t_star = np.array([1, 5, 4, 1, 1, 1, 2, 1])
    theta = np.full(8, 0.3)
    fire = O.unlock_test(u, D, theta, 8, t_star, p)
    #      all hold | 8-5=3 not >3 | 8-4=4 | D == eps | u < theta | D < eps | fine | u == theta
    assert fire.tolist() == [True, False, True, False, False, False, True, False]
    assert not O.unlock_test(u, D, np.full(8, np.inf), 8, t_star, p).any()        # no reference uncertainty: nothing


def test_active_uncertainty_threshold_is_numpy_percentile_per_sequence():
    rng = np.random.default_rng(3)
    N, B = 9, 3
    idx = np.array([0, 2, 3, 7, 8, 18, 19, 20, 21, 22, 23, 24])                   # sequence 1 has no active row
    conf = rng.random(len(idx))
    th = O.active_uncertainty_threshold(conf, idx, B, N, 20.0)
    assert th[1] == np.inf
    np.testing.assert_allclose(th[0], np.percentile(1 - conf[:5], 20.0), rtol=1e-12)
    np.testing.assert_allclose(th[2], np.percentile(1 - conf[5:], 20.0), rtol=1e-12)


def test_probe_is_a_dense_forward_over_the_cached_keys_and_changes_nothing():
    """probe_rows: the locked rows as queries against the caches as they stand.  Pinned against the independent dense
    torch forward in which the K/V of EVERY position are overridden by the cache contents (so each probed row's result
    is what that forward gives at its position), and by stationarity: if nothing changed since the rows locked, the
    probe reproduces their frozen posterior and the drift is 0."""
    c, oc, w, wn = _small(seed=11)
    B, N, V = 2, 12, c["vocab"]
    tokens, mask = inputs.make_tokens(B, N, 7, V, 5)
    tk, mk = tokens.numpy(), mask.numpy()
    st = O.OracleState(oc, B, N)
    us = O.UnlockState(B, N, V)
    zero = np.zeros((B, N), np.uint8)
    O.step(st, wn, tk, mk, zero, 1e-3)
    r2 = O.step(st, wn, tk, mk, zero, 1e-3)                                       # stationary: unmasked rows lock
    O.record_locks(us, 2, zero, r2, N)
    lock = r2["new_lock"]
    assert lock.sum() == 14 and np.all(us.t_star[lock == 1] == 2) and np.all(us.t_star[lock == 0] == -1)
    K0, V0 = st.K.copy(), st.V.copy()
    idx, logits, logp, conf = O.probe_rows(st, wn, tk, lock)
    assert np.array_equal(st.K, K0) and np.array_equal(st.V, V0)                  # line 11 is not executed
    assert list(idx) == [b * N + i for b in range(B) for i in range(7)]
    bb, ii = idx // N, idx % N
    np.testing.assert_allclose(logp, us.frozen_logp[bb, ii], rtol=0, atol=1e-11)
    assert np.all(np.abs(O.kl_rows(logp, us.frozen_logp[bb, ii])) < 1e-12)
    # a context shift: the sampler reveals tokens, one more step rewrites the active rows' K/V
    tk2, mk2 = tk.copy(), mk.copy()
    tk2[:, 7:10] = [[3, 4, 5], [9, 8, 7]]
    mk2[:, 7:10] = 0
    O.step(st, wn, tk2, mk2, lock, 1e-3)
    idx, logits, logp, conf = O.probe_rows(st, wn, tk2, lock)
    for b in range(B):
        allpos = torch.arange(N)
        ov = {l: (allpos, torch.from_numpy(st.K[l, b]), torch.from_numpy(st.V[l, b])) for l in range(c["n_layers"])}
        ref = DR.dense_forward(c, _w64(w), torch.from_numpy(tk2[b]), kv_override=ov).numpy()
        got = logits[idx // N == b]
        assert np.max(np.abs(got - ref[:7])) <= 1e-11 * np.max(np.abs(ref))
    drift = O.kl_rows(logp, us.frozen_logp[bb, ii])
    want = DR.kl_torch(torch.from_numpy(logits), torch.from_numpy(us.frozen_logp[bb, ii])).numpy()
    np.testing.assert_allclose(drift, want, rtol=1e-9, atol=1e-15)
    assert np.all(drift > 1e-9)                                                   # the frozen posteriors are stale now


def test_unlock_cycle_by_hand_cool_down_and_stricter_relock():
    """One position through the whole cycle on a tiny model, every decision checked by hand: it locks, the context
    shifts, the probe un-locks it only once all three conditions hold (the interval is the last to be met), it is
    active again from the next step and its K/V are rewritten then, it cannot lock during the cool-down, and
    afterwards only under rho * eps."""
    c, oc, w, wn = _small(seed=11)
    B, N, V = 1, 12, c["vocab"]
    tokens, mask = inputs.make_tokens(B, N, 7, V, 5)
    tk, mk = tokens.numpy(), mask.numpy()
    st = O.OracleState(oc, B, N)
    us = O.UnlockState(B, N, V)
    eps = 1e-3
    P = O.UnlockParams(period=1, eps_unlock=1e-9, d_interval=2, d_cool=2, rho=1e-30, m=0.0)
    zero = np.zeros((B, N), np.uint8)
    O.step(st, wn, tk, mk, zero, eps)                                             # t = 1
    r = O.step(st, wn, tk, mk, zero, eps)                                         # t = 2: rows 0..6 lock (stationary)
    O.record_locks(us, 2, zero, r, N)
    lock = r["new_lock"]
    pr = O.probe_unlock(st, us, wn, tk, lock, 2, r["conf"], r["active_idx"], P)
    assert not pr["unlocked"].any() and np.array_equal(pr["new_lock"], lock)      # no drift, and t - t* = 0
    tk2, mk2 = tk.copy(), mk.copy()
    tk2[0, 7:10] = [3, 4, 5]
    mk2[0, 7:10] = 0
    for t in (3, 4):                                                              # drift is there, the interval is not met
        before = lock.copy()
        e_rows, may = O.relock_thresholds(us, eps, P.rho, t)
        r = O.step(st, wn, tk2, mk2, lock, eps, kl_eps_rows=e_rows, may_lock=may)
        O.record_locks(us, t, before, r, N)
        lock = r["new_lock"]
        pr = O.probe_unlock(st, us, wn, tk2, lock, t, r["conf"], r["active_idx"], P)
        early = us.t_star[0, pr["locked_idx"]] == 2
        assert np.all(pr["drift"][early] > P.eps_unlock)
        assert not pr["unlocked"].any(), t                                         # 3 - 2 and 4 - 2 are not > 2
        lock = pr["new_lock"]
    # t = 5: theta = min uncertainty of the active rows (m = 0); un-lock exactly the early rows above it
    before = lock.copy()
    e_rows, may = O.relock_thresholds(us, eps, P.rho, 5)
    r = O.step(st, wn, tk2, mk2, lock, eps, kl_eps_rows=e_rows, may_lock=may)
    O.record_locks(us, 5, before, r, N)
    lock = r["new_lock"]
    pr = O.probe_unlock(st, us, wn, tk2, lock, 5, r["conf"], r["active_idx"], P)
    li = pr["locked_idx"]
    want = (pr["u"] > pr["theta"][0]) & (pr["drift"] > P.eps_unlock) & (5 - us.t_star[0, li] > 2)
    assert np.array_equal(pr["unlocked"], want) and want.any()
    assert np.all(us.t_star[0, li[want]] == 2)                                    # only rows locked long enough ago
    freed = li[want]
    assert np.all(pr["new_lock"][0, freed] == 0) and np.all(us.cool_until[0, freed] == 7) and us.relock[0, freed].all()
    lock = pr["new_lock"]
    K_before = st.K[1, 0, freed].copy()            # second block: its keys depend on the context (the first block's do not)
    # t = 6, 7: active again (K/V rewritten with the current context), cannot lock (cool-down); D = inf at t = 6 anyway
    for t in (6, 7):
        e_rows, may = O.relock_thresholds(us, eps, P.rho, t)
        assert not may[0, freed].any() and np.all(e_rows[0, freed] == eps * P.rho)
        r = O.step(st, wn, tk2, mk2, lock, eps, kl_eps_rows=e_rows, may_lock=may)
        assert set(freed) <= set(r["active_idx"])
        assert not r["new_lock"][0, freed].any(), t
        lock = r["new_lock"]
    assert np.all(np.any(st.K[1, 0, freed] != K_before, axis=(1, 2)))
    # t = 8: cool-down over, but the threshold is rho * eps: D = 0 (stationary again) passes, a tiny positive D would not
    e_rows, may = O.relock_thresholds(us, eps, P.rho, 8)
    assert may[0, freed].all()
    r = O.step(st, wn, tk2, mk2, lock, eps, kl_eps_rows=e_rows, may_lock=may)
    rows = [int(np.flatnonzero(r["active_idx"] == p)[0]) for p in freed]
    assert np.all(r["kl"][rows] <= 1e-12)
    exact0 = r["kl"][rows] <= e_rows[0, freed]
    assert np.array_equal(r["new_lock"][0, freed].astype(bool), exact0)
    assert np.array_equal(O.sure_test(np.array([1e-31, 1e-4]), np.zeros(2), np.array([1e-33, 1e-3])), [False, True])


def test_selection_skip_rule_by_hand():
    """The selection surrogate's rule on a hand case: floor(0.2 * unlocked) eligible positions with the lowest scores,
    never a locked or a masked one, ties to the lower position, capped by the number of eligible positions."""
    lock = np.array([[0, 0, 1, 0, 0, 0, 0, 0, 0, 0, 0], [0, 0, 0, 0, 0, 1, 1, 1, 1, 1, 1]], np.uint8)
    mask = np.array([[0, 0, 0, 1, 0, 0, 0, 0, 0, 0, 0], [1, 1, 1, 1, 0, 0, 0, 0, 0, 0, 0]], np.uint8)
    sc = np.array([[.5, .1, .0, .0, .3, .1, .9, .8, .7, .6, .4], [.1, .2, .3, .4, .9, .0, .0, .0, .0, .0, .0]], np.float32)
    skip = O.selection_skip(lock, mask, sc, 0.8)
    # sequence 0: 10 unlocked -> 2 skipped: scores .1 at positions 1 and 5 (position 2 is locked, 3 masked)
    # sequence 1: 5 unlocked -> 1 skipped: the only eligible position is 4
    assert skip.tolist() == [[0, 1, 0, 0, 0, 1, 0, 0, 0, 0, 0], [0, 0, 0, 0, 1, 0, 0, 0, 0, 0, 0]]
    assert O.selection_skip(lock, mask, sc, 1.0).sum() == 0
    mask[1, 4] = 1
    assert O.selection_skip(lock, mask, sc, 0.5)[1].sum() == 0        # nothing eligible
    # sequence 0 at k = 0.5: 5 of the eligible scores .5 .1 .3 .1 .9 .8 .7 .6 .4 -> .1 .1 .3 .4 .5
    assert O.selection_skip(lock, mask, sc, 0.5)[0].tolist() == [1, 1, 0, 0, 1, 1, 0, 0, 0, 0, 1]
