"""Parity at the sizes of the benchmark configurations that the other GPU tests only reach scaled down:

  * long context (batch 4, N = 4096, LLaDA-8B layer shape, full vocabulary) with every row active, half of them
    and 5 % of them: dense attention over 32 key blocks, the CTA-pair GEMM path, 16384 logit rows;
  * the tensor-core attention alone at N = 4096, all 32 heads, 1024 ... 4096 active rows per sequence;
  * the single-sequence stack (32 layers, batch 1, N = 512) driven by the semi-autoregressive sampler loop;
  * the sure-test kernel alone at 820 and 4096 rows x vocabulary 126464 (the grid wraps many times);
  * the selection hybrid of Experiment 5 (sampler.run(select_fraction=0.8)) against the oracle, decision by decision.

At these sizes the oracle computes seeded samples of rows one by one (every 128-row tile of every sampled sequence is
hit), everything integer is compared in full.
"""
import numpy as np
import pytest
import torch

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import binding as SL
from paper_2602_06412_b200 import inputs, sampler
from tests.parity_util import f64, rel_err_rows, to_dev
from tests.test_gpu_teacher_forced import _check_step, _two_steps, tile_covering_sample

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("ratio", [1.0, 0.5, 0.05])
def test_long_context_full_vocab(ratio):
    """Batch 4, N = 4096 (prompt 3584 + 512 to generate), two LLaDA-8B-shaped layers, vocabulary 126464, under the
    contiguous-prefix-plus-random lock pattern at M/N = 1, 0.5 and 0.05 (ragged per sequence).  The first step computes
    all 16384 rows (dense attention, two-tile items), the second the locked pattern."""
    cfg = inputs.model_shape("llada8b", n_layers=2)
    B, N = 4, 4096
    na = [min(N, int(N * ratio * f)) for f in (1.0, 1.2, 0.8, 1.0)] if ratio < 1.0 else [N] * B
    w0, w1 = _two_steps(cfg, B=B, N=N, n_prompt=3584, n_active=na, seed=61, layers=[0, 1], seqs=[1, 2], n_rows=16,
                        w_device=DEV, lock_fn=inputs.contiguous_plus_random_lock)
    print("worst stage errors, long context, full vocabulary, ratio", ratio, w0, w1)


@pytest.mark.parametrize("n_act", [[4096, 1024], [2048, 4096, 1500, 4096]])
def test_attention_tensor_cores_long_context(n_act):
    """tcgen05 attention at N = 4096 with all 32 heads of the LLaDA-8B shape (a head's keys and values of one
    sequence are 2 MB, a sequence's 67 MB): 1024 ... 4096 active rows per sequence.  The oracle computes sampled query
    rows of every 128-row tile, for every head."""
    B, N, H, dh = len(n_act), 4096, 32, 128
    lock = inputs.contiguous_plus_random_lock(B, N, n_act, 13)
    idx, offs = O.active_set(lock.numpy())
    M = len(idx)
    g = torch.Generator(device=DEV).manual_seed(N + B)
    q = (torch.randn((B * N, H, dh), generator=g, device=DEV) * 2.0).to(torch.bfloat16)
    Kc = torch.randn((B * N, H, dh), generator=g, device=DEV).to(torch.bfloat16)
    Vc = torch.randn((B * N, H, dh), generator=g, device=DEV).to(torch.bfloat16)
    o = torch.full((B * N, H, dh), 5.0, dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    SL.surelock_attention(q, Kc, Vc, torch.from_numpy(idx).to(DEV), torch.from_numpy(offs).to(DEV),
                          torch.tensor([M], dtype=torch.int32, device=DEV), B, N, o, impl=0, dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    rng = np.random.default_rng(5)
    worst = 0.0
    for b in range(B):
        r0, r1 = int(offs[b]), int(offs[b + 1])
        S = tile_covering_sample(r0, r1, 48, rng)
        rows = torch.from_numpy(r0 + S).to(DEV)
        ref = O.attention_rows(f64(q[rows]), f64(Kc[b * N:(b + 1) * N]), f64(Vc[b * N:(b + 1) * N]))
        worst = max(worst, rel_err_rows(f64(o[rows]).reshape(len(S), -1), ref))
    assert worst < 2e-2, worst
    assert (o[M:] == 5.0).all()                                      # rows beyond M untouched


def test_single_sequence_stack_under_the_semi_autoregressive_sampler():
    """The whole 32-layer LLaDA-8B-shaped stack, batch 1, prompt 256 + 256 to generate, decoded by sampler.run
    (blocks of 32, one reveal per step, KL eps 1e-3).  The oracle checks steps stage by stage from the GPU's traced
    inputs: layers 0, 15 and 31, rows of every tile, logits, KL on the GPU's logits of two consecutive steps, lock
    decisions, and the active list bit for bit.  With random weights nothing locks by itself in the first steps, so
    after the third step a forced seeded pattern locks everything except the current block and a few prompt rows (as
    a caller may: those rows' K/V are in the cache): the later steps run in the weight-streaming regime (M ~ 50)."""
    cfg = inputs.model_shape("llada8b")
    B, N, n_prompt, blk, steps = 1, 512, 256, 32, 10
    w_dev = inputs.make_weights(cfg, 71, dtype=torch.bfloat16, device=DEV)
    ctx = SL.surelock_init(cfg, w_dev, N, B)
    SL.surelock_set_option(ctx, "trace_layers", 1)
    SL.surelock_set_option(ctx, "strict_tc", 1)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 71)
    tokens, mask = tokens.to(DEV), mask.to(DEV)
    seen = dict(M=[], prev_logits=None, prev_rop=None, worst=[])
    checked = (0, 1, 2, 6, 7, 8, 9)

    def observer(t, out, lock_in, lock_out, tok, msk):
        assert SL.surelock_status_poll(ctx) == 0
        M = out.M()
        seen["M"].append(M)
        if t in checked:
            w = _check_step(cfg, w_dev, ctx, out, lock_in.cpu(), msk.cpu(), 1e-3, seen["prev_logits"], seen["prev_rop"],
                            [0, 15, 31], [0], 16, 100 + t, lock_out, tokens=tok)
            seen["worst"].append(w)
        seen["prev_logits"] = out.logits[:M].clone()          # what the next step will read as "previous"
        rop = np.full(B * N, -1, np.int64)
        rop[out.active_idx[:M].cpu().numpy()] = np.arange(M)
        seen["prev_rop"] = rop
        if t == 2:                                            # forced pattern: keep the first block and 20 prompt rows
            forced = torch.ones((B, N), dtype=torch.uint8)
            forced[0, n_prompt:n_prompt + blk] = 0
            forced[0, torch.randperm(n_prompt, generator=torch.Generator().manual_seed(5))[:20]] = 0
            lock_out |= forced.to(DEV)

    res = sampler.run(ctx, tokens, mask, n_prompt, blk, steps=steps, kl_eps=1e-3, observer=observer)
    assert SL.surelock_status_poll(ctx) == 0 and SL.surelock_last_fallback_count(ctx) == 0
    print("single-sequence sampler: M trace", res["M_trace"], "worst stage errors", seen["worst"])
    assert res["M_trace"] == seen["M"] and res["M_trace"][:3] == [N, N, N] and res["M_trace"][3] == blk + 20
    assert all(a >= b for a, b in zip(res["M_trace"], res["M_trace"][1:]))
    assert res["unmasked_per_step"] == [1] * steps


@pytest.mark.parametrize("rows", [820, 4096])
def test_softmax_kl_sure_alone_many_rows(rows):
    """The sure-test kernel alone at vocabulary 126464 with more rows than the grid holds at once (820 = 5 % of the
    long-context batch, 4096).  Inputs as in the small case (KL spanning the paper's thresholds 5e-8 ... 5e-2, identical
    and peaked rows); the oracle checks a seeded sample of 96 rows spread over the whole range, the other rows are held
    to the properties that need no oracle (identical rows exactly 0, KL finite and >= 0, masked rows never lock)."""
    V, eps = 126464, 1e-3
    cur, prev, mask = inputs.kl_logit_pairs(rows, V, 17, dtype=torch.bfloat16, device=DEV)
    rop = torch.arange(rows, dtype=torch.int32, device=DEV)
    pos = torch.arange(rows, dtype=torch.int32, device=DEV)
    kl = torch.empty(rows, dtype=torch.float32, device=DEV)
    conf, lse = torch.empty_like(kl), torch.empty_like(kl)
    am = torch.empty(rows, dtype=torch.int32, device=DEV)
    lock = torch.zeros(rows, dtype=torch.uint8, device=DEV)
    n = torch.tensor([rows], dtype=torch.int32, device=DEV)
    SL.surelock_softmax_kl_sure(cur, prev, rop, None, pos, n, mask, lock, eps, kl, conf, am, lse)
    torch.cuda.synchronize()
    rng = np.random.default_rng(rows)
    S = np.unique(np.concatenate([np.linspace(0, rows - 1, 48).astype(np.int64), rng.integers(0, rows, 48), [7, 27]]))
    St = torch.from_numpy(S).to(DEV)
    z, y = f64(cur[St]), f64(prev[St])
    ref_kl = O.kl_from_logits(z, y)
    ref_conf, ref_am = O.posterior_stats(z)
    got = kl[St].cpu().numpy().astype(np.float64)
    err = np.abs(got - ref_kl)
    assert np.all(err <= 1e-3 * ref_kl + 1e-9), err.max()
    assert ref_kl[ref_kl > 0].min() < 1e-5 and ref_kl.max() > 1e-2               # the sample spans the threshold range
    assert np.array_equal(am[St].cpu().numpy(), ref_am)
    np.testing.assert_allclose(conf[St].cpu().numpy(), ref_conf, rtol=2e-5)
    m_np = mask.cpu().numpy()
    want = O.sure_test(ref_kl, m_np[S], eps)
    near = np.abs(ref_kl - eps) <= 1e-3 * eps
    lk = lock.cpu().numpy().astype(bool)
    assert np.array_equal(lk[S][~near], want[~near])
    kl_all = kl.cpu().numpy()
    assert np.isfinite(kl_all).all() and (kl_all >= 0).all()
    same = (np.arange(rows) % 20) == 7
    assert np.all(kl_all[same] == 0.0) and np.all(lk[same] == (m_np[same] == 0))  # identical posteriors: D = 0 locks
    assert not lk[m_np == 1].any()
    assert np.array_equal(lk, (kl_all <= np.float32(eps)) & (m_np == 0))                       # the decision is the test on the kernel's own D


@pytest.mark.parametrize("surelock", [True, False])
def test_selection_hybrid_against_the_oracle(surelock):
    """Experiment 5 on the tiny fp32 model, 64 steps: sampler.run with the selection surrogate at k = 0.8 (with
    SureLock: the combination; without: selection alone) beside the oracle driven by the same seeded scores.  Skip
    masks, active lists, M trace, lock masks, revealed tokens and mask states must agree exactly at every step."""
    cfg = inputs.model_shape("tiny")
    oc = O.ModelCfg(**cfg)
    B, N, n_prompt, blk, steps, k, eps, seed = 2, 128, 64, 32, 64, 0.8, 1e-3, 4
    w = inputs.make_weights(cfg, 9, dtype=torch.float32)
    wn = inputs.weights_to_numpy(w)
    ctx = SL.surelock_init(cfg, to_dev(w), N, B)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 9)
    tok_o, mask_o = tokens.numpy().copy(), mask.numpy().copy()
    st = O.OracleState(oc, B, N, prev_policy="previous_step")        # the reading the library serves
    lock_o = np.zeros((B, N), np.uint8)
    mask_tok = cfg["vocab"] - 1
    log = []

    def observer(t, out, lock_in, lock_out, tok, msk):
        nonlocal lock_o, tok_o, mask_o
        skip = O.selection_skip(lock_o, mask_o, inputs.selection_scores(B, N, t, seed).numpy(), k)
        r = O.step(st, wn, tok_o, mask_o, lock_o, eps, skip=skip)
        M = out.M()
        assert np.array_equal(lock_in.cpu().numpy(), lock_o | skip), t             # same rows skipped, same rows locked
        assert M == len(r["active_idx"]) and np.array_equal(out.active_idx[:M].cpu().numpy(), r["active_idx"]), t
        assert np.array_equal(tok.cpu().numpy(), tok_o) and np.array_equal(msk.cpu().numpy(), mask_o), t
        kl_g, kl_r = out.kl[:M].cpu().numpy().astype(np.float64), r["kl"]
        fin = np.isfinite(kl_r)
        assert np.array_equal(np.isfinite(kl_g), fin), t                           # a returning row starts over: D = inf
        assert np.all(np.abs(kl_g[fin] - kl_r[fin]) <= 1e-3 * kl_r[fin] + 1e-9), t
        assert rel_err_rows(f64(out.logits[:M]), r["logits"]) < 1e-4, t
        assert np.array_equal(lock_out.cpu().numpy(), r["new_lock"]), t            # lock decisions
        log.append(M)
        lock_o = r["new_lock"] if surelock else np.zeros((B, N), np.uint8)
        blk_i = min(t // blk, (N - n_prompt + blk - 1) // blk - 1)
        lo = n_prompt + blk_i * blk
        tok_o, mask_o, _ = O.update_mask(tok_o, mask_o, r["conf"], r["argmax"], r["active_idx"], lo, min(lo + blk, N), 1,
                                         mask_tok)

    res = sampler.run(ctx, tokens.to(DEV), mask.to(DEV), n_prompt, blk, steps=steps, kl_eps=eps, surelock=surelock,
                      select_fraction=k, select_seed=seed, observer=observer)
    assert SL.surelock_status_poll(ctx) == 0
    assert res["M_trace"] == log and res["masked_at_end"] == 0
    assert mask_o.sum() == 0
    if surelock:
        assert res["locked_at_end"] == int(lock_o.sum()) > 0
