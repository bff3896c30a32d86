"""The decoding harness: the on-device unmasking policy against the oracle and, on the GPU, the sampler loop with and
without SureLock (trace invariants and the paper's run metrics)."""
import numpy as np
import pytest
import torch

from paper_2602_06412_b200 import inputs, sampler


@pytest.mark.gpu
@pytest.mark.parametrize("B,N,lo,hi,k", [(4, 40, 16, 32, 1), (4, 40, 16, 32, 3), (3, 700, 0, 700, 5), (2, 1536, 512, 576, 64),
                                         (1, 64, 10, 10, 2), (5, 33, 0, 33, 0)])
def test_update_mask_kernel_matches_the_oracle(B, N, lo, hi, k):
    """surelock_update_mask (Algorithm 1 line 16) against the oracle, bit-exact: ragged active sets, ties in the
    confidence (coarse values), a sequence whose block is already revealed, a fully masked block, argmax equal to the
    mask token, an empty block, k = 0, more reveals asked for than masked positions."""
    from oracle import surelock_oracle as O
    from paper_2602_06412_b200 import binding as SL
    rng = np.random.default_rng(B * 1000 + N + k)
    V = 50
    mask_tok = V - 1
    tokens = rng.integers(0, V - 1, (B, N)).astype(np.int32)
    mask = (rng.random((B, N)) < 0.5).astype(np.uint8)
    if hi > lo:
        mask[min(1, B - 1), lo:hi] = 0
        mask[B - 1, lo:hi] = 1
    tokens[mask == 1] = mask_tok
    lock = ((rng.random((B, N)) < 0.4) & (mask == 0)).astype(np.uint8)
    idx, offs = O.active_set(lock)
    conf = np.round(rng.random(len(idx)), 1).astype(np.float32)
    am = rng.integers(0, V, len(idx)).astype(np.int32)
    t_ref, m_ref, rev_ref = O.update_mask(tokens, mask, conf, am, idx, lo, hi, k, mask_tok)
    dev = "cuda"
    t_d, m_d = torch.from_numpy(tokens).to(dev), torch.from_numpy(mask).to(dev)
    rev = torch.full((B,), -1, dtype=torch.int32, device=dev)
    SL.surelock_update_mask(torch.from_numpy(conf).to(dev), torch.from_numpy(am).to(dev),
                            torch.from_numpy(idx.astype(np.int32)).to(dev), torch.from_numpy(offs.astype(np.int32)).to(dev),
                            B, N, lo, hi, k, mask_tok, t_d, m_d, rev)
    torch.cuda.synchronize()
    assert np.array_equal(t_d.cpu().numpy(), t_ref) and np.array_equal(m_d.cpu().numpy(), m_ref)
    assert np.array_equal(rev.cpu().numpy(), rev_ref)


def test_flop_accounting_matches_section_2_3_formula():
    cfg = inputs.model_shape("llada8b")
    # per-position, summed over steps: the value the paper prints for N_gen = 64, 32 steps, N_p = 64 (4.488e11)
    per_pos = 32 * sampler.algorithmic_flops_per_step(cfg, 4, 128) / (4 * 128)
    assert abs(per_pos / 4.488e11 - 1) < 4e-4


@pytest.mark.gpu
def test_sampler_run_with_and_without_surelock():
    from paper_2602_06412_b200 import binding as SL
    from tests.parity_util import to_dev
    cfg = inputs.model_shape("tiny")
    w = to_dev(inputs.make_weights(cfg, 9, dtype=torch.float32))
    B, N, n_prompt, blk = 2, 128, 64, 32
    res = {}
    for mode in (True, False):
        ctx = SL.surelock_init(cfg, w, N, B)
        tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 9)
        tokens, mask = tokens.cuda(), mask.cuda()
        res[mode] = sampler.run(ctx, tokens, mask, n_prompt, blk, steps=64, kl_eps=1e-3, surelock=mode)
        assert SL.surelock_status_poll(ctx) == 0
        assert res[mode]["masked_at_end"] == 0 and int((tokens == cfg["vocab"] - 1).sum()) == 0
        assert res[mode]["unmasked_per_step"] == [B] * 64
    sure, base = res[True], res[False]
    assert base["M_trace"] == [B * N] * 64 and base["r_bar"] == 1.0 and base["locked_at_end"] == 0
    M = sure["M_trace"]
    assert M[0] == M[1] == B * N                       # D_1 = inf: the first step cannot lock
    assert all(a >= b for a, b in zip(M, M[1:])) and M[-1] < B * N
    assert abs(sure["r_bar"] - sum(M) / (64 * B * N)) < 1e-12 and sure["flops_ratio"] == sure["r_bar"] < 1.0
    assert abs(sure["f_prop_per_position"] / sure["f_base_per_position"] - sure["r_bar"]) < 1e-12
    assert sure["e2e_tps"] > 0 and len(sure["step_tps"]) == 64


@pytest.mark.gpu
def test_selection_hybrid_run():
    """Experiment 5's three settings on a tiny model: selection alone computes a fixed fraction of all positions,
    SureLock alone the unlocked ones, the combination that fraction of the unlocked ones (never skipping a masked
    position), so it computes no more than selection alone; decoding still completes."""
    from paper_2602_06412_b200 import binding as SL
    from tests.parity_util import to_dev
    cfg = inputs.model_shape("tiny")
    w = to_dev(inputs.make_weights(cfg, 9, dtype=torch.float32))
    B, N, n_prompt, blk, steps, k = 2, 128, 64, 32, 64, 0.8
    res = {}
    for name, sure, frac in (("sure", True, None), ("select", False, k), ("hybrid", True, k)):
        ctx = SL.surelock_init(cfg, w, N, B)
        tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 9)
        tokens, mask = tokens.cuda(), mask.cuda()
        res[name] = sampler.run(ctx, tokens, mask, n_prompt, blk, steps=steps, kl_eps=1e-3, surelock=sure,
                                select_fraction=frac, select_seed=4)
        assert SL.surelock_status_poll(ctx) == 0
        assert res[name]["masked_at_end"] == 0 and res[name]["unmasked_per_step"] == [B] * steps
    sel, hyb, sure = res["select"], res["hybrid"], res["sure"]
    # selection alone: floor(0.2 * N) positions per sequence skipped whenever enough unmasked ones exist
    for t, M in enumerate(sel["M_trace"]):
        masked = B * max(N - n_prompt - t, 0)                           # one reveal per sequence and step
        assert B * N - B * int(N * (1 - k)) <= M <= B * N and M >= masked
    assert sel["locked_at_end"] == 0
    # (a skipped row cannot lock in the step in which it returns, so the combination locks later than SureLock alone;
    # with these synthetic posteriors, where rows lock right after being revealed, it need not beat SureLock alone)
    assert hyb["r_bar"] < sel["r_bar"] < 1.0 and sure["r_bar"] < 1.0 and hyb["locked_at_end"] > 0
    assert all(m <= s for m, s in zip(hyb["M_trace"][2:], sel["M_trace"][2:]))


def test_selection_skip_mask_properties():
    g = torch.Generator().manual_seed(1)
    B, N = 3, 50
    lock = (torch.rand((B, N), generator=g) < 0.3).to(torch.uint8)
    mask = ((torch.rand((B, N), generator=g) < 0.3) & (lock == 0)).to(torch.uint8)
    mask[2] = (lock[2] == 0).to(torch.uint8)                             # every unlocked position still masked
    skip = sampler.selection_skip_mask(lock, mask, 0.8, 5, 7)
    assert not (skip & lock).any() and not (skip & mask).any()          # only computed, unmasked positions are skipped
    for b in range(B):
        unlocked = int((lock[b] == 0).sum())
        eligible = int(((lock[b] == 0) & (mask[b] == 0)).sum())
        assert int(skip[b].sum()) == min(int(unlocked * 0.2), eligible)
    assert torch.equal(skip, sampler.selection_skip_mask(lock, mask, 0.8, 5, 7))   # seeded
    assert not torch.equal(skip, sampler.selection_skip_mask(lock, mask, 0.8, 6, 7))


@pytest.mark.gpu
def test_sampler_run_with_unlocking():
    """The decoding loop with optional un-locking switched on: the run completes, the active-row trace may now grow
    again after a probe step, and every un-lock the probe reports shows up as that growth."""
    from paper_2602_06412_b200 import binding as SL
    from tests.parity_util import to_dev
    cfg = inputs.model_shape("tiny")
    w = to_dev(inputs.make_weights(cfg, 13, dtype=torch.float32, std=0.08))
    B, N, n_prompt, blk, steps = 2, 96, 40, 28, 40
    ctx = SL.surelock_init(cfg, w, N, B)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 13)
    res = sampler.run(ctx, tokens.cuda(), mask.cuda(), n_prompt, blk, steps=steps, kl_eps=1e-3,
                      unlock=dict(period=2, eps_unlock=2e-5, d_interval=1, d_cool=2, rho=0.25, m_percent=50.0))
    assert SL.surelock_status_poll(ctx) == 0
    un, M = res["unlocked_per_step"], res["M_trace"]
    assert sum(un) > 0 and all(u == 0 for u in un[0::2])                # probes after steps 2, 4, ... (indices 1, 3, ...)
    grew = [t for t in range(1, steps) if M[t] > M[t - 1]]
    assert grew and all(un[t - 1] > 0 for t in grew)                    # the active set only grows through an un-lock
    assert res["unmasked_per_step"] == [B] * steps


@pytest.mark.gpu
def test_sampler_run_bf16_through_the_few_row_kernels():
    """The decoding loop on a bf16 model of the LLaDA-8B layer shape with one short sequence: from the third step on the
    row bound (<= 128) selects the layer chain kernel for every step (N = 128 is a single key block, so attention stays
    on the general kernel); the run completes, the active-row trace never grows, no status is raised."""
    from paper_2602_06412_b200 import binding as SL
    cfg = inputs.model_shape("llada8b", n_layers=2, vocab=4096)
    w = inputs.make_weights(cfg, 21, dtype=torch.bfloat16, device="cuda")
    B, N, n_prompt, blk, steps = 1, 128, 64, 32, 64
    ctx = SL.surelock_init(cfg, w, N, B)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 21)
    tokens, mask = tokens.cuda(), mask.cuda()
    res = sampler.run(ctx, tokens, mask, n_prompt, blk, steps=steps, kl_eps=1e-3)
    assert SL.surelock_status_poll(ctx) == 0 and SL.surelock_last_step_paths(ctx) == 1
    assert res["masked_at_end"] == 0 and res["unmasked_per_step"] == [B] * steps
    M = res["M_trace"]
    assert M[0] == B * N and all(a >= b for a, b in zip(M, M[1:]))
    # the same with optional un-locking switched on (probe steps run on the general kernels, a row that returns to the
    # active set may make the bound too small for a step: further passes)
    ctx = SL.surelock_init(cfg, w, N, B)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 21)
    res = sampler.run(ctx, tokens.cuda(), mask.cuda(), n_prompt, blk, steps=steps, kl_eps=1e-3,
                      unlock=dict(period=2, eps_unlock=2e-5, d_interval=1, d_cool=2, rho=0.25, m_percent=50.0))
    assert SL.surelock_status_poll(ctx) == 0
    assert res["masked_at_end"] == 0 and res["unmasked_per_step"] == [B] * steps
