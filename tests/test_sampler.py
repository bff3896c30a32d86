"""The decoding harness: the unmasking policy (pure torch, checked on CPU against a loop) and, on the GPU, the
sampler loop with and without SureLock (trace invariants and the paper's run metrics)."""
import numpy as np
import pytest
import torch

from paper_2602_06412_b200 import inputs, sampler


def test_update_mask_policy_matches_a_plain_loop():
    g = torch.Generator().manual_seed(3)
    B, N, lo, hi, mask_tok = 4, 40, 16, 32, 99
    for k in (1, 3):
        tokens = torch.randint(0, 50, (B, N), generator=g, dtype=torch.int32)
        mask = (torch.rand((B, N), generator=g) < 0.5).to(torch.uint8)
        mask[1, lo:hi] = 0                                  # a sequence whose block is already fully revealed
        mask[2, lo:hi] = 1
        conf = torch.rand((B, N), generator=g)
        conf[2, lo + 3] = conf[2, lo + 7] = 2.0             # a tie: the lower index wins
        am = torch.randint(0, 100, (B, N), generator=g, dtype=torch.int32)
        am[2, lo + 3] = mask_tok                            # the argmax happens to be the mask token: reveal token 0
        t_ref, m_ref = tokens.clone(), mask.clone()
        for b in range(B):
            for _ in range(k):
                cand = [i for i in range(lo, hi) if m_ref[b, i] == 1]
                if not cand:
                    break
                best = max(cand, key=lambda i: (float(conf[b, i]), -i))
                t_ref[b, best] = 0 if int(am[b, best]) == mask_tok else int(am[b, best])
                m_ref[b, best] = 0
        sampler.update_mask(tokens, mask, conf, am, lo, hi, k, mask_tok)
        assert torch.equal(tokens, t_ref) and torch.equal(mask, m_ref)


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
