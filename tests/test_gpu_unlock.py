"""Optional un-locking (App. "Optional Unlocking") on the GPU against the oracle, step by step on the tiny fp32 model:
the step's lock update with per-position thresholds and cool-down, the recorded t*, the frozen posteriors, the probe
(proxy posteriors of the locked rows against the caches, which it must not change), the drift, theta_t, and the
un-lock decisions, which must agree exactly outside the tolerance bands around the three thresholds."""
import copy

import numpy as np
import pytest
import torch

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import binding as SL
from paper_2602_06412_b200 import inputs
from tests.parity_util import f64, rel_err_rows, to_dev

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("dtype,gate", [(torch.float32, None), (torch.float32, 60.0), (torch.bfloat16, None)])
def test_unlock_cycle_matches_the_oracle(dtype, gate):
    cfg = inputs.model_shape("tiny")
    oc = O.ModelCfg(**cfg)
    B, N, n_prompt, eps, steps = 2, 96, 40, 1e-3, 18
    P = O.UnlockParams(period=2, eps_unlock=2e-5, d_interval=1, d_cool=2, rho=0.25, m=50.0)
    w = inputs.make_weights(cfg, 13, dtype=dtype, std=0.08)
    wn = inputs.weights_to_numpy(w)
    ctx = SL.surelock_init(cfg, to_dev(w), N, B)
    SL.surelock_set_unlocking(ctx, P.period, P.eps_unlock, P.d_interval, P.d_cool, P.rho, P.m)
    if gate is not None:
        SL.surelock_set_confidence_gate(ctx, gate)
    is_bf16 = dtype == torch.bfloat16
    rnd = (lambda a: torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()) if is_bf16 else None
    tol = 5e-2 if is_bf16 else 2e-4
    st = O.OracleState(oc, B, N)
    us = O.UnlockState(B, N, cfg["vocab"])
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], 13)
    lock = torch.zeros((B, N), dtype=torch.uint8)
    V = cfg["vocab"]
    n_unlocked_total, n_relocked, probes = 0, 0, 0
    prev_gpu = {}
    for t in range(1, steps + 1):
        lock_in = lock.clone()
        lock_d = lock.to(DEV)
        tok_d, mask_d = tokens.to(DEV), mask.to(DEV)
        out = SL.surelock_step(ctx, tok_d, mask_d, lock_d, eps)
        assert SL.surelock_status_poll(ctx) == 0
        e_rows, may = O.relock_thresholds(us, eps, P.rho, t)
        ref = O.step(st, wn, tokens.numpy(), mask.numpy(), lock_in.numpy(), eps, logits_round=rnd, kl_eps_rows=e_rows,
                     may_lock=may, conf_gate_m=gate)
        M = out.M()
        idx = ref["active_idx"]
        assert M == len(idx) and np.array_equal(out.active_idx[:M].cpu().numpy(), idx)
        g_logits = f64(out.logits[:M])
        assert rel_err_rows(g_logits, ref["logits"]) < tol, t
        # the lock update: the oracle's rule on the KL of the logits the GPU materialised
        bb, ii = idx // N, idx % N
        have = np.array([int(p) in prev_gpu for p in idx])
        kl_ref = np.full(M, np.inf)
        if have.any():
            kl_ref[have] = O.kl_from_logits(g_logits[have], np.stack([prev_gpu[int(p)] for p in idx[have]]))
        kl_gpu = out.kl[:M].cpu().numpy().astype(np.float64)
        assert np.array_equal(np.isfinite(kl_gpu), have)
        assert np.all(np.abs(kl_gpu[have] - kl_ref[have]) <= 1e-3 * kl_ref[have] + 1e-9), t
        eps_i = e_rows[bb, ii]
        want = O.sure_test(kl_ref, mask.numpy()[bb, ii], eps_i) & (may[bb, ii] != 0)
        near = np.isfinite(kl_ref) & (np.abs(kl_ref - eps_i) <= 1e-3 * eps_i)
        if gate is not None:
            conf_gpu = out.conf[:M].cpu().numpy().astype(np.float64)
            gp, theta = O.confidence_gate(conf_gpu, mask.numpy()[bb, ii] == 0, bb, B, gate)
            want &= gp
            near |= np.abs((1.0 - conf_gpu) - theta[bb]) <= 1e-6
        new_lock = lock_d.cpu()
        got = new_lock.numpy()[bb, ii].astype(bool)
        assert np.array_equal(got[~near], want[~near]), (t, "lock decisions")
        assert torch.all(new_lock >= lock_in)
        assert not got[(us.cool_until[bb, ii] >= t)].any(), (t, "no lock during the cool-down")
        n_relocked += int((got & us.relock[bb, ii]).sum())
        # both sides go on from the GPU's decisions
        ref["new_lock"] = new_lock.numpy().copy()
        ref["logp"] = O.log_softmax(g_logits)                        # p_{t*} as the GPU holds it: its own logits
        O.record_locks(us, t, lock_in.numpy(), ref, N)
        for r, p in enumerate(idx):
            prev_gpu[int(p)] = g_logits[r]
        for p in set(prev_gpu) - set(int(p) for p in idx):            # "previous" means the step just taken
            del prev_gpu[p]
        lock = new_lock.clone()
        # the caller's unmasking, from the oracle's posteriors (as in the other side-by-side tests)
        conf_o, am_o = O.posterior_stats(ref["logits"])
        for b in range(B):
            rows = [r for r in range(M) if bb[r] == b and mask[b, ii[r]] == 1]
            if rows:
                r = max(rows, key=lambda r: (conf_o[r], -r))
                tokens[b, ii[r]] = int(am_o[r]) if am_o[r] != V - 1 else 0
                mask[b, ii[r]] = 0
        # ---- the probe
        kv_before = [t_.clone() for t_ in SL.surelock_kv_cache(ctx, 1)]
        lock_d = lock.to(DEV)
        po = SL.surelock_probe_unlock(ctx, tokens.to(DEV), lock_d)
        assert SL.surelock_status_poll(ctx) == 0
        assert po.step == t and po.probed == (t % P.period == 0)
        if not po.probed:
            assert torch.equal(lock_d.cpu(), lock)
            continue
        probes += 1
        for a, b_ in zip(kv_before, SL.surelock_kv_cache(ctx, 1)):    # the probe writes nothing into the caches
            assert torch.equal(a.view(torch.uint8), b_.view(torch.uint8))
        conf_act = out.conf[:M].cpu().numpy().astype(np.float64)
        pr = O.probe_unlock(st, copy.deepcopy(us), wn, tokens.numpy(), lock.numpy(), t,
                            conf_act, idx, P, logits_round=rnd)
        n = int(po.n_probed.item())
        li = pr["locked_idx"]
        assert n == len(li) and np.array_equal(po.probed_idx[:n].cpu().numpy(), li)
        np.testing.assert_allclose(po.theta.cpu().numpy(), pr["theta"], rtol=1e-5, atol=1e-7)
        if n == 0:
            continue
        lb, lp = li // N, li % N
        has_star = us.t_star[lb, lp] >= 0
        drift_g = po.drift[:n].cpu().numpy().astype(np.float64)
        assert np.all(np.isinf(drift_g[~has_star]))
        if not is_bf16:                                               # fp32 path: free running against the all-fp64 probe
            d_ref = pr["drift"][has_star]
            assert np.all(np.abs(drift_g[has_star] - d_ref) <= 2e-3 * d_ref + 1e-8), (t, "drift")
            np.testing.assert_allclose(po.conf[:n].cpu().numpy(), 1.0 - pr["u"], rtol=2e-4)
        # decisions: the oracle's rule on the GPU's own proxy statistics, exact outside the bands
        u_g = 1.0 - po.conf[:n].cpu().numpy().astype(np.float64)
        th = po.theta.cpu().numpy().astype(np.float64)[lb]
        fire = O.unlock_test(u_g, drift_g, th, t, us.t_star[lb, lp], P) & has_star
        band = (np.abs(u_g - th) <= 1e-6) | (np.abs(drift_g - P.eps_unlock) <= 1e-3 * P.eps_unlock)
        after = lock_d.cpu().numpy()
        got_unlock = (after[lb, lp] == 0)
        assert np.array_equal(got_unlock[~band], fire[~band]), (t, "un-lock decisions")
        assert np.array_equal(after[lock.numpy() == 0], lock.numpy()[lock.numpy() == 0])   # nothing else changes
        assert int(po.n_unlocked.item()) == int(got_unlock.sum())
        # both sides go on from the GPU's decisions; the bookkeeping must agree
        us.cool_until[lb[got_unlock], lp[got_unlock]] = t + P.d_cool
        us.relock[lb[got_unlock], lp[got_unlock]] = True
        assert np.array_equal(po.cool_until.cpu().numpy().reshape(B, N), us.cool_until)
        assert np.array_equal(po.t_star.cpu().numpy().reshape(B, N), us.t_star)
        n_unlocked_total += int(got_unlock.sum())
        lock = torch.from_numpy(after.copy())
    assert probes == steps // P.period
    assert n_unlocked_total > 0, "the scenario must un-lock something"
    print("un-locked", n_unlocked_total, "re-locked later", n_relocked, "locked at the end", int(lock.sum()))


def test_unlocking_argument_checks():
    cfg = inputs.model_shape("tiny")
    ctx = SL.surelock_init(cfg, to_dev(inputs.make_weights(cfg, 3, dtype=torch.float32)), 32, 1)
    tokens, mask = inputs.make_tokens(1, 32, 16, cfg["vocab"], 3)
    lock = torch.zeros((1, 32), dtype=torch.uint8, device=DEV)
    with pytest.raises(SL.SurelockError):
        SL.surelock_probe_unlock(ctx, tokens.to(DEV), lock)              # un-locking was never switched on
    for bad in (dict(period=0), dict(rho=1.5), dict(m_percent=101.0), dict(eps_unlock=float("nan")), dict(d_cool=-1)):
        with pytest.raises(SL.SurelockError):
            SL.surelock_set_unlocking(ctx, **bad)
    SL.surelock_set_unlocking(ctx, period=3)
    SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, 1e-3)
    po = SL.surelock_probe_unlock(ctx, tokens.to(DEV), lock)
    assert po.step == 1 and not po.probed                                 # only every third step
    SL.surelock_set_unlocking(ctx, off=True)
    SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0
