"""Side-by-side driver of the CUDA step and the CPU oracle for parity tests (and the smoke check).

Both sides receive the same tokens, mask state and lock mask at every step.  The unmasking policy (Algorithm 1
line 16, outside the library) is played by this driver from the ORACLE's posteriors: among the masked positions
of each sequence the most confident one is revealed with its argmax token.  Lock decisions entering the next
step are the GPU's, after they have been checked against the oracle's (so a decision inside the tolerance band
cannot make the two runs drift apart); an optional forced seeded schedule adds more locks.
"""
import numpy as np
import torch

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import binding as SL
from paper_2602_06412_b200 import inputs
from tests.parity_util import f64, rel_err_rows, rel_err_stats, to_dev


def run_side_by_side(cfg, dtype, B, N, n_prompt, steps, kl_eps, seed, tol_logits, tol_hidden=None, std=0.02,
                     forced_p=0.0, kl_tol=1e-3, kl_floor=1e-9, check_kl_free_running=False, log=None, conf_gate_m=None,
                     tol_rms=None, tol_p9999=None):
    """Returns the per-step trace of M.  Raises AssertionError on the first parity violation.

    tol_logits / tol_hidden bound the MAXIMUM relative error of a step's logits / hidden states against the all-fp64
    oracle; tol_rms and tol_p9999, when given, also bound the root mean square and the 99.99th percentile of the
    same per-entry error (the free-running bf16 runs: the maximum over 10^5..10^6 entries is a tail statistic of
    the rounding noise, the RMS and the percentile are what a wrong kernel would move first)."""
    tol_hidden = tol_hidden or tol_logits
    w = inputs.make_weights(cfg, seed, dtype=dtype, std=std)
    wn = inputs.weights_to_numpy(w)
    wd = to_dev(w)
    oc = O.ModelCfg(**cfg)
    ctx = SL.surelock_init(cfg, wd, N, B)
    theta_view = SL.surelock_set_confidence_gate(ctx, conf_gate_m) if conf_gate_m is not None else None
    st = O.OracleState(oc, B, N)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], seed)
    lock = torch.zeros((B, N), dtype=torch.uint8)
    V = cfg["vocab"]
    is_bf16 = dtype == torch.bfloat16
    prev_gpu_logits = {}                       # flat position -> np row of the GPU's previous logits
    trace = []
    round_fn = None
    if is_bf16:
        round_fn = lambda a: torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    for t in range(steps):
        lock_in = lock.clone()
        lock_d = lock.to("cuda")
        out = SL.surelock_step(ctx, tokens.to("cuda"), mask.to("cuda"), lock_d, kl_eps)
        assert SL.surelock_status_poll(ctx) == 0
        ref = O.step(st, wn, tokens.numpy(), mask.numpy(), lock_in.numpy(), kl_eps, logits_round=round_fn)
        M = out.M()
        trace.append(M)
        # ---- integer work: bit exact
        assert M == len(ref["active_idx"]), (t, M, len(ref["active_idx"]))
        assert np.array_equal(out.active_idx[:M].cpu().numpy(), ref["active_idx"])
        assert np.array_equal(out.row_offsets.cpu().numpy(), ref["row_offsets"])
        if M == 0:
            break
        # ---- hidden states and logits, free running against fp64
        e_h = rel_err_rows(f64(out.hidden[:M]), ref["hidden"])
        g_logits = f64(out.logits[:M])
        e_l = rel_err_rows(g_logits, ref["logits"])
        assert e_h < tol_hidden, (t, "hidden", e_h)
        assert e_l < tol_logits, (t, "logits", e_l)
        s_h, s_l = rel_err_stats(f64(out.hidden[:M]), ref["hidden"]), rel_err_stats(g_logits, ref["logits"])
        if tol_rms is not None:
            assert s_h["rms"] < tol_rms and s_l["rms"] < tol_rms, (t, "rms", s_h, s_l)
        if tol_p9999 is not None:
            assert s_h["p9999"] < tol_p9999 and s_l["p9999"] < tol_p9999, (t, "p99.99", s_h, s_l)
        # ---- KL / confidence / argmax: the oracle's formulas evaluated on the logits the GPU materialised
        idx = ref["active_idx"]
        have = np.array([int(p) in prev_gpu_logits for p in idx])
        kl_ref = np.full(M, np.inf)
        if have.any():
            prevs = np.stack([prev_gpu_logits[int(p)] for p in idx[have]])
            kl_ref[have] = O.kl_from_logits(g_logits[have], prevs)
        kl_gpu = out.kl[:M].cpu().numpy().astype(np.float64)
        assert np.all(np.isinf(kl_gpu[~have]))
        err = np.abs(kl_gpu[have] - kl_ref[have])
        assert np.all(err <= kl_tol * kl_ref[have] + kl_floor), (t, "kl", err.max())
        if check_kl_free_running:                                   # fp32 path: also against the all-fp64 run
            fr = ref["kl"]
            fin = np.isfinite(fr)
            assert np.array_equal(fin, have)
            assert np.all(np.abs(kl_gpu[fin] - fr[fin]) <= kl_tol * fr[fin] + kl_floor), (t, "kl free-running")
        conf_ref, am_ref = O.posterior_stats(g_logits)
        assert np.array_equal(out.argmax[:M].cpu().numpy(), am_ref), (t, "argmax")
        np.testing.assert_allclose(out.conf[:M].cpu().numpy(), conf_ref, rtol=1e-4)
        # ---- lock decisions: exact outside the tolerance band around the threshold
        bb, ii = idx // N, idx % N
        want = O.sure_test(kl_ref, mask.numpy()[bb, ii], kl_eps)
        near = np.isfinite(kl_ref) & (np.abs(kl_ref - kl_eps) <= kl_tol * kl_eps)
        if conf_gate_m is not None:          # the gate, evaluated by the oracle on the confidences the GPU produced
            conf_gpu = out.conf[:M].cpu().numpy().astype(np.float64)
            gate, theta = O.confidence_gate(conf_gpu, mask.numpy()[bb, ii] == 0, bb, B, conf_gate_m)
            want = want & gate
            th_gpu = theta_view.cpu().numpy().astype(np.float64)
            fin_t = np.isfinite(theta)
            assert np.array_equal(np.isfinite(th_gpu), fin_t)
            np.testing.assert_allclose(th_gpu[fin_t], theta[fin_t], rtol=1e-5, atol=1e-7)
            near = near | (np.abs((1.0 - conf_gpu) - theta[bb]) <= 1e-6)
        new_lock = lock_d.cpu()
        got = new_lock.numpy()[bb, ii].astype(bool)
        assert np.array_equal(got[~near], want[~near]), (t, "lock decisions")
        assert torch.all(new_lock >= lock_in), (t, "lock mask must be monotone")
        expect_new = torch.zeros((B, N), dtype=torch.bool)
        expect_new[torch.from_numpy(bb[got]).long(), torch.from_numpy(ii[got]).long()] = True
        assert torch.equal(new_lock.bool() & ~lock_in.bool(), expect_new), (t, "only tested active rows lock")
        if log is not None:
            log.append(dict(t=t, M=M, e_hidden=e_h, e_logits=e_l, hidden=s_h, logits=s_l, kl_err=float(err.max()) if have.any() else 0.0,
                            locked=int(new_lock.sum())))
        for r, p in enumerate(idx):
            prev_gpu_logits[int(p)] = g_logits[r]
        # ---- frozen K/V of locked rows: compare cache bytes of layer 0 and the last layer over time
        # (done by the caller through surelock_kv_cache when wanted)
        lock = new_lock.clone()
        if forced_p > 0 and t >= 1:
            lock = inputs.bernoulli_lock_schedule(lock, mask == 0, forced_p, seed * 977 + t)
        # ---- the caller's unmasking policy, from the oracle's posteriors
        conf_o, am_o = O.posterior_stats(ref["logits"])
        for b in range(B):
            rows = [r for r in range(M) if bb[r] == b and mask[b, ii[r]] == 1]
            if rows:
                r = max(rows, key=lambda r: (conf_o[r], -r))
                tokens[b, ii[r]] = int(am_o[r]) if am_o[r] != V - 1 else 0
                mask[b, ii[r]] = 0
    return trace, ctx, st
