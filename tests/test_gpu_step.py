"""Whole-step GPU parity against the CPU oracle: the tiny fp32 model (free running, sampler loop, natural and
forced lock schedules), a bf16 model through the same step, the single-layer call at LLaDA-8B layer shape, the
host-buffer entry point, and the invariants of the cache (locked rows' bytes never change)."""
import numpy as np
import pytest
import torch

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import binding as SL
from paper_2602_06412_b200 import inputs
from tests.parity_util import f64, rel_err_rows, to_dev
from tests.stepper import run_side_by_side

pytestmark = pytest.mark.gpu
DEV = "cuda"
# Whole-step bf16 runs against the ALL-fp64 oracle (free running: every bf16 rounding of an activation since the
# embedding is in the difference).  The 2e-2 bar of the bf16 path is enforced stage by stage, from the GPU's own traced
# inputs, in test_gpu_teacher_forced.py; here the per-entry relative error is rounding noise that has passed through
# 2-3 layers, and what is bounded is its distribution: root mean square <= 1e-2 (measured 0.43-0.61 %), 99.99th
# percentile <= 3e-2 (measured 2.0-2.5 %), maximum over 10^5..10^6 entries <= 5e-2 (measured 2.2-3.5 %).
BF16_FREE_RUNNING = dict(tol_logits=5e-2, tol_rms=1e-2, tol_p9999=3e-2)


def test_tiny_fp32_sampler_natural_locks():
    cfg = inputs.model_shape("tiny")
    log = []
    trace, ctx, st = run_side_by_side(cfg, torch.float32, B=1, N=128, n_prompt=64, steps=64, kl_eps=1e-3, seed=1,
                                      tol_logits=1e-4, check_kl_free_running=True, log=log)
    assert trace[0] == 128 and trace[1] == 128          # D_1 = inf: nothing can lock before the second step
    assert min(trace) < 128                             # and SureLock does shrink the active set afterwards
    assert all(a >= b for a, b in zip(trace, trace[1:]))


def test_tiny_fp32_forced_lock_schedule_and_peaked_posteriors():
    cfg = inputs.model_shape("tiny")
    # larger weights give peaked, moving posteriors: KL spreads on both sides of the threshold
    trace, ctx, st = run_side_by_side(cfg, torch.float32, B=2, N=96, n_prompt=40, steps=24, kl_eps=1e-3, seed=2,
                                      tol_logits=2e-4, std=0.08, forced_p=0.25, check_kl_free_running=True,
                                      kl_floor=1e-8)
    assert trace[-1] < trace[0]


def test_tiny_bf16_step():
    cfg = inputs.model_shape("tiny")
    run_side_by_side(cfg, torch.bfloat16, B=2, N=128, n_prompt=64, steps=10, kl_eps=1e-3, seed=3, std=0.05, forced_p=0.2,
                     **BF16_FREE_RUNNING)


def test_bf16_head_dim_128_ragged_batch():
    cfg = inputs.model_shape("tiny", d_model=512, n_heads=4, head_dim=128, d_ff=1536, vocab=4096, n_layers=3)
    run_side_by_side(cfg, torch.bfloat16, B=3, N=200, n_prompt=90, steps=8, kl_eps=1e-3, seed=4, std=0.04, forced_p=0.3,
                     **BF16_FREE_RUNNING)


def test_confidence_gate_in_the_step():
    """Algorithm 1 line 21 with the paper's default m = 20 %: fewer rows lock than with the KL criterion alone."""
    cfg = inputs.model_shape("tiny")
    plain, _, _ = run_side_by_side(cfg, torch.float32, B=2, N=96, n_prompt=40, steps=12, kl_eps=1e-3, seed=5,
                                   tol_logits=1e-4)
    gated, _, _ = run_side_by_side(cfg, torch.float32, B=2, N=96, n_prompt=40, steps=12, kl_eps=1e-3, seed=5,
                                   tol_logits=1e-4, conf_gate_m=20.0)
    assert gated[2] > plain[2]                       # at the third step the gate has held most candidates back
    assert all(a >= b for a, b in zip(gated, gated[1:]))
    run_side_by_side(cfg, torch.bfloat16, B=3, N=128, n_prompt=64, steps=6, kl_eps=1e-3, seed=6, std=0.05, conf_gate_m=40.0,
                     **BF16_FREE_RUNNING)


def test_locked_rows_cache_bytes_never_change_and_active_rows_are_rewritten():
    cfg = inputs.model_shape("tiny")
    w = inputs.make_weights(cfg, 5, dtype=torch.bfloat16, std=0.05)
    B, N = 2, 128
    ctx = SL.surelock_init(cfg, to_dev(w), N, B)
    tokens, mask = inputs.make_tokens(B, N, 64, cfg["vocab"], 5)
    lock = torch.zeros((B, N), dtype=torch.uint8, device=DEV)
    SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, 0.0)
    snap = [[t.clone() for t in SL.surelock_kv_cache(ctx, l)] for l in range(cfg["n_layers"])]
    lock2 = inputs.random_lock(B, N, [50, 3], 6).to(DEV)
    tok2 = tokens.clone()
    tok2[:, 64:80] = 7
    SL.surelock_step(ctx, tok2.to(DEV), mask.to(DEV), lock2.clone(), 0.0)
    torch.cuda.synchronize()
    locked = lock2.reshape(-1).bool()
    for l in range(cfg["n_layers"]):
        k, v = SL.surelock_kv_cache(ctx, l)
        for new, old in ((k, snap[l][0]), (v, snap[l][1])):
            assert torch.equal(new[locked].view(torch.int16), old[locked].view(torch.int16))
        changed = (k.view(torch.int16) != snap[l][0].view(torch.int16)).flatten(1).any(1)
        assert not (changed & locked).any()
        if l > 0:                                       # deeper layers see the new tokens through attention
            assert (changed & ~locked).sum() >= (~locked).sum() // 2
    assert SL.surelock_status_poll(ctx) == 0


def test_step_is_deterministic_and_host_entry_point_matches():
    cfg = inputs.model_shape("tiny")
    w = to_dev(inputs.make_weights(cfg, 7, dtype=torch.bfloat16, std=0.05))
    B, N = 2, 128
    tokens, mask = inputs.make_tokens(B, N, 64, cfg["vocab"], 7)
    results = []
    for use_host in (False, False, True):
        ctx = SL.surelock_init(cfg, w, N, B)
        lock = torch.zeros((B, N), dtype=torch.uint8)
        outs = []
        for t in range(3):
            if use_host:
                tk, mk, lk = tokens.clone().pin_memory(), mask.clone().pin_memory(), lock.clone().pin_memory()
                n = torch.zeros(1, dtype=torch.int32).pin_memory()
                R = B * N
                ai = torch.zeros(R, dtype=torch.int32).pin_memory()
                kl, cf = torch.zeros(R).pin_memory(), torch.zeros(R).pin_memory()
                am = torch.zeros(R, dtype=torch.int32).pin_memory()
                SL.surelock_step_host(ctx, tk, mk, lk, 1e-3, n, ai, kl, cf, am)
                M = int(n.item())
                outs.append((M, ai[:M].clone(), kl[:M].clone(), cf[:M].clone(), am[:M].clone(), lk.clone()))
                lock = lk.clone()
            else:
                ld = lock.to(DEV)
                o = SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), ld, 1e-3)
                M = o.M()
                outs.append((M, o.active_idx[:M].cpu(), o.kl[:M].cpu(), o.conf[:M].cpu(), o.argmax[:M].cpu(), ld.cpu()))
                lock = ld.cpu()
        assert SL.surelock_status_poll(ctx) == 0
        results.append(outs)
    for a, b in ((results[0], results[1]), (results[0], results[2])):
        for sa, sb in zip(a, b):
            assert sa[0] == sb[0]
            for x, y in zip(sa[1:], sb[1:]):
                assert torch.equal(x, y)                # bitwise: same inputs, same outputs, device or host buffers


def test_argument_errors_are_reported_not_fatal():
    cfg = inputs.model_shape("tiny")
    w = to_dev(inputs.make_weights(cfg, 8, dtype=torch.float32))
    ctx = SL.surelock_init(cfg, w, 32, 1)
    tokens, mask = inputs.make_tokens(1, 32, 16, cfg["vocab"], 8)
    lock = torch.zeros((1, 32), dtype=torch.uint8, device=DEV)
    with pytest.raises(SL.SurelockError):
        SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, float("nan"))
    with pytest.raises(SL.SurelockError):
        SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, -1.0)
    with pytest.raises(SL.SurelockError):
        SL.surelock_step(ctx, None, mask.to(DEV), lock, 1e-3)
    bad = dict(cfg, head_dim=48, n_heads=4)
    with pytest.raises(SL.SurelockError):
        SL.surelock_init(bad, w, 32, 1)
    # an out-of-range token is skipped and reported through the status word; the context stays usable
    tk = tokens.clone()
    tk[0, 3] = cfg["vocab"] + 5
    SL.surelock_step(ctx, tk.to(DEV), mask.to(DEV), lock, 1e-3)
    assert SL.surelock_status_poll(ctx) == 4
    SL.surelock_reset(ctx)
    SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0


@pytest.mark.parametrize("M_list", [[1024, 512, 256, 128, 32]])
def test_single_layer_llada_shape(M_list):
    """Single LLaDA-8B-shaped layer, N=1024: cache pre-filled by one full pass, then seeded random active subsets."""
    cfg = inputs.model_shape("llada8b", n_layers=1, vocab=0)
    oc = O.ModelCfg(**cfg)
    N, d = 1024, cfg["d_model"]
    lw = inputs.make_layer_weights(cfg, 0, 21, dtype=torch.bfloat16)
    w = dict(layers=[lw])
    wn = inputs.weights_to_numpy(w)["layers"][0]
    ctx = SL.surelock_init(cfg, to_dev(w), N, 1)
    H0 = inputs.hidden_states(N, d, 1)
    H1 = inputs.hidden_states(N, d, 2)
    out_buf = torch.zeros((N, d), dtype=torch.float32, device=DEV)
    Kc = np.zeros((N, cfg["n_heads"], cfg["head_dim"]))
    Vc = np.zeros_like(Kc)
    for M in M_list:
        if M == N:
            lock = torch.zeros((1, N), dtype=torch.uint8)
            Hin = H0
        else:
            lock = inputs.random_lock(1, N, [M], 100 + M)
            Hin = H1
        o = SL.surelock_layer_step(ctx, 0, Hin.to(DEV), lock.to(DEV), out_buf)
        assert SL.surelock_status_poll(ctx) == 0
        idx, _ = O.active_set(lock.numpy())
        assert o.M() == M and np.array_equal(o.active_idx[:M].cpu().numpy(), idx)
        # the oracle's cache holds the GPU's (bf16) cache before this pass: stage-wise, teacher-forced
        kg, vg = SL.surelock_kv_cache(ctx, 0)
        ref = O.layer_rows(oc, wn, f64(Hin[idx]), idx.astype(np.int64), Kc, Vc)
        e = rel_err_rows(f64(out_buf[:M]), ref)
        assert e < 2e-2, (M, e)
        ek = rel_err_rows(f64(kg).reshape(N, -1), Kc.reshape(N, -1))
        ev = rel_err_rows(f64(vg).reshape(N, -1), Vc.reshape(N, -1))
        assert ek < 2e-2 and ev < 2e-2, (M, ek, ev)
        Kc[:] = f64(kg)
        Vc[:] = f64(vg)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-4), (torch.bfloat16, 5e-2)])
def test_degenerate_active_sets(dtype, tol):
    """The degenerate cases of the active set: every position locked (M = 0: nothing is computed or written, the call
    still succeeds), one sequence of the batch fully locked next to a sequence with a single active row, and a row that
    returns to the active set after a step in which it was not computed (D = inf in its first step back)."""
    cfg = inputs.model_shape("tiny")
    B, N, eps = 3, 96, 1e-3
    w = inputs.make_weights(cfg, 11, dtype=dtype, std=0.05)
    wn, wd = inputs.weights_to_numpy(w), to_dev(w)
    ctx = SL.surelock_init(cfg, wd, N, B)
    st = O.OracleState(O.ModelCfg(**cfg), B, N)
    tokens, mask = inputs.make_tokens(B, N, 40, cfg["vocab"], 11)
    rnd = (lambda a: torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()) \
        if dtype == torch.bfloat16 else None
    gpu_logits = []                                      # the logits the GPU materialised, step by step

    def both(lock):
        ld = lock.to(DEV)
        out = SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), ld, eps)
        assert SL.surelock_status_poll(ctx) == 0
        ref = O.step(st, wn, tokens.numpy(), mask.numpy(), lock.numpy(), eps, logits_round=rnd)
        M = out.M()
        assert M == len(ref["active_idx"])
        assert np.array_equal(out.active_idx[:M].cpu().numpy(), ref["active_idx"])
        assert np.array_equal(out.row_offsets.cpu().numpy(), ref["row_offsets"])
        if M:
            assert rel_err_rows(f64(out.logits[:M]), ref["logits"]) < tol
        gpu_logits.append(f64(out.logits[:M]))
        return out, ref, ld.cpu()

    lock = torch.zeros((B, N), dtype=torch.uint8)
    both(lock)                                                           # step 1: everything active
    kv_before = [t.clone() for t in SL.surelock_kv_cache(ctx, 0)]
    # every position locked
    full = torch.ones((B, N), dtype=torch.uint8)
    out, ref, after = both(full)
    assert out.M() == 0 and torch.equal(after, full)
    for a, b in zip(kv_before, SL.surelock_kv_cache(ctx, 0)):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
    # sequence 0 fully locked, sequence 1 with one active row, sequence 2 ragged
    lock = torch.ones((B, N), dtype=torch.uint8)
    lock[1, 57] = 0
    lock[2, 5:70:3] = 0
    out, ref, after = both(lock)
    M = out.M()
    assert M == 1 + len(range(5, 70, 3)) and out.row_offsets.cpu().tolist() == [0, 0, 1, M]
    assert torch.isinf(out.kl[:M]).all()                                 # none of them was computed in the previous step
    assert torch.equal(after, lock)                                      # so none of them can lock
    # the same rows once more: now they have a previous posterior
    out, ref, after = both(lock)
    kl = out.kl[:M].cpu().numpy().astype(np.float64)
    assert np.isfinite(kl).all()
    # the same packed rows in both steps: the oracle's KL on the logits the GPU stored in these two steps
    kl_ref = O.kl_from_logits(gpu_logits[-1], gpu_logits[-2])
    assert np.all(np.abs(kl - kl_ref) <= 1e-3 * kl_ref + 1e-9)
    if dtype == torch.float32:                           # fp32 path: also against the all-fp64 run
        fin = np.isfinite(ref["kl"])
        assert fin.all() and np.all(np.abs(kl - ref["kl"]) <= 1e-3 * ref["kl"] + 1e-6)


@pytest.mark.parametrize("p_lock", [0.3, 0.65])
def test_checkpoint_resume_continues_bit_for_bit(p_lock):
    """surelock_state_export / _import: a second ctx that imports the state taken after three steps takes the fourth
    step exactly as the first one does (same packing, logits, KL, lock decisions, cache bytes); a state of another
    shape is refused.  With the faster lock schedule the fourth step has few active rows and runs on the kernels the
    row bound selects (the bound is the row count two steps back: the state carries the pending counts, so the
    importing ctx makes the same choice)."""
    cfg = inputs.model_shape("tiny", d_model=512, n_heads=4, head_dim=128, d_ff=1536, vocab=4096, n_layers=2)
    B, N, eps = 2, 160, 1e-3
    wd = to_dev(inputs.make_weights(cfg, 21, dtype=torch.bfloat16, std=0.04))
    a = SL.surelock_init(cfg, wd, N, B)
    tokens, mask = inputs.make_tokens(B, N, 60, cfg["vocab"], 21)
    tok_d, mask_d = tokens.to(DEV), mask.to(DEV)
    lock = torch.zeros((B, N), dtype=torch.uint8, device=DEV)
    for t in range(3):
        SL.surelock_step(a, tok_d, mask_d, lock, eps)
        lockable = (mask == 0) if p_lock < 0.5 else torch.ones_like(mask)   # (a forced pattern may lock masked rows)
        lock = inputs.bernoulli_lock_schedule(lock.cpu(), lockable, p_lock, 500 + t).to(DEV)
    state = SL.surelock_state_export(a)
    b = SL.surelock_init(cfg, wd, N, B)
    SL.surelock_state_import(b, state)
    la, lb = lock.clone(), lock.clone()
    oa = SL.surelock_step(a, tok_d, mask_d, la, eps)
    ob = SL.surelock_step(b, tok_d, mask_d, lb, eps)
    assert SL.surelock_status_poll(a) == 0 and SL.surelock_status_poll(b) == 0
    M = oa.M()
    assert M == ob.M() and 0 < M < B * N
    assert SL.surelock_last_step_paths(a) == SL.surelock_last_step_paths(b)
    assert (SL.surelock_last_step_paths(a) != 0) == (p_lock > 0.5)
    assert torch.equal(oa.active_idx[:M], ob.active_idx[:M])
    assert torch.equal(oa.logits[:M].view(torch.int16), ob.logits[:M].view(torch.int16))
    assert torch.equal(oa.kl[:M].view(torch.int32), ob.kl[:M].view(torch.int32)) and torch.isfinite(oa.kl[:M]).any()
    assert torch.equal(la, lb)
    for l in range(cfg["n_layers"]):
        for x, y in zip(SL.surelock_kv_cache(a, l), SL.surelock_kv_cache(b, l)):
            assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    other = SL.surelock_init(cfg, wd, N + 32, B)
    with pytest.raises(SL.SurelockError):
        SL.surelock_state_import(other, state)
    with pytest.raises(SL.SurelockError):
        SL.surelock_state_import(b, state[: len(state) // 2])


def test_cache_check_flags_a_locked_position_without_keys_and_values():
    """The "check_cache" switch: a position that enters a step locked although no step ever wrote its K/V (the one
    precondition the host cannot see) is reported as device status 5; legal schedules, a declared pre-fill and an
    imported state pass; surelock_reset invalidates the positions again."""
    cfg = inputs.model_shape("tiny")
    B, N, eps = 2, 96, 1e-3
    wd = to_dev(inputs.make_weights(cfg, 31, dtype=torch.float32))
    ctx = SL.surelock_init(cfg, wd, N, B)
    tokens, mask = inputs.make_tokens(B, N, 40, cfg["vocab"], 31)
    tok_d, mask_d = tokens.to(DEV), mask.to(DEV)
    SL.surelock_set_option(ctx, "check_cache", 1)
    n0 = None
    lock = torch.zeros((B, N), dtype=torch.uint8, device=DEV)
    for t in range(4):                                    # every position is active in the first step: all later locks are legal
        SL.surelock_step(ctx, tok_d, mask_d, lock, eps)
        n0 = SL.surelock_last_launch_count(ctx)
        lock = inputs.bernoulli_lock_schedule(lock.cpu(), mask == 0, 0.3, 700 + t).to(DEV)
    assert SL.surelock_status_poll(ctx) == 0
    SL.surelock_set_option(ctx, "check_cache", 0)
    SL.surelock_step(ctx, tok_d, mask_d, lock.clone(), eps)
    assert SL.surelock_last_launch_count(ctx) == n0 - 1   # the check is one launch, and only when switched on

    SL.surelock_reset(ctx)                                # cache contents are undefined again
    SL.surelock_set_option(ctx, "check_cache", 1)
    lock = torch.zeros((B, N), dtype=torch.uint8, device=DEV)
    lock[1, 7] = 1                                        # locked before any step computed it
    SL.surelock_step(ctx, tok_d, mask_d, lock, eps)
    assert SL.surelock_status_poll(ctx) == 5
    SL.surelock_reset(ctx)                                # clears the status word
    assert SL.surelock_status_poll(ctx) == 0

    SL.surelock_set_option(ctx, "check_cache", 2)         # the caller vouches for the caches (pre-fill)
    lock = torch.zeros((B, N), dtype=torch.uint8, device=DEV)
    lock[1, 7] = 1
    SL.surelock_step(ctx, tok_d, mask_d, lock, eps)
    assert SL.surelock_status_poll(ctx) == 0

    state = SL.surelock_state_export(ctx)                 # an imported state counts as a filled cache
    other = SL.surelock_init(cfg, wd, N, B)
    SL.surelock_set_option(other, "check_cache", 1)
    SL.surelock_state_import(other, state)
    SL.surelock_step(other, tok_d, mask_d, lock, eps)
    assert SL.surelock_status_poll(other) == 0


def test_cuda_core_fallback_is_counted_and_can_be_refused():
    """A bf16 shape the tensor-core kernels do not take (d_ff not a multiple of 8 elements is refused at init, so the
    case here is a head count whose hidden width is not a multiple of 256: the fused QKV launch declines) runs on the
    CUDA-core kernels and is counted; with "strict_tc" the step reports SL_EUNSUPPORTED instead.  The shapes of the
    benchmark configurations never fall back."""
    cfg = inputs.model_shape("tiny", d_model=192, n_heads=3, head_dim=64, d_ff=512, vocab=1024)
    w = to_dev(inputs.make_weights(cfg, 41, dtype=torch.bfloat16, std=0.05))
    B, N = 2, 64
    ctx = SL.surelock_init(cfg, w, N, B)
    tokens, mask = inputs.make_tokens(B, N, 32, cfg["vocab"], 41)
    lock = torch.zeros((B, N), dtype=torch.uint8, device=DEV)
    SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0
    assert SL.surelock_last_fallback_count(ctx) == cfg["n_layers"]            # the fused QKV launch of every layer
    SL.surelock_reset(ctx)
    assert SL.surelock_last_fallback_count(ctx) == 0
    SL.surelock_set_option(ctx, "strict_tc", 1)
    with pytest.raises(SL.SurelockError, match="not supported"):
        SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), lock, 1e-3)
    # a shape every tensor-core kernel takes never falls back
    cfg2 = inputs.model_shape("tiny")
    ctx2 = SL.surelock_init(cfg2, to_dev(inputs.make_weights(cfg2, 42, dtype=torch.bfloat16)), N, B)
    SL.surelock_set_option(ctx2, "strict_tc", 1)
    tokens2, mask2 = inputs.make_tokens(B, N, 32, cfg2["vocab"], 42)
    SL.surelock_step(ctx2, tokens2.to(DEV), mask2.to(DEV), lock, 1e-3)
    assert SL.surelock_status_poll(ctx2) == 0 and SL.surelock_last_fallback_count(ctx2) == 0


@pytest.mark.gpu
def test_layer_chain_grid_barrier_wait_runs_out_and_is_reported():
    """Failure detection without a fault, in the persistent layer chain kernel: one CTA is told to skip the first grid
    barrier of the next launch, so every other CTA's bounded wait (about 1 s) runs out; all roles leave, tensor memory is
    freed, the kernel returns and the step reports device status 2.  Nothing hangs or traps: after surelock_reset the same
    context repeats, bit for bit, what a fresh context computes."""
    import time
    cfg = inputs.model_shape("llada8b", n_layers=1, vocab=4096)
    w = inputs.make_weights(cfg, 77, dtype=torch.bfloat16, device=DEV)
    B, N = 1, 256
    tokens, mask = inputs.make_tokens(B, N, 64, cfg["vocab"], 77)
    tokens, mask = tokens.to(DEV), mask.to(DEV)
    lock = inputs.random_lock(B, N, [20], 78).to(DEV)

    def two_steps(ctx, diag):
        SL.surelock_step(ctx, tokens, mask, torch.zeros((B, N), dtype=torch.uint8, device=DEV), 1e-3)
        SL.surelock_set_option(ctx, "row_bound", 20)
        if diag:
            SL.surelock_set_option(ctx, "debug_chain_skip_barrier", 5 + 1)
        l1 = lock.clone()
        out = SL.surelock_step(ctx, tokens, mask, l1, 1e-3)
        return out, l1

    ctx = SL.surelock_init(cfg, w, N, B)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    two_steps(ctx, True)
    st = SL.surelock_status_poll(ctx)                                # synchronises
    waited = time.perf_counter() - t0
    assert st == 2                                                   # a bounded wait of a GEMM kernel ran out
    assert SL.surelock_last_step_paths(ctx) & 1
    assert 0.3 < waited < 20.0, waited                               # it did wait, and the wait did end
    SL.surelock_reset(ctx)
    SL.surelock_set_option(ctx, "row_bound", 0)
    out_a, lock_a = two_steps(ctx, False)
    assert SL.surelock_status_poll(ctx) == 0
    logits_a = out_a.logits[:20].clone()
    ctx2 = SL.surelock_init(cfg, w, N, B)
    out_b, lock_b = two_steps(ctx2, False)
    assert SL.surelock_status_poll(ctx2) == 0
    assert torch.equal(logits_a.view(torch.int16), out_b.logits[:20].view(torch.int16)) and torch.equal(lock_a, lock_b)


@pytest.mark.gpu
def test_few_row_kernels_with_no_active_row():
    """A step whose bound on the row count selects the layer chain kernel and the split-key attention, but in which
    every position is locked (M = 0): the kernels run as empty launches, nothing is written (caches, lock mask), no
    status is raised; one active row right after works too."""
    cfg = inputs.model_shape("llada8b", n_layers=2, vocab=4096)
    w = inputs.make_weights(cfg, 5, dtype=torch.bfloat16, device=DEV)
    B, N = 1, 256
    ctx = SL.surelock_init(cfg, w, N, B)
    tokens, mask = inputs.make_tokens(B, N, 64, cfg["vocab"], 5)
    tokens, mask = tokens.to(DEV), mask.to(DEV)
    SL.surelock_step(ctx, tokens, mask, torch.zeros((B, N), dtype=torch.uint8, device=DEV), 1e-3)
    SL.surelock_set_option(ctx, "row_bound", 16)
    snap = [[t.clone() for t in SL.surelock_kv_cache(ctx, l)] for l in range(cfg["n_layers"])]
    lock = torch.ones((B, N), dtype=torch.uint8, device=DEV)
    out = SL.surelock_step(ctx, tokens, mask, lock, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0 and SL.surelock_last_step_paths(ctx) == 3
    assert int(out.n_active.item()) == 0 and bool(lock.all())
    for l in range(cfg["n_layers"]):
        k, v = SL.surelock_kv_cache(ctx, l)
        assert torch.equal(k.view(torch.int16), snap[l][0].view(torch.int16))
        assert torch.equal(v.view(torch.int16), snap[l][1].view(torch.int16))
    lock1 = inputs.random_lock(B, N, [1], 9).to(DEV)
    out = SL.surelock_step(ctx, tokens, mask, lock1, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0 and int(out.n_active.item()) == 1
    assert bool(torch.isfinite(out.logits[:1].float()).all())
