"""Stage-wise (teacher-forced) parity of the bf16 path inside the whole step, up to the full benchmark size.

Every stage is checked with the GPU's OWN input to that stage, so the bf16 rounding of earlier stages does not
accumulate into the comparison and the 2e-2 bar applies stage by stage:
  * K/V written by a layer  = oracle QKV + RoPE of that layer's traced block input          (rows a3-a6)
  * attention sub-block     = traced block input + oracle attention (over the GPU's cache: fresh + frozen rows)
                              through the O-projection                                         (rows a7, a8)
  * FFN sub-block           = oracle RMSNorm + SwiGLU FFN + residual of the traced input of that sub-block (a3, a9, a10)
  * logits                  = oracle final norm + LM head of the traced last block output     (rows a3, a11)
  * KL / conf / argmax / lock decisions = oracle formulas on the logits the GPU materialised  (row a12)
  * active_idx / row_offsets / M bit-exact                                                     (row a1)
At the full size (LLaDA-8B shape, batch 8, N = 1536, the configuration bench.py times) the oracle computes a
seeded sample of layers, sequences and rows one by one.
"""
import numpy as np
import pytest
import torch

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import binding as SL
from paper_2602_06412_b200 import inputs
from tests.parity_util import f64, rel_err_rows, to_dev

pytestmark = pytest.mark.gpu
DEV = "cuda"
TOL = 2e-2


def _ti(a):
    return torch.from_numpy(np.asarray(a)).long().to(DEV)


def _np_layer(lw):
    return {k: v.detach().to("cpu", torch.float32).numpy() for k, v in lw.items()}


def tile_covering_sample(r0, r1, n_rows, rng):
    """Rows (relative to r0) of the packed range [r0, r1) of one sequence: one seeded row out of every 128-row tile of
    the GLOBAL packed order that the range touches (the GEMMs' row tiles; every second one is the peer CTA of a
    256-row pair tile), one out of every 128-row tile counted from r0 (the attention kernel's query tiles), the first
    and the last row, and seeded extra rows up to n_rows."""
    rows = {0, r1 - r0 - 1}
    for t in range(r0 // 128, (r1 - 1) // 128 + 1):
        lo, hi = max(t * 128, r0), min((t + 1) * 128, r1)
        rows.add(int(rng.integers(lo, hi)) - r0)
    for lo in range(0, r1 - r0, 128):
        rows.add(int(rng.integers(lo, min(lo + 128, r1 - r0))))
    while len(rows) < min(n_rows, r1 - r0):
        rows.add(int(rng.integers(0, r1 - r0)))
    return np.array(sorted(rows), dtype=np.int64)


def _check_step(cfg, w_dev, ctx, out, lock_in, mask, kl_eps, prev_logits_view, prev_row_of_pos, layers, seqs, n_rows,
                seed, lock_after, tokens=None):
    oc = O.ModelCfg(**cfg)
    B, N, L = ctx.B, ctx.N, cfg["n_layers"]
    idx, offs = O.active_set(lock_in.numpy())
    M = out.M()
    assert M == len(idx)
    assert np.array_equal(out.active_idx[:M].cpu().numpy(), idx)
    assert np.array_equal(out.row_offsets.cpu().numpy(), offs)
    trace = SL.surelock_layer_trace(ctx)
    rng = np.random.default_rng(seed)
    worst = dict(kv=0.0, attn=0.0, ffn=0.0, logits=0.0, kl=0.0)
    sample_rows = {}
    for b in seqs:
        r0, r1 = int(offs[b]), int(offs[b + 1])
        if r1 > r0:
            sample_rows[b] = tile_covering_sample(r0, r1, n_rows, rng)
    if tokens is not None:
        # the block input of the first layer is the embedding of the active rows' tokens (Algorithm 1 line 7): a copy,
        # compared bit for bit (the fp32 stream holds the bf16 table entry widened: its bits shifted left by 16)
        emb_bits = w_dev["tok_emb"].view(torch.int16).cpu().numpy().astype(np.int32)
        tok = tokens.cpu().numpy().reshape(-1)
        got = trace[0, :M].view(torch.int32).cpu().numpy()
        assert np.array_equal(got, emb_bits[tok[idx]] << 16)
    for l in layers:
        lw = _np_layer(w_dev["layers"][l])
        kg, vg = SL.surelock_kv_cache(ctx, l)
        for b, S in sample_rows.items():
            r0, r1 = int(offs[b]), int(offs[b + 1])
            pos = (idx[r0:r1] - b * N).astype(np.int64)
            x_in = f64(trace[2 * l, r0:r1])
            q, k, v = O.qkv_rows(oc, lw, x_in, pos)
            Kg, Vg = f64(kg[b * N:(b + 1) * N]), f64(vg[b * N:(b + 1) * N])
            worst["kv"] = max(worst["kv"], rel_err_rows(Kg[pos].reshape(len(pos), -1), k.reshape(len(pos), -1)),
                              rel_err_rows(Vg[pos].reshape(len(pos), -1), v.reshape(len(pos), -1)))
            o = O.attention_rows(q[S], Kg, Vg)
            x1 = x_in[S] + o @ np.asarray(lw["wo"], np.float64).T
            x_mid = f64(trace[2 * l + 1, r0:r1][_ti(S)])                       # the GPU's input to the FFN sub-block
            worst["attn"] = max(worst["attn"], rel_err_rows(x_mid, x1))
            x2 = O.ffn_rows(oc, lw, x_mid)
            worst["ffn"] = max(worst["ffn"], rel_err_rows(f64(trace[2 * l + 2, r0:r1][_ti(S)]), x2))
    # final norm + LM head on sampled rows
    rows = np.concatenate([int(offs[b]) + S for b, S in sample_rows.items()])
    head = w_dev["lm_head"].detach().to("cpu", torch.float32).numpy()
    gain = w_dev["final_norm_g"].detach().to("cpu", torch.float32).numpy()
    ref_logits = O.rmsnorm(f64(trace[2 * L][_ti(rows)]), gain, cfg["rms_eps"]) @ np.asarray(head, np.float64).T
    g_logits = f64(out.logits[_ti(rows)])
    worst["logits"] = rel_err_rows(g_logits, ref_logits)
    # softmax / KL / lock test on the GPU's own logits
    conf_ref, am_ref = O.posterior_stats(g_logits)
    assert np.array_equal(out.argmax[_ti(rows)].cpu().numpy(), am_ref)
    np.testing.assert_allclose(out.conf[_ti(rows)].cpu().numpy(), conf_ref, rtol=1e-4)
    kl_gpu = out.kl[_ti(rows)].cpu().numpy().astype(np.float64)
    pos_flat = idx[rows]
    if prev_logits_view is None:
        assert np.all(np.isinf(kl_gpu))
        kl_ref = np.full(len(rows), np.inf)
    else:
        prow = prev_row_of_pos[pos_flat]
        assert np.all(prow >= 0)
        kl_ref = O.kl_from_logits(g_logits, f64(prev_logits_view[_ti(prow)]))
        err = np.abs(kl_gpu - kl_ref)
        assert np.all(err <= 1e-3 * kl_ref + 1e-9), err.max()
        worst["kl"] = float(np.max(err / (kl_ref + 1e-30) * (kl_ref > 1e-6)))
    want = O.sure_test(kl_ref, mask.numpy().reshape(-1)[pos_flat], kl_eps)
    near = np.isfinite(kl_ref) & (np.abs(kl_ref - kl_eps) <= 1e-3 * kl_eps)
    got = lock_after.cpu().numpy().reshape(-1)[pos_flat].astype(bool)
    assert np.array_equal(got[~near], want[~near])
    assert max(worst["kv"], worst["attn"], worst["ffn"], worst["logits"]) < TOL, worst
    return worst


def _two_steps(cfg, B, N, n_prompt, n_active, seed, layers, seqs, n_rows, std=0.02, w_device="cpu",
               lock_fn=inputs.random_lock, row_bound_after_first=0, option="gemm_stream", expect_paths=None):
    w = inputs.make_weights(cfg, seed, dtype=torch.bfloat16, std=std, device=w_device)
    w_dev = w if w_device != "cpu" else to_dev(w)
    ctx = SL.surelock_init(cfg, w_dev, N, B)
    SL.surelock_set_option(ctx, "trace_layers", 1)
    tokens, mask = inputs.make_tokens(B, N, n_prompt, cfg["vocab"], seed)
    lock0 = torch.zeros((B, N), dtype=torch.uint8)
    l0 = lock0.to(DEV)
    out0 = SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), l0, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0
    w0 = _check_step(cfg, w_dev, ctx, out0, lock0, mask, 1e-3, None, None, layers, seqs, n_rows, seed, l0, tokens=tokens)
    assert not l0.any()                                              # first step: D = inf, nothing locks
    prev_rop = np.arange(B * N, dtype=np.int64)                      # step 0 packed every position in order
    snap = [[t.clone() for t in SL.surelock_kv_cache(ctx, l)] for l in layers]
    # the sampler reveals some tokens, the caller forces a ragged lock pattern
    tok2 = tokens.clone()
    g = torch.Generator().manual_seed(seed)
    for b in range(B):
        tok2[b, n_prompt:n_prompt + 8] = torch.randint(0, cfg["vocab"] - 1, (8,), generator=g, dtype=torch.int32)
    mask2 = mask.clone()
    mask2[:, n_prompt:n_prompt + 8] = 0
    lock1 = lock_fn(B, N, n_active, seed + 1)
    l1 = lock1.to(DEV)
    if row_bound_after_first:
        SL.surelock_set_option(ctx, option, 1)
        if option != "layer_chain":
            SL.surelock_set_option(ctx, "layer_chain", 0)          # so that the kernel under test really runs
        SL.surelock_set_option(ctx, "row_bound", row_bound_after_first)
    out1 = SL.surelock_step(ctx, tok2.to(DEV), mask2.to(DEV), l1, 1e-3)
    assert SL.surelock_status_poll(ctx) == 0
    if expect_paths is not None:                                     # the few-row kernels under test really ran
        assert SL.surelock_last_step_paths(ctx) == expect_paths
    w1 = _check_step(cfg, w_dev, ctx, out1, lock1, mask2, 1e-3, out0.logits, prev_rop, layers, seqs, n_rows, seed + 7, l1,
                     tokens=tok2)
    locked = lock1.reshape(-1).bool().to(DEV)
    for i, l in enumerate(layers):                                   # frozen rows: bytes unchanged by the second step
        k, v = SL.surelock_kv_cache(ctx, l)
        assert torch.equal(k[locked].view(torch.int16), snap[i][0][locked].view(torch.int16))
        assert torch.equal(v[locked].view(torch.int16), snap[i][1][locked].view(torch.int16))
    assert torch.all(l1.cpu() >= lock1)
    return w0, w1


def test_small_model_every_layer_every_row():
    cfg = inputs.model_shape("tiny", d_model=512, n_heads=4, head_dim=128, d_ff=1536, vocab=4096, n_layers=3)
    _two_steps(cfg, B=3, N=200, n_prompt=90, n_active=[150, 37, 1], seed=31, layers=[0, 1, 2], seqs=[0, 1, 2],
               n_rows=200, std=0.04)


def test_head_dim_64_model():
    cfg = inputs.model_shape("tiny", n_layers=2)
    _two_steps(cfg, B=2, N=300, n_prompt=100, n_active=[300, 130], seed=32, layers=[0, 1], seqs=[0, 1], n_rows=300,
               std=0.05)


def test_llada8b_full_size_sampled():
    """The configuration bench.py times: 32 layers, d=4096, vocab 126464, batch 8, N=1536, ragged active sets."""
    cfg = inputs.model_shape("llada8b")
    B, N = 8, 1536
    na = [int(N * 0.5 * f) for f in (1.3, 0.7, 1.0, 0.9, 1.25, 0.75, 1.1, 1.0)]
    w0, w1 = _two_steps(cfg, B=B, N=N, n_prompt=512, n_active=na, seed=33, layers=[0, 13, 31], seqs=[0, 5], n_rows=16,
                        w_device=DEV)
    print("worst stage errors, full size:", w0, w1)


def test_long_context_contiguous_plus_random_locks():
    """Attention-dominated shape: LLaDA-8B layer shape (2 layers), batch 4, N = 4096, 5 % active rows under the
    contiguous-prefix-plus-random lock pattern (one sequence keeps a single active row)."""
    cfg = inputs.model_shape("llada8b", n_layers=2, vocab=8192)
    B, N = 4, 4096
    na = [int(N * 0.05), int(N * 0.065), 1, int(N * 0.035)]
    w0, w1 = _two_steps(cfg, B=B, N=N, n_prompt=3584, n_active=na, seed=41, layers=[0, 1], seqs=[0, 2, 3], n_rows=8,
                        w_device=DEV, lock_fn=inputs.contiguous_plus_random_lock)
    print("worst stage errors, long context:", w0, w1)


@pytest.mark.parametrize("n_active", [[23], [103], [305]])
def test_single_sequence_few_active_rows(n_active):
    """Weight-streaming regime of the GEMMs (single sequence, N = 512, LLaDA-8B layer shape, 2 layers): M = 23 and 103
    take one row tile (32 / 128 activation rows per stage, K split with the fused QKV, SwiGLU and residual epilogues
    finishing in the workspace), M = 305 three row tiles."""
    cfg = inputs.model_shape("llada8b", n_layers=2, vocab=8192)
    w0, w1 = _two_steps(cfg, B=1, N=512, n_prompt=128, n_active=n_active, seed=50 + n_active[0], layers=[0, 1], seqs=[0],
                        n_rows=12, w_device=DEV)
    print("worst stage errors, single sequence:", n_active, w0, w1)


@pytest.mark.parametrize("n_active,bound", [([23], 23), ([103], 128), ([60], 16), ([9, 1, 14], 32)])
def test_weight_streaming_step_with_a_row_bound(n_active, bound):
    """The step with the "gemm_stream" and "row_bound" options set, so that the second step (M <= 128) runs every contraction
    (fused QKV with rotary embedding and cache scatter, output projection, SwiGLU, down projection, LM head) on the
    weight-streaming kernel; bound 16 with 60 active rows makes that kernel take four passes over the weights."""
    cfg = inputs.model_shape("llada8b", n_layers=2, vocab=8192)
    B = len(n_active)
    w0, w1 = _two_steps(cfg, B=B, N=512, n_prompt=128, n_active=n_active, seed=90 + n_active[0], layers=[0, 1],
                        seqs=list(range(B)), n_rows=12, w_device=DEV, row_bound_after_first=bound)
    print("worst stage errors, weight streaming:", n_active, bound, w0, w1)


@pytest.mark.parametrize("n_active,bound", [([23], 23), ([9, 1, 14], 32), ([60], 64), ([5], 16), ([60], 16), ([101], 128), ([70, 50], 120), ([150], 128)])
def test_layer_chain_step_with_a_row_bound(n_active, bound):
    """The step with the "layer_chain" option (on by default for bounds of at most 128 rows): in the second step the output projection, the SwiGLU FFN and
    the next layer's Q/K/V projections (rotary embedding, cache scatter) of every layer run as one persistent kernel with
    the RMSNorms folded in; stage by stage against the oracle from the traced inputs, like the kernel-per-contraction path.
    Bound 16 with 60 active rows (128 with 150): the bound was too small, the kernel makes four (two) passes and still
    computes every row."""
    cfg = inputs.model_shape("llada8b", n_layers=3, vocab=8192)
    B = len(n_active)
    w0, w1 = _two_steps(cfg, B=B, N=512, n_prompt=128, n_active=n_active, seed=190 + n_active[0], layers=[0, 1, 2],
                        seqs=list(range(B)), n_rows=12, w_device=DEV, row_bound_after_first=bound, option="layer_chain",
                        expect_paths=3 if B <= 2 else 1)
    print("worst stage errors, layer chain:", n_active, bound, w0, w1)


@pytest.mark.gpu
@pytest.mark.parametrize("N,n_active", [(700, [40]), (1536, [17]), (300, [90, 30])])
def test_split_key_attention_with_few_rows(N, n_active):
    """Steps with at most 128 active rows and one or two sequences take the attention kernel that splits the keys of a
    (sequence, head) over several CTAs (on by default): a key count that is no multiple of 128 (the last block is
    masked, 6 blocks over 3 splits; 3 blocks over 2), twelve blocks over four splits, two sequences; stage by stage
    against the oracle like every other path."""
    cfg = inputs.model_shape("llada8b", n_layers=2, vocab=8192)
    B = len(n_active)
    w0, w1 = _two_steps(cfg, B=B, N=N, n_prompt=64, n_active=n_active, seed=300 + N, layers=[0, 1], seqs=list(range(B)),
                        n_rows=12, w_device=DEV, row_bound_after_first=sum(n_active), option="layer_chain", expect_paths=3)
    print("worst stage errors, split-key attention:", N, n_active, w0, w1)
