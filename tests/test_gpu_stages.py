"""Stage-wise GPU parity: each kernel, called through the C ABI, against the CPU oracle on the same seeded inputs.

Integer and byte work is compared bit for bit; floating point within the stated tolerances:
hidden states / logits / GEMM and attention outputs 2e-2 max relative error (bf16 path; the fp32 path is held to
1e-4), KL 1e-3 relative (plus 1e-9 absolute so that "KL of identical posteriors is 0" is testable), lock
decisions exact except where the oracle's KL lies within 1e-3 relative of the threshold.
"""
import numpy as np
import pytest
import torch

from oracle import surelock_oracle as O
from paper_2602_06412_b200 import binding as SL
from paper_2602_06412_b200 import inputs
from tests.parity_util import f64, rel_err_rows

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _compact(lock):
    B, N = lock.shape
    d = lock.to(DEV).contiguous()
    idx = torch.full((B * N,), -7, dtype=torch.int32, device=DEV)
    offs = torch.full((B + 1,), -7, dtype=torch.int32, device=DEV)
    n = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    rop = torch.full((B * N,), -7, dtype=torch.int32, device=DEV)
    scratch = torch.empty(SL.surelock_compact_scratch_bytes(B * N), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    SL.surelock_compact(d, B, N, idx, offs, n, rop, scratch, status)
    torch.cuda.synchronize()
    assert status.item() == 0
    return idx.cpu().numpy(), offs.cpu().numpy(), int(n.item()), rop.cpu().numpy()


def _check_compact(lock):
    idx, offs, M, rop = _compact(lock)
    ridx, roffs = O.active_set(lock.numpy())
    assert M == len(ridx)
    assert np.array_equal(idx[:M], ridx)
    assert np.array_equal(offs, roffs)
    assert np.all(idx[M:] == -7)                                     # nothing written past M
    want = np.full(lock.numel(), -1, np.int32)
    want[ridx] = np.arange(M, dtype=np.int32)
    assert np.array_equal(rop, want)


@pytest.mark.parametrize("B,N", [(1, 128), (3, 37), (1, 1), (5, 16), (8, 1536), (4, 4096), (2, 4099), (7, 5)])
def test_compact_random(B, N):
    g = torch.Generator().manual_seed(B * 1000 + N)
    for p in (0.5, 0.05, 0.95):
        _check_compact((torch.rand((B, N), generator=g) < p).to(torch.uint8))


def test_compact_degenerate_masks():
    for B, N in [(1, 128), (4, 4096), (3, 37)]:
        _check_compact(torch.zeros((B, N), dtype=torch.uint8))       # nothing locked: M = B*N
        _check_compact(torch.ones((B, N), dtype=torch.uint8))        # everything locked: M = 0
        one = torch.ones((B, N), dtype=torch.uint8)
        one[B - 1, N - 1] = 0
        _check_compact(one)                                          # single active row, the very last flag
        one = torch.zeros((B, N), dtype=torch.uint8)
        one[0, 0] = 1
        _check_compact(one)
    # any non-zero byte counts as locked
    lk = torch.tensor([[0, 2, 0, 255, 0, 1, 0, 0]], dtype=torch.uint8)
    idx, offs, M, _ = _compact(lk)
    assert list(idx[:M]) == [0, 2, 4, 6, 7]


def test_compact_many_chunks_lookback():
    B, N = 3, (1 << 20) + 5                                          # 769 chunks of 4096 flags, ragged tail
    g = torch.Generator().manual_seed(9)
    lock = (torch.rand((B, N), generator=g) < 0.4).to(torch.uint8)
    idx, offs, M, rop = _compact(lock)
    flat = lock.numpy().reshape(-1)
    ref = np.flatnonzero(flat == 0).astype(np.int32)                 # same definition as oracle.active_set, vectorised
    small, _ = O.active_set(lock[:, :2000].numpy())                  # and the oracle itself on a slice
    assert np.array_equal(small, np.concatenate([np.flatnonzero(lock[b, :2000].numpy() == 0) + b * 2000 for b in range(B)]))
    assert M == len(ref) and np.array_equal(idx[:M], ref)
    assert list(offs) == [0] + list(np.cumsum((lock.numpy() == 0).sum(1)))


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_kv_scatter_layout_bit_exact(dtype):
    B, N, H, dh = 2, 300, 4, 64
    lock = inputs.random_lock(B, N, [123, 7], 3)
    idx, _ = O.active_set(lock.numpy())
    M = len(idx)
    g = torch.Generator().manual_seed(1)
    k = torch.randn((B * N, H * dh), generator=g).to(dtype).to(DEV)
    v = torch.randn((B * N, H * dh), generator=g).to(dtype).to(DEV)
    kc0 = torch.randn((B * N, H * dh), generator=g).to(dtype).to(DEV)
    vc0 = torch.randn((B * N, H * dh), generator=g).to(dtype).to(DEV)
    kc, vc = kc0.clone(), vc0.clone()
    SL.surelock_kv_scatter(k, v, torch.from_numpy(idx).to(DEV), torch.tensor([M], dtype=torch.int32, device=DEV), kc, vc)
    torch.cuda.synchronize()
    want_k, want_v = kc0.clone(), vc0.clone()
    li = torch.from_numpy(idx).long().to(DEV)
    want_k[li] = k[:M]
    want_v[li] = v[:M]
    as_bits = lambda t: t.view(torch.int16 if dtype == torch.bfloat16 else torch.int32)
    assert torch.equal(as_bits(kc), as_bits(want_k)) and torch.equal(as_bits(vc), as_bits(want_v))


def _kl_case(rows, V, dtype, seed, eps=1e-3, use_lse=False):
    cur, prev, mask = inputs.kl_logit_pairs(rows, V, seed, dtype=dtype)
    rop = torch.arange(rows, dtype=torch.int32)
    rop[rows // 3] = -1                                              # one row without a previous posterior
    perm = torch.randperm(rows, generator=torch.Generator().manual_seed(seed))
    prev_shuf = torch.empty_like(prev)                               # previous rows live at other packed rows
    prev_shuf[perm] = prev
    rop_pos = torch.where(rop >= 0, perm.to(torch.int32), rop)
    pos = torch.arange(rows, dtype=torch.int32)
    lock = torch.zeros(rows, dtype=torch.uint8)
    d = lambda t: t.to(DEV)
    kl = torch.empty(rows, dtype=torch.float32, device=DEV)
    conf = torch.empty_like(kl)
    am = torch.empty(rows, dtype=torch.int32, device=DEV)
    lse = torch.empty_like(kl)
    lock_d = d(lock)
    n = torch.tensor([rows], dtype=torch.int32, device=DEV)
    prev_lse = None
    if use_lse:                                                      # produce lse of the previous rows with the kernel itself
        pl = torch.empty_like(kl)
        SL.surelock_softmax_kl_sure(d(prev_shuf), None, None, None, None, n, d(torch.ones(rows, dtype=torch.uint8)),
                                    torch.zeros(rows, dtype=torch.uint8, device=DEV), 0.0, kl.clone(), conf.clone(),
                                    am.clone(), pl)
        prev_lse = pl
    SL.surelock_softmax_kl_sure(d(cur), d(prev_shuf), d(rop_pos), prev_lse, d(pos), n, d(mask), lock_d, eps, kl, conf, am, lse)
    torch.cuda.synchronize()
    z, y = f64(cur), f64(prev)
    ref_kl = O.kl_from_logits(z, y)
    ref_kl[rows // 3] = np.inf
    ref_conf, ref_am = O.posterior_stats(z)
    got_kl = kl.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref_kl)
    assert np.all(np.isinf(got_kl[~fin]))
    err = np.abs(got_kl[fin] - ref_kl[fin])
    assert np.all(err <= 1e-3 * ref_kl[fin] + 1e-9), (err.max(), ref_kl[fin][np.argmax(err / (ref_kl[fin] + 1e-30))])
    same = (np.arange(rows) % 20) == 7
    same[rows // 3] = False
    assert np.all(got_kl[same] == 0.0)                               # identical posteriors: exactly 0
    assert np.array_equal(am.cpu().numpy(), ref_am)
    np.testing.assert_allclose(conf.cpu().numpy(), ref_conf, rtol=2e-5)
    np.testing.assert_allclose(lse.cpu().numpy(), (z - O.log_softmax(z))[:, 0], rtol=0, atol=2e-5)
    want = O.sure_test(ref_kl, mask.numpy(), eps)
    near = fin & (np.abs(ref_kl - eps) <= 1e-3 * eps)
    got = lock_d.cpu().numpy().astype(bool)
    assert np.array_equal(got[~near], want[~near])
    assert not got[mask.numpy() == 1].any()
    return got_kl, ref_kl


def test_softmax_kl_sure_llada_vocab_bf16():
    got, ref = _kl_case(96, 126464, torch.bfloat16, 5)
    fin = np.isfinite(ref) & (ref > 0)
    assert ref[fin].min() < 1e-5 and ref[fin].max() > 1e-2           # the case really spans the threshold range


def test_softmax_kl_sure_with_kept_lse():
    _kl_case(40, 126464, torch.bfloat16, 6, use_lse=True)


def test_softmax_kl_sure_small_vocab_fp32_and_bf16():
    _kl_case(33, 2048, torch.float32, 7)
    _kl_case(33, 2048, torch.bfloat16, 8)
    _kl_case(5, 8, torch.bfloat16, 9)                                # a single 128-bit vector per row
    _kl_case(600, 512, torch.float32, 10, eps=5e-5)                  # more rows than CTAs


def test_softmax_kl_sure_first_step_and_empty():
    rows, V = 12, 2048
    cur, prev, mask = inputs.kl_logit_pairs(rows, V, 3, dtype=torch.float32)
    kl = torch.full((rows,), -1.0, device=DEV)
    conf = torch.full((rows,), -1.0, device=DEV)
    am = torch.full((rows,), -1, dtype=torch.int32, device=DEV)
    lock = torch.zeros(rows, dtype=torch.uint8, device=DEV)
    n = torch.tensor([rows], dtype=torch.int32, device=DEV)
    # no previous posterior at all: D = inf, nothing locks (first step)
    SL.surelock_softmax_kl_sure(cur.to(DEV), None, None, None, None, n, torch.zeros(rows, dtype=torch.uint8, device=DEV),
                                lock, 1e9, kl, conf, am)
    torch.cuda.synchronize()
    assert torch.isinf(kl).all() and not lock.any()
    # M = 0: outputs untouched
    kl.fill_(-1.0)
    SL.surelock_softmax_kl_sure(cur.to(DEV), prev.to(DEV), None, None, None, torch.zeros(1, dtype=torch.int32, device=DEV),
                                mask.to(DEV), lock, 1e-3, kl, conf, am)
    torch.cuda.synchronize()
    assert (kl == -1.0).all()


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-4), (torch.bfloat16, 2e-2)])
@pytest.mark.parametrize("M,n_out,K", [(70, 200, 132), (1, 64, 64), (257, 96, 1024)])
def test_gemm_cuda_cores(dtype, tol, M, n_out, K):
    if dtype == torch.bfloat16:
        n_out, K = (n_out + 7) // 8 * 8, (K + 7) // 8 * 8
    g = torch.Generator().manual_seed(M + K)
    A = torch.randn((M + 5, K), generator=g).to(dtype)
    W = (torch.randn((n_out, K), generator=g) * 0.05).to(dtype)
    out = torch.full((M + 5, n_out), 3.0, dtype=dtype, device=DEV)
    SL.surelock_gemm(A.to(DEV), W.to(DEV), out, torch.tensor([M], dtype=torch.int32, device=DEV), impl=1)
    torch.cuda.synchronize()
    ref = f64(A[:M]) @ f64(W).T
    assert rel_err_rows(f64(out[:M]), ref) < tol
    assert (out[M:] == 3.0).all()                                    # rows beyond M untouched


@pytest.mark.parametrize("split", [False, True])
@pytest.mark.parametrize("M,n_out,K", [(1, 256, 64), (100, 256, 256), (128, 512, 4096), (129, 136, 200), (300, 4096, 512),
                                       (1000, 1024, 1024), (0, 256, 256), (32, 4096, 12288), (130, 1024, 8192),
                                       (20, 4096, 4096), (60, 12288, 4096), (128, 4096, 12288), (305, 4096, 12288),
                                       (305, 12288, 4096), (700, 12288, 1024), (638, 4096, 12288), (1534, 4096, 4096)])
def test_gemm_tensor_cores(M, n_out, K, split):
    """Covers every tiling regime: one row tile with 32 / 64 / 128 activation rows per stage and K split (the last
    arriver finishes alone, or the splits of a tile finish it together), a few row tiles with K split, single-CTA tiles
    in one round, CTA pairs."""
    g = torch.Generator().manual_seed(M * 7 + K)
    cap = M + 37
    A = torch.randn((cap, K), generator=g).to(torch.bfloat16)
    W = (torch.randn((n_out, K), generator=g) * 0.05).to(torch.bfloat16)
    out = torch.full((cap, n_out), 3.0, dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    wsp = torch.zeros(SL.surelock_gemm_workspace_bytes(), dtype=torch.uint8, device=DEV) if split else None
    Ad, Wd, n = A.to(DEV), W.to(DEV), torch.tensor([M], dtype=torch.int32, device=DEV)
    SL.surelock_gemm(Ad, Wd, out, n, impl=0, dev_status=status, workspace=wsp)
    torch.cuda.synchronize()
    assert status.item() == 0
    if M:
        ref = f64(A[:M]) @ f64(W).T
        assert rel_err_rows(f64(out[:M]), ref) < 2e-2
    assert (out[M:] == 3.0).all()                                    # rows beyond M untouched
    if split:                                                        # the workspace is left reusable, the result is deterministic
        out2 = torch.full_like(out, 3.0)
        SL.surelock_gemm(Ad, Wd, out2, n, impl=0, dev_status=status, workspace=wsp)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), out2.view(torch.int16))


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("M,n_out,K", [(20, 4096, 4096), (100, 4096, 12288), (128, 4096, 4096), (129, 136, 200), (305, 4096, 4096),
                                       (638, 4096, 4096), (700, 1024, 12288), (1312, 4096, 4096), (0, 256, 256)])
def test_gemm_residual_epilogue(M, n_out, K, impl):
    """x += A W^T into the fp32 residual stream (the output and down projections): every path of the epilogue: plain
    read-modify-write (few activation rows per stage, or a ragged last unit), bulk reductions by the L2 from the
    single-CTA tiles, from the K-split finisher and from the CTA-pair path (one partly filled round, several rounds);
    rows beyond M stay untouched and two runs give the same bits."""
    if impl == 1 and M * n_out * K > 3e10:
        pytest.skip("CUDA-core kernel: small shapes only")
    g = torch.Generator().manual_seed(M * 11 + K)
    cap = M + 37
    A = torch.randn((cap, K), generator=g).to(torch.bfloat16)
    W = (torch.randn((n_out, K), generator=g) * 0.05).to(torch.bfloat16)
    x0 = torch.randn((cap, n_out), generator=g)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    wsp = torch.zeros(SL.surelock_gemm_workspace_bytes(), dtype=torch.uint8, device=DEV)
    Ad, Wd, n = A.to(DEV), W.to(DEV), torch.tensor([M], dtype=torch.int32, device=DEV)
    outs = []
    for _ in range(2):
        x = x0.to(DEV)
        SL.surelock_gemm_fused(Ad, Wd, None, x, n, 1, impl=impl, dev_status=status, workspace=wsp)
        torch.cuda.synchronize()
        outs.append(x)
    assert status.item() == 0
    x = outs[0]
    if M:
        ref = f64(x0[:M]) + f64(A[:M]) @ f64(W).T
        assert rel_err_rows(f64(x[:M]), ref) < (2e-2 if impl == 0 else 1e-4) and torch.isfinite(x[:M]).all()
        # bf16 operands are exact and the sums are fp32: the stream must come out far inside the parity bar
        assert np.abs(f64(x[:M]) - ref).max() < 1e-3 * (1 + np.abs(ref).max())
    assert torch.equal(x[M:].cpu(), x0[M:])                          # rows beyond M untouched, bit for bit
    assert torch.equal(outs[0].view(torch.int32), outs[1].view(torch.int32))


@pytest.mark.parametrize("M,n_out,K", [(20, 1024, 4096), (129, 136, 200), (305, 12288, 1024), (1312, 2048, 4096)])
def test_gemm_swiglu_epilogue(M, n_out, K):
    """silu(A Wg^T) * (A Wu^T) in one launch (gate and up projections), against the oracle's silu."""
    g = torch.Generator().manual_seed(M * 13 + K)
    cap = M + 5
    A = torch.randn((cap, K), generator=g).to(torch.bfloat16)
    Wg = (torch.randn((n_out, K), generator=g) * 0.03).to(torch.bfloat16)
    Wu = (torch.randn((n_out, K), generator=g) * 0.03).to(torch.bfloat16)
    out = torch.full((cap, n_out), 3.0, dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    wsp = torch.zeros(SL.surelock_gemm_workspace_bytes(), dtype=torch.uint8, device=DEV)
    SL.surelock_gemm_fused(A.to(DEV), Wg.to(DEV), Wu.to(DEV), out, torch.tensor([M], dtype=torch.int32, device=DEV), 2,
                           dev_status=status, workspace=wsp)
    torch.cuda.synchronize()
    assert status.item() == 0
    ref = O.silu(f64(A[:M]) @ f64(Wg).T) * (f64(A[:M]) @ f64(Wu).T)
    assert rel_err_rows(f64(out[:M]), ref) < 2e-2
    assert (out[M:] == 3.0).all()
    with pytest.raises(SL.SurelockError):
        SL.surelock_gemm_fused(A.to(DEV), Wg.to(DEV), None, out, torch.tensor([M], dtype=torch.int32, device=DEV), 2)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-4), (torch.bfloat16, 2e-2)])
@pytest.mark.parametrize("B,N,H,dh,n_act", [(2, 77, 3, 64, [20, 77]), (1, 200, 2, 128, [9]), (3, 33, 1, 64, [0, 33, 1])])
def test_attention_cuda_cores(dtype, tol, B, N, H, dh, n_act):
    lock = inputs.random_lock(B, N, n_act, 11)
    idx, offs = O.active_set(lock.numpy())
    M = len(idx)
    g = torch.Generator().manual_seed(N)
    q = torch.randn((B * N, H, dh), generator=g).to(dtype)
    Kc = torch.randn((B * N, H, dh), generator=g).to(dtype)
    Vc = torch.randn((B * N, H, dh), generator=g).to(dtype)
    o = torch.zeros((B * N, H, dh), dtype=dtype, device=DEV)
    SL.surelock_attention(q.to(DEV), Kc.to(DEV), Vc.to(DEV), torch.from_numpy(idx).to(DEV) if M else torch.zeros(1, dtype=torch.int32, device=DEV),
                          torch.from_numpy(offs).to(DEV), torch.tensor([M], dtype=torch.int32, device=DEV), B, N, o, impl=1)
    torch.cuda.synchronize()
    for b in range(B):
        r0, r1 = offs[b], offs[b + 1]
        if r1 == r0:
            continue
        ref = O.attention_rows(f64(q[r0:r1]), f64(Kc[b * N:(b + 1) * N]), f64(Vc[b * N:(b + 1) * N]))
        assert rel_err_rows(f64(o[r0:r1]).reshape(r1 - r0, -1), ref) < tol


@pytest.mark.parametrize("B,N,H,dh,n_act,qscale", [
    (2, 77, 3, 64, [20, 77], 1.0), (1, 200, 2, 128, [9], 1.0), (3, 33, 1, 64, [0, 33, 1], 1.0),
    (2, 300, 2, 128, [300, 150], 1.0), (1, 1536, 4, 128, [700], 1.0), (2, 640, 2, 64, [129, 640], 6.0),
    (1, 1024, 2, 128, [1024], 8.0)])
def test_attention_tensor_cores(B, N, H, dh, n_act, qscale):
    """tcgen05 attention: ragged per-sequence tiles, key counts that are not multiples of the 128-key block, and
    (qscale > 1) score ranges that make the running maximum move so the lazy rescaling of O is exercised."""
    lock = inputs.random_lock(B, N, n_act, 12)
    idx, offs = O.active_set(lock.numpy())
    M = len(idx)
    g = torch.Generator().manual_seed(N + dh)
    q = (torch.randn((B * N, H, dh), generator=g) * qscale).to(torch.bfloat16)
    Kc = torch.randn((B * N, H, dh), generator=g).to(torch.bfloat16)
    Vc = torch.randn((B * N, H, dh), generator=g).to(torch.bfloat16)
    o = torch.full((B * N, H, dh), 5.0, dtype=torch.bfloat16, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    SL.surelock_attention(q.to(DEV), Kc.to(DEV), Vc.to(DEV), torch.from_numpy(idx).to(DEV),
                          torch.from_numpy(offs).to(DEV), torch.tensor([M], dtype=torch.int32, device=DEV), B, N, o, impl=0,
                          dev_status=status)
    torch.cuda.synchronize()
    assert status.item() == 0
    for b in range(B):
        r0, r1 = offs[b], offs[b + 1]
        if r1 == r0:
            continue
        ref = O.attention_rows(f64(q[r0:r1]), f64(Kc[b * N:(b + 1) * N]), f64(Vc[b * N:(b + 1) * N]))
        assert rel_err_rows(f64(o[r0:r1]).reshape(r1 - r0, -1), ref) < 2e-2, (b,)
    assert (o[M:] == 5.0).all()                                      # rows beyond M untouched


def _split_attention_case(B, N, H, dh, n_act, qscale, splits, diag_skip=-1, seed=13):
    lock = inputs.random_lock(B, N, n_act, seed)
    idx, offs = O.active_set(lock.numpy())
    M = len(idx)
    g = torch.Generator().manual_seed(N + dh + seed)
    q = (torch.randn((B * N, H, dh), generator=g) * qscale).to(torch.bfloat16)
    Kc = torch.randn((B * N, H, dh), generator=g).to(torch.bfloat16)
    Vc = torch.randn((B * N, H, dh), generator=g).to(torch.bfloat16)
    o = torch.full((B * N, H, dh), 5.0, dtype=torch.bfloat16, device=DEV)
    ws = torch.zeros(SL.surelock_attention_split_workspace_bytes(B, H, dh), dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    args = (q.to(DEV), Kc.to(DEV), Vc.to(DEV), torch.from_numpy(offs).to(DEV), B, N, o, ws)
    return args, dict(splits=splits, diag_skip=diag_skip, dev_status=status), (q, Kc, Vc, offs, M, o, ws, status)


@pytest.mark.parametrize("B,N,H,dh,n_act,qscale,splits", [
    (1, 512, 32, 128, [23], 1.0, 0), (1, 700, 8, 128, [128], 1.0, 3), (2, 300, 4, 64, [90, 1], 1.0, 0),
    (1, 1024, 2, 128, [64], 8.0, 4), (1, 1536, 4, 128, [150], 6.0, 6), (3, 200, 2, 128, [0, 77, 5], 1.0, 2),
    (1, 128, 2, 64, [7], 1.0, 1), (1, 1000, 16, 128, [33], 1.0, 8)])
def test_attention_split_keys(B, N, H, dh, n_act, qscale, splits):
    """Attention for few query rows with the keys of a (sequence, head) split over several CTAs, alone, against the
    oracle: the number of splits a step would choose (0) and given ones, a key count that is no multiple of 128 (the last
    block masked), score ranges that move the running maximum inside a split (rescaling) and between splits (the
    combination's weights), a sequence without active rows, one with more than 128 (two query tiles, the slots reused
    after a second meeting), a single split (written directly), and a repeat on the same workspace (the counters only
    grow)."""
    args, kw, (q, Kc, Vc, offs, M, o, ws, status) = _split_attention_case(B, N, H, dh, n_act, qscale, splits)
    for rep in range(2):
        o.fill_(5.0)
        SL.surelock_attention_split(*args, **kw)
        torch.cuda.synchronize()
        assert status.item() == 0
        for b in range(B):
            r0, r1 = offs[b], offs[b + 1]
            if r1 == r0:
                continue
            ref = O.attention_rows(f64(q[r0:r1]), f64(Kc[b * N:(b + 1) * N]), f64(Vc[b * N:(b + 1) * N]))
            assert rel_err_rows(f64(o[r0:r1]).reshape(r1 - r0, -1), ref) < 2e-2, (b, rep)
        assert (o[M:] == 5.0).all()                                  # rows beyond M untouched


def test_attention_split_changing_split_count_on_one_workspace():
    """Calls with different numbers of key splits follow one another on the same workspace (a meeting advances the
    pair's counter by the same amount whatever the number of splits)."""
    args, kw, (q, Kc, Vc, offs, M, o, ws, status) = _split_attention_case(1, 1024, 4, 128, [50], 1.0, 2)
    ref = O.attention_rows(f64(q[:M]), f64(Kc[:1024]), f64(Vc[:1024]))
    for splits in (2, 3, 4, 8, 1, 3, 2):
        kw["splits"] = splits
        o.fill_(5.0)
        SL.surelock_attention_split(*args, **kw)
        torch.cuda.synchronize()
        assert status.item() == 0, splits
        assert rel_err_rows(f64(o[:M]).reshape(M, -1), ref) < 2e-2, splits


def test_attention_split_arguments():
    args, kw, _ = _split_attention_case(1, 512, 32, 128, [10], 1.0, 5)
    with pytest.raises(SL.SurelockError):                            # 5 x 32 CTAs do not fit the GPU at one per SM
        SL.surelock_attention_split(*args, **kw)
    args, kw, _ = _split_attention_case(1, 256, 2, 128, [10], 1.0, 2, diag_skip=4)
    with pytest.raises(SL.SurelockError):                            # there is no CTA 4
        SL.surelock_attention_split(*args, **kw)


def test_attention_split_bounded_wait_runs_out_and_is_reported():
    """Failure detection without a fault: one CTA of a (sequence, head) is told not to arrive at the meeting of the
    splits, so its siblings' bounded wait (about 0.2 s) runs out: they store device status 3 (attention timeout) and
    the kernel returns; nothing hangs or traps.  The other heads are computed as usual, and after the workspace has
    been zeroed again the same call gives the oracle's answer."""
    import time
    B, N, H, dh = 1, 512, 4, 128
    args, kw, (q, Kc, Vc, offs, M, o, ws, status) = _split_attention_case(B, N, H, dh, [20], 1.0, 4, diag_skip=4 * 2 + 1)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    SL.surelock_attention_split(*args, **kw)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert status.item() == 3                                        # attention: a bounded wait ran out
    assert 0.05 < waited < 5.0, waited                               # it did wait, and the wait did end
    ref = O.attention_rows(f64(q[:M]), f64(Kc[:N]), f64(Vc[:N]))    # [M][H * dh]
    got = f64(o[:M]).reshape(M, H, dh)
    for h in (0, 1, 3):                                              # head 2 is the one that was left incomplete
        assert rel_err_rows(got[:, h], ref.reshape(M, H, dh)[:, h]) < 2e-2
    status.zero_()
    ws.zero_()
    kw["diag_skip"] = -1
    SL.surelock_attention_split(*args, **kw)
    torch.cuda.synchronize()
    assert status.item() == 0
    assert rel_err_rows(f64(o[:M]).reshape(M, -1), ref) < 2e-2


@pytest.mark.parametrize("B,N,m", [(1, 128, 20.0), (3, 200, 50.0), (4, 4096, 20.0), (2, 33, 0.0), (2, 33, 100.0), (5, 8, 37.5)])
def test_conf_gate_lock(B, N, m):
    """Confidence gate alone: per-sequence percentile threshold and gated lock decisions against the oracle."""
    g = torch.Generator().manual_seed(B * 100 + N)
    n_act = [int(x) for x in torch.randint(0, N + 1, (B,), generator=g)]
    n_act[0] = N
    if B > 1:
        n_act[1] = 0                                                 # a sequence without active rows
    lock = inputs.random_lock(B, N, n_act, 21)
    idx, offs = O.active_set(lock.numpy())
    M = len(idx)
    conf = torch.rand(max(M, 1), generator=g)
    conf[:: 7] = conf[0]                                             # ties
    kl = torch.rand(max(M, 1), generator=g) * 2e-3
    mask = (torch.rand((B, N), generator=g) < 0.4).to(torch.uint8)
    if B > 2:
        mask[2] = 1                                                  # a sequence without candidates
    lock_d = lock.to(DEV)
    theta = torch.full((B,), 7.0, device=DEV)
    SL.surelock_conf_gate_lock(conf.to(DEV), kl.to(DEV), torch.from_numpy(idx).to(DEV) if M else torch.zeros(1, dtype=torch.int32, device=DEV),
                               torch.from_numpy(offs).to(DEV), B, N, mask.to(DEV), lock_d, 1e-3, m, theta)
    torch.cuda.synchronize()
    bb, ii = idx // N, idx % N
    cand = mask.numpy()[bb, ii] == 0
    gate, th = O.confidence_gate(f64(conf[:M]), cand, bb, B, m)
    want = gate & O.sure_test(f64(kl[:M]), mask.numpy()[bb, ii], 1e-3)
    thg = theta.cpu().numpy().astype(np.float64)
    fin = np.isfinite(th)
    assert np.array_equal(np.isfinite(thg), fin) and np.all(thg[~fin] < 0)
    np.testing.assert_allclose(thg[fin], th[fin], rtol=1e-6, atol=1e-7)
    near = np.abs((1.0 - f64(conf[:M])) - th[bb]) <= 1e-6
    new = lock_d.cpu().numpy()
    got = new[bb, ii].astype(bool)
    assert np.array_equal(got[~near], want[~near])
    assert np.array_equal(new[lock.numpy() == 1], lock.numpy()[lock.numpy() == 1])   # locked rows stay locked
    assert not got[~cand].any()


@pytest.mark.parametrize("epi", [0, 1, 2])
@pytest.mark.parametrize("M,n_out,K", [(1, 256, 256), (7, 4096, 4096), (23, 4096, 12288), (32, 12288, 4096), (33, 4096, 4096),
                                       (64, 1024, 8192), (103, 4096, 4096), (128, 4096, 12288), (16, 136, 200), (0, 256, 512)])
def test_gemm_weight_streaming_few_rows(M, n_out, K, epi):
    """The weight-streaming (swapped-operand) kernel (impl = 2; at most 128 rows of activations): every
    row padding (16 / 32 / 64 / 128), cluster sizes 1 ... 8 (K split through distributed shared memory), one and several
    32-row reduction chunks, a ragged feature tile, all three fused epilogues; rows beyond M untouched, two runs give
    the same bits."""
    g = torch.Generator().manual_seed(M * 17 + K + epi)
    cap = max(M, 1)
    A = torch.randn((cap, K), generator=g).to(torch.bfloat16)
    W = (torch.randn((n_out, K), generator=g) * 0.05).to(torch.bfloat16)
    W2 = (torch.randn((n_out, K), generator=g) * 0.05).to(torch.bfloat16) if epi == 2 else None
    x0 = torch.randn((cap, n_out), generator=g)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    Ad, Wd, n = A.to(DEV), W.to(DEV), torch.tensor([M], dtype=torch.int32, device=DEV)
    W2d = W2.to(DEV) if W2 is not None else None
    outs = []
    for _ in range(2):
        out = x0.to(DEV) if epi == 1 else torch.full((cap, n_out), 3.0, dtype=torch.bfloat16, device=DEV)
        SL.surelock_gemm_fused(Ad, Wd, W2d, out, n, epi, impl=2, dev_status=status)
        torch.cuda.synchronize()
        outs.append(out)
    assert status.item() == 0
    out = outs[0]
    if M:
        acc = f64(A[:M]) @ f64(W).T
        ref = acc if epi == 0 else (f64(x0[:M]) + acc if epi == 1 else O.silu(acc) * (f64(A[:M]) @ f64(W2).T))
        assert rel_err_rows(f64(out[:M]), ref) < 2e-2
        if epi == 1:
            assert np.abs(f64(out[:M]) - ref).max() < 1e-3 * (1 + np.abs(ref).max())
    if epi == 1:
        assert torch.equal(out[M:].cpu(), x0[M:])
        assert torch.equal(outs[0].view(torch.int32), outs[1].view(torch.int32))
    else:
        assert (out[M:] == 3.0).all()
        assert torch.equal(outs[0].view(torch.int16), outs[1].view(torch.int16))


def test_gemm_weight_streaming_refuses_what_it_does_not_take():
    A = torch.zeros((200, 256), dtype=torch.bfloat16, device=DEV)
    W = torch.zeros((256, 256), dtype=torch.bfloat16, device=DEV)
    out = torch.zeros((200, 256), dtype=torch.bfloat16, device=DEV)
    n = torch.tensor([5], dtype=torch.int32, device=DEV)
    with pytest.raises(SL.SurelockError, match="not supported"):
        SL.surelock_gemm(A, W, out, n, impl=2)                       # more than 128 rows of capacity
    with pytest.raises(SL.SurelockError, match="not supported"):
        SL.surelock_gemm(A[:8].float(), W.float(), out[:8].float(), n, impl=2)   # fp32


def test_compaction_bounded_wait_runs_out_and_is_reported():
    """Failure detection without a fault: the compaction is launched with its chunk tickets starting at 1, so the
    count of chunk 0 is never published and every running chunk's look-back polls into its bound (about 70 ms), stores
    device status 1 and returns.  Nothing hangs or traps; the same buffers then serve a normal call, whose result is
    right, and a context on the same device still steps."""
    import time
    B, N = 1, 3 * 4096 + 100                                         # four chunks: three of them run and wait
    g = torch.Generator().manual_seed(3)
    lock = (torch.rand((B, N), generator=g) < 0.5).to(torch.uint8)
    d = lock.to(DEV)
    idx = torch.full((B * N,), -7, dtype=torch.int32, device=DEV)
    offs = torch.full((B + 1,), -7, dtype=torch.int32, device=DEV)
    n = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    rop = torch.full((B * N,), -7, dtype=torch.int32, device=DEV)
    scratch = torch.empty(SL.surelock_compact_scratch_bytes(B * N) + 64, dtype=torch.uint8, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    SL.surelock_compact_from_ticket(d, B, N, idx, offs, n, rop, scratch, 1, status)
    torch.cuda.synchronize()
    waited = time.perf_counter() - t0
    assert status.item() == 1                                        # SL_DEV_COMPACT_TIMEOUT
    assert 0.02 < waited < 5.0, waited                               # it did wait, and the wait did end
    # the device is fine: the ordinary call on the same buffers gives the oracle's answer
    status.zero_()
    SL.surelock_compact(d, B, N, idx, offs, n, rop, scratch, status)
    torch.cuda.synchronize()
    ridx, roffs = O.active_set(lock.numpy())
    assert status.item() == 0 and int(n.item()) == len(ridx)
    assert np.array_equal(idx[:len(ridx)].cpu().numpy(), ridx) and np.array_equal(offs.cpu().numpy(), roffs)
    # first_ticket = 0 is the ordinary compaction
    idx2 = torch.full_like(idx, -7)
    SL.surelock_compact_from_ticket(d, B, N, idx2, offs, n, rop, scratch, 0, status)
    torch.cuda.synchronize()
    assert status.item() == 0 and torch.equal(idx2[:len(ridx)], idx[:len(ridx)])
    # and a context created afterwards works
    cfg = inputs.model_shape("tiny")
    from tests.parity_util import to_dev
    ctx = SL.surelock_init(cfg, to_dev(inputs.make_weights(cfg, 2, dtype=torch.float32)), 64, 1)
    tokens, mask = inputs.make_tokens(1, 64, 32, cfg["vocab"], 2)
    SL.surelock_step(ctx, tokens.to(DEV), mask.to(DEV), torch.zeros((1, 64), dtype=torch.uint8, device=DEV), 1e-3)
    assert SL.surelock_status_poll(ctx) == 0
