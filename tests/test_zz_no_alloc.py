"""The allocation-free compaction entry point gives the same results as the ordinary one.

`surelock_compact_noalloc` exists for callers that are given buffers but may not allocate device memory (a plug-in
inside a process whose pool allocator owns all memory, or a loop that cannot afford cudaMalloc's device-wide
synchronisation); its scratch words live in a fixed array inside the library.  Because that array is shared by all
calls and keeps the last call's contents, the test makes two calls in a row with different masks and sizes and
compares each, bit for bit, with `surelock_compact`, which gets fresh caller-provided scratch.  This file is named
so that pytest collects it last: a run that stops at the first failure has then already run every other test.
"""
import pytest
import torch

from paper_2602_06412_b200 import binding as SL

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run(fn_noalloc, lock):
    B, N = lock.shape
    d = lock.to(DEV)
    outs = []
    for noalloc in (False, True):
        idx = torch.full((B * N,), -3, dtype=torch.int32, device=DEV)
        offs = torch.full((B + 1,), -3, dtype=torch.int32, device=DEV)
        n = torch.full((1,), -3, dtype=torch.int32, device=DEV)
        rop = torch.full((B * N,), -3, dtype=torch.int32, device=DEV)
        status = torch.zeros(1, dtype=torch.int32, device=DEV)
        if noalloc:
            SL.surelock_compact_noalloc(d, B, N, idx, offs, n, rop, status)
        else:
            scratch = torch.empty(SL.surelock_compact_scratch_bytes(B * N), dtype=torch.uint8, device=DEV)
            SL.surelock_compact(d, B, N, idx, offs, n, rop, scratch, status)
        torch.cuda.synchronize()
        assert status.item() == 0
        outs.append((idx, offs, n, rop))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    return int(outs[1][2].item())


def test_noalloc_compaction_matches_on_two_calls_in_a_row():
    g = torch.Generator().manual_seed(77)
    first = (torch.rand((5, 40000), generator=g) < 0.3).to(torch.uint8)      # 49 chunks, ragged tail
    second = (torch.rand((3, 1537), generator=g) < 0.7).to(torch.uint8)      # fewer chunks: stale words stay behind
    m1 = _run(SL.surelock_compact_noalloc, first)
    m2 = _run(SL.surelock_compact_noalloc, second)
    assert m1 == int((first == 0).sum()) and m2 == int((second == 0).sum())
    m3 = _run(SL.surelock_compact_noalloc, first)                            # and growing again
    assert m3 == m1


def test_noalloc_compaction_rejects_sizes_beyond_its_capacity():
    cap = SL.surelock_compact_noalloc_max_flags()
    assert cap == 1 << 24
    B, N = 2, cap // 2 + 1
    one = torch.zeros(16, dtype=torch.uint8, device=DEV)                     # never read: the call must refuse first
    i32 = torch.zeros(16, dtype=torch.int32, device=DEV)
    with pytest.raises(SL.SurelockError, match="capacity"):
        SL.surelock_compact_noalloc(one, B, N, i32, i32, i32, None, None)


def test_noalloc_compaction_takes_no_device_memory():
    """The property in the name: after a warm-up call (which also fetches the array's address), further calls leave
    the amount of free device memory exactly where it was."""
    g = torch.Generator().manual_seed(78)
    lock = (torch.rand((4, 30000), generator=g) < 0.5).to(torch.uint8).to(DEV)
    B, N = lock.shape
    idx = torch.empty(B * N, dtype=torch.int32, device=DEV)
    offs = torch.empty(B + 1, dtype=torch.int32, device=DEV)
    n = torch.empty(1, dtype=torch.int32, device=DEV)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    SL.surelock_compact_noalloc(lock, B, N, idx, offs, n, None, status)          # warm-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        SL.surelock_compact_noalloc(lock, B, N, idx, offs, n, None, status)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0 and status.item() == 0
    assert int(n.item()) == int((lock == 0).sum())
