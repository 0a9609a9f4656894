"""hma_decode_attention_static: decode attention for callers that cannot allocate device memory.

Some users of the library have no workspace to hand over: their memory pool was carved up at start-up, or
they run where the surrounding framework forbids allocation.  This entry point keeps its scratch in an
array inside the library.  The test drives it through the C ABI twice in a row, on different batches, and
compares each result with hma_decode_attention given an ordinary workspace, under the same tolerance the
other attention tests use; the second call must not be disturbed by what the first one left in the array.
It also checks that a batch too large for the array is refused.  Collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2606_29986_b200 import hma
from helpers import Scenario, bf16_bits, check_attention

pytestmark = pytest.mark.gpu


def _both(sc, dtype):
    ref = sc.attention(0, dtype)
    out = torch.full_like(ref, float("nan"))
    hma.hma_decode_attention_static(sc.cache, 0, sc.q, out, sc.table, sc.ctx, 1.0 / np.sqrt(128.0))
    torch.cuda.synchronize()
    return ref, out


def test_static_scratch_matches_workspace_entry_point_twice():
    first = Scenario([700, 33, 16, 0, 2100], 32, 8, seed=101, permute=True)
    second = Scenario([90, 4000, 1, 250], 64, 8, seed=102, permute=True)
    for sc in (first, second):                          # two calls in a row on the shared array
        ref64, _ = sc.oracle()
        r32, o32 = _both(sc, torch.float32)
        r16, o16 = _both(sc, torch.bfloat16)
        check_attention(o32.cpu().numpy(), bf16_bits(o16), ref64)
        assert np.abs(o32.cpu().numpy() - r32.cpu().numpy()).max() <= 1e-2
        assert torch.equal(o32, r32) and torch.equal(o16, r16)     # same kernels, same order: identical bits
        assert hma.hma_error_flags(sc.cache) == 0
    # and the first batch again, after the array has held the second one
    r32, o32 = _both(first, torch.float32)
    assert torch.equal(o32, r32)


def test_static_scratch_takes_the_largest_batch_it_promises():
    sc = Scenario([40 + 3 * i for i in range(64)], 16, 8, seed=104, permute=True)      # 64 sequences x 8 kv heads = 512 segments
    ws = hma.hma_decode_attention_workspace_bytes(sc.cache.desc, 64)
    assert ws <= hma.hma_decode_attention_static_limit_bytes() < ws + 2 * 8 * 4160       # 65 sequences would not fit
    r32, o32 = _both(sc, torch.float32)
    assert torch.equal(o32, r32)
    assert hma.hma_error_flags(sc.cache) == 0


def test_static_scratch_rejects_what_does_not_fit():
    assert hma.hma_decode_attention_static_limit_bytes() < 16 * 1024 * 1024
    lens = [16] * 80                                                # 80 sequences x 8 kv heads = 640 segments > 512
    sc = Scenario(lens, 8, 8, seed=103)
    out = torch.zeros((80, 8, 128), dtype=torch.bfloat16, device="cuda")
    n0 = hma.hma_launch_count()
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention_static(sc.cache, 0, sc.q, out, sc.table, sc.ctx, 0.1)
    assert e.value.status == hma.HMA_ERR_STATIC_LIMIT and "scratch" in str(e.value)
    assert hma.hma_launch_count() == n0                             # nothing was enqueued
    sc.attention(0, torch.bfloat16)                                 # the ordinary entry point takes the same batch
