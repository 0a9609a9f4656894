"""hma_decode_attention_plan / hma_decode_attention_planned: the kernel's set-up computed once per decode step.

The planned call must give, bit for bit, what the self-planning call gives (same kernel body, same work split; when no
segment is longer than 8 pages the plan cuts the work differently and the results agree within the kernel's own error), for one and for
several query tokens per sequence and for both cache formats, and stay within the oracle's tolerance; a plan made for
another launch shape must be refused without touching the outputs.
"""
import numpy as np
import pytest
import torch

from paper_2606_29986_b200 import hma
from helpers import Scenario, bf16_bits, check_attention

pytestmark = pytest.mark.gpu
SCALE = 1.0 / np.sqrt(128.0)


@pytest.mark.parametrize("fmt", [hma.HMA_KV_BFP8, hma.HMA_KV_BF16])
@pytest.mark.parametrize("lens,hq,hkv", [([700, 33, 16, 0, 2100, 5, 300], 32, 8), ([1] * 40 + [47] * 9, 8, 2), ([0, 0, 5000], 40, 8)])
def test_planned_call_equals_self_planned_call(fmt, lens, hq, hkv):
    sc = Scenario(lens, hq, hkv, seed=400 + hq, permute=True, fmt=fmt, layers=2)
    plan = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx)
    assert plan.numel() == hma.hma_decode_attention_plan_bytes(sc.B)
    ref64, _ = sc.oracle(1)
    for layer in (0, 1):                                   # one plan serves every layer
        for dt in (torch.float32, torch.bfloat16):
            ref = sc.attention(layer, dt)
            out = torch.full_like(ref, float("nan"))
            hma.hma_decode_attention_planned(sc.cache, layer, sc.q, out, sc.table, sc.ctx, SCALE, plan, sc.workspace)
            torch.cuda.synchronize()
            if max(lens) > 128:
                assert torch.equal(out.view(torch.int16 if dt == torch.bfloat16 else torch.int32),
                                   ref.view(torch.int16 if dt == torch.bfloat16 else torch.int32))
            else:
                # no segment longer than 8 pages: the plan gives every segment to one warp, the self-planning call cuts them
                # up; the FP16 softmax weights are then rounded against other running maxima, so the two results agree within
                # the kernel's own error (both are checked against the oracle below), not to the bit
                assert float((out.float() - ref.float()).abs().max()) <= (5e-3 if dt == torch.float32 else 2.0 ** -6)
            if layer == 1 and dt == torch.float32:
                o32 = out
            if layer == 1 and dt == torch.bfloat16:
                o16 = out
    check_attention(o32.cpu().numpy(), bf16_bits(o16), ref64)
    assert hma.hma_error_flags(sc.cache) == 0
    # the workspace's counters are back at zero: the self-planning call still works on it
    assert torch.equal(sc.attention(0, torch.float32), sc.attention(0, torch.float32))


@pytest.mark.parametrize("q_len", [2, 3, 4])
def test_planned_call_with_several_query_tokens(q_len):
    sc = Scenario([300, 17, 64, 1000, q_len], 16, 4, seed=410 + q_len, permute=True)
    g = torch.Generator(device="cuda")
    g.manual_seed(7)
    q = torch.randn((sc.B, q_len, 16, 128), generator=g, device="cuda").to(torch.bfloat16)
    ws = hma.new_workspace(sc.desc, sc.B * q_len)
    ref = torch.full((sc.B, q_len, 16, 128), float("nan"), dtype=torch.float32, device="cuda")
    hma.hma_decode_attention_multi(sc.cache, 0, q, ref, sc.table, sc.ctx, SCALE, ws)
    plan = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx, q_len=q_len)
    out = torch.full_like(ref, float("nan"))
    hma.hma_decode_attention_planned(sc.cache, 0, q, out, sc.table, sc.ctx, SCALE, plan, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int32), ref.view(torch.int32))
    assert hma.hma_error_flags(sc.cache) == 0


def test_a_plan_for_another_shape_is_refused():
    sc = Scenario([200, 50, 900], 16, 4, seed=420, permute=True)
    other = Scenario([200, 50, 900, 10], 16, 4, seed=421, permute=True)
    plan_other = hma.hma_decode_attention_plan(other.cache, other.table, other.ctx)
    out = torch.full((sc.B, 16, 128), 7.0, dtype=torch.float32, device="cuda")
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, plan_other, sc.workspace)
    torch.cuda.synchronize()
    assert hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_PLAN      # read and cleared
    assert bool((out == 7.0).all())                                     # nothing was computed
    # a plan for two query tokens does not fit a one-token call either, nor a buffer that was never planned into
    plan2 = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx, q_len=2)
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, plan2, sc.workspace)
    blank = torch.zeros(hma.hma_decode_attention_plan_bytes(sc.B), dtype=torch.uint8, device="cuda")
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, blank, sc.workspace)
    torch.cuda.synchronize()
    assert hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_PLAN and bool((out == 7.0).all())
    # and the right plan afterwards works on the same workspace
    plan = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx)
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, plan, sc.workspace)
    torch.cuda.synchronize()
    assert torch.equal(out, sc.attention(0, torch.float32)) and hma.hma_error_flags(sc.cache) == 0


def test_a_plan_lasts_until_a_sequence_starts_a_new_page():
    sc = Scenario([200, 50, 900, 33], 16, 4, seed=440, permute=True)
    plan = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx)
    # shorter contexts inside the same pages (as if the plan had been made a few decode steps ago): still the right plan
    ctx = torch.tensor([195, 49, 897, 33], dtype=torch.int32, device="cuda")
    ref = torch.empty((sc.B, 16, 128), dtype=torch.float32, device="cuda")
    out = torch.empty_like(ref)
    hma.hma_decode_attention(sc.cache, 0, sc.q, ref, sc.table, ctx, SCALE, sc.workspace)
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, ctx, SCALE, plan, sc.workspace)
    torch.cuda.synchronize()
    assert torch.equal(out, ref) and hma.hma_error_flags(sc.cache) == 0
    assert not torch.equal(ref, sc.attention(0, torch.float32))          # and the lengths did matter
    # one sequence a page shorter: the plan no longer fits, the call says so (and stays inside its memory)
    ctx[2] = 880
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, ctx, SCALE, plan, sc.workspace)
    torch.cuda.synchronize()
    assert hma.hma_error_flags(sc.cache) & hma.HMA_FLAG_BAD_PLAN          # (a page without a valid token may raise more)
    hma.hma_decode_attention_workspace_init(sc.workspace)                 # a void call may leave counters behind
    assert torch.equal(sc.attention(0, torch.float32), sc.attention(0, torch.float32))


def test_plan_argument_checks():
    sc = Scenario([40], 8, 2, seed=430)
    need = hma.hma_decode_attention_plan_bytes(1)
    assert need > 0 and hma.hma_decode_attention_plan_bytes(-1) == 0 and hma.hma_decode_attention_plan_bytes(5000) == 0
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx, plan=small)
    assert e.value.status == hma.HMA_ERR_WORKSPACE_TOO_SMALL
    big = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx, plan=big[16:])
    assert e.value.status == hma.HMA_ERR_ALIGNMENT
    out = torch.empty((1, 8, 128), dtype=torch.float32, device="cuda")
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, None, sc.workspace)
    assert e.value.status == hma.HMA_ERR_INVALID_ARG
    n0 = hma.hma_launch_count()
    plan = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx)
    hma.hma_decode_attention_planned(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, plan, sc.workspace)
    assert hma.hma_launch_count() == n0 + 2                             # one plan launch, one attention launch
