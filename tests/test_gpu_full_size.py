"""Sampled parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times.

Three layers of each workload are built exactly as the benchmark builds them (GPU-generated values, real block tables,
permuted pages where the workload says so); the outputs of the shortest, longest, first and last sequence are
compared with the oracle run on the wire bytes copied back from the device."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["qwen3-8b-b64-ctx4k", "qwen3-14b-b128-lognormal", "qwen3-32b-b32-ctx8k", "qwen3-32b-b256-trace"])
def test_sampled_parity_full_batch(name):
    import bench
    from paper_2606_29986_b200 import hma
    wl = bench.Workload(name, torch.device("cuda", 0), with_bf16=False, with_ingest=False, layers=3)
    from helpers import parity_sample
    res = parity_sample(wl)
    print(name, res)
    assert len(res) >= 2
    for r in res:
        assert r["f32_max_abs"] <= 1e-2 and r["f32_rel_l2"] <= 2e-3, (name, r)      # the bar, literally, on the F32 output
        assert r["bf16_is_rne_of_f32"], (name, r)                                     # BF16 output = exact rounding of it
        assert r["planned_equals_self_planned"], (name, r)
        assert r["bf16_max_abs"] <= 1e-2 + 2.0 ** -8 * 25.0, (name, r)
        # rel-L2 of the BF16 output: the literal bar where the oracle's own rounded result meets it, else within 5 % of that floor
        assert r["bf16_rel_l2"] <= (2e-3 if r["bf16_floor_rel_l2"] <= 1.9e-3 else 1.05 * r["bf16_floor_rel_l2"]), (name, r)
    assert hma.hma_error_flags(wl.caches["bfp8"]) == 0
    # the read probe moves the same records without touching the outputs
    before = wl.out.view(torch.int16).clone()
    hma.hma_kv_read_probe(wl.caches["bfp8"], 0, wl.table, wl.ctx, wl.workspace)
    torch.cuda.synchronize()
    assert torch.equal(before, wl.out.view(torch.int16))


def test_longest_supported_context_and_limits():
    from paper_2606_29986_b200 import hma
    from helpers import Scenario, check_attention, bf16_bits
    sc = Scenario([32768, 17], 64, 8, seed=77, permute=True)
    ref64, _ = sc.oracle()
    check_attention(sc.attention(0, torch.float32).cpu().numpy(), bf16_bits(sc.attention(0, torch.bfloat16)), ref64)
    # a batch beyond the kernel's limit is refused, not mis-run
    big = 5000
    q = torch.zeros((big, 64, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    tbl = torch.zeros((big, 1), dtype=torch.int32, device="cuda")
    ctx = torch.zeros(big, dtype=torch.int32, device="cuda")
    ws = hma.new_workspace(sc.desc, big)
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention(sc.cache, 0, q, out, tbl, ctx, 0.1, ws)
    assert e.value.status == hma.HMA_ERR_UNSUPPORTED_SHAPE
    # 1024 empty sequences are fine: every row is zero
    q2, out2 = q[:1024], torch.ones((1024, 64, 128), dtype=torch.bfloat16, device="cuda")
    hma.hma_decode_attention(sc.cache, 0, q2, out2, tbl[:1024], ctx[:1024], 0.1, ws)
    torch.cuda.synchronize()
    assert not out2.any()


def test_sampled_parity_full_batch_several_query_tokens_and_two_caches():
    """The headline workload through the planned forms of hma_decode_attention_multi (two query tokens per sequence) and of
    hma_decode_attention_mixed (64 BF16 tail tokens per sequence), compared with the oracle on the sampled sequences."""
    import bench
    from oracle import oracle as orc
    from paper_2606_29986_b200 import hma, synth
    from helpers import bf16_bits
    dev = torch.device("cuda", 0)
    wl = bench.Workload("qwen3-32b-b32-ctx8k", dev, with_bf16=False, with_ingest=False, layers=2)
    c = wl.caches["bfp8"]
    rel = lambda x, ref: float(np.sqrt(((x - ref) ** 2).sum() / (ref ** 2).sum()))
    # ---- two query tokens per sequence
    q2 = synth.make_q(wl.B * 2, wl.hq, 777, dev).view(wl.B, 2, wl.hq, 128)
    out2 = torch.full((wl.B, 2, wl.hq, 128), float("nan"), dtype=torch.float32, device=dev)
    ws2 = hma.new_workspace(c.desc, wl.B * 2, dev)
    plan2 = hma.hma_decode_attention_plan(c, wl.table, wl.ctx, q_len=2)
    # ---- two caches: 64 tail tokens per sequence in a BF16 cache
    S = 64
    tl = np.full(wl.B, S, np.int32)
    ttab_np, tpages, _ = synth.block_table(tl, True, 5)
    tail = hma.KVCache(hma.make_desc(wl.L, wl.hq, wl.hkv, tpages, hma.HMA_KV_BF16), dev, fill=0xFF)
    ttab, tlens = torch.from_numpy(ttab_np).to(dev), torch.from_numpy(tl).to(dev)
    g = torch.Generator(device=dev)
    g.manual_seed(5)
    tk = torch.randn((wl.L, wl.B, wl.hkv, S, 128), generator=g, device=dev).to(torch.bfloat16)
    tv = (torch.randn((wl.L, wl.B, wl.hkv, S, 128), generator=g, device=dev) * 3).to(torch.bfloat16)
    for l in range(wl.L):
        for b in range(wl.B):
            hma.hma_kv_ingest_layer(tail, l, tk[l, b].contiguous(), tv[l, b].contiguous(), hma.HMA_WIRE_BF16_ROWS, 0, wl.hkv,
                                    ttab[b].contiguous(), 0, S)
    wsm = hma.new_workspace(c.desc, wl.B, dev, copies=2)
    pplan = hma.hma_decode_attention_plan(c, wl.table, wl.ctx)
    tplan = hma.hma_decode_attention_plan(tail, ttab, tlens)
    outm = torch.full((wl.B, wl.hq, 128), float("nan"), dtype=torch.float32, device=dev)
    checked = 0
    for (l, b), (kw, vw) in sorted(wl.sample_wires.items()):
        hma.hma_decode_attention_planned(c, l, q2, out2, wl.table, wl.ctx, wl.sm_scale, plan2, ws2)
        hma.hma_decode_attention_mixed_planned(c, tail, l, wl.q[l], outm, wl.table, wl.ctx, ttab, tlens, wl.sm_scale, pplan, tplan, wsm)
        torch.cuda.synchronize(dev)
        ref2, _ = orc.decode_attention_multi(bf16_bits(q2[b:b + 1]), [kw], [vw], wl.hkv, wl.sm_scale)
        got2 = out2[b].cpu().numpy().astype(np.float64)
        assert np.abs(got2 - ref2[0]).max() <= 1e-2 and rel(got2, ref2[0]) <= 2e-3, (l, b, np.abs(got2 - ref2[0]).max(), rel(got2, ref2[0]))
        refm, _ = orc.decode_attention_mixed(bf16_bits(wl.q[l][b:b + 1]), [kw], [vw], [bf16_bits(tk[l, b])], [bf16_bits(tv[l, b])],
                                             wl.hkv, wl.sm_scale)
        gotm = outm[b].cpu().numpy().astype(np.float64)
        assert np.abs(gotm - refm[0]).max() <= 1e-2 and rel(gotm, refm[0]) <= 2e-3, (l, b, np.abs(gotm - refm[0]).max(), rel(gotm, refm[0]))
        checked += 1
    assert checked >= 2
    assert hma.hma_error_flags(c) == 0 and hma.hma_error_flags(tail) == 0
