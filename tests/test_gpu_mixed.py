"""GPU parity of attention over a BFP8 prefix cache plus a BF16 tail cache (decode-side KV kept in BF16)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2606_29986_b200 import hma, synth
from helpers import Scenario, bf16_bits, check_attention

pytestmark = pytest.mark.gpu


def _tail_scenario(sc, tail_lens, seed):
    """A BF16 cache holding tail_lens[b] decode-side tokens per sequence, filled with plain BF16 rows."""
    tail_lens = np.asarray(tail_lens, np.int32)
    table_np, num_pages, _ = synth.block_table(tail_lens, True, seed, 2)
    desc = hma.make_desc(1, sc.hq, sc.hkv, num_pages, hma.HMA_KV_BF16)
    cache = hma.KVCache(desc, "cuda", fill=0xFF)          # NaN patterns in everything that is not written
    table = torch.from_numpy(table_np).cuda()
    rng = np.random.default_rng(seed)
    ks, vs = [], []
    for b, S in enumerate(tail_lens):
        S = int(S)
        k = torch.from_numpy(rng.standard_normal((sc.hkv, S, 128)).astype(np.float32)).to(torch.bfloat16)
        v = torch.from_numpy((rng.standard_normal((sc.hkv, S, 128)) * 3).astype(np.float32)).to(torch.bfloat16)
        ks.append(bf16_bits(k))
        vs.append(bf16_bits(v))
        if S:
            # token by token, as a decode loop would append them
            pages = table[b, :(S + 15) // 16].contiguous()
            half = S // 2
            for t0, n in ((0, half), (half, S - half)):
                if n == 0:
                    continue
                first, last = t0 // 16, (t0 + n - 1) // 16
                hma.hma_kv_ingest_layer(cache, 0, k[:, t0:t0 + n].contiguous().cuda(), v[:, t0:t0 + n].contiguous().cuda(),
                                        hma.HMA_WIRE_BF16_ROWS, 0, sc.hkv, pages[first:last + 1].contiguous(), t0, n)
    torch.cuda.synchronize()
    return cache, table, torch.from_numpy(tail_lens).cuda(), ks, vs


@pytest.mark.parametrize("hq,hkv", [(64, 8), (40, 8), (4, 2)])
def test_bfp8_prefix_plus_bf16_tail(hq, hkv):
    prefix_lens = [700, 33, 0, 16, 2500]
    tail_lens = [5, 0, 40, 130, 17]
    sc = Scenario(prefix_lens, hq, hkv, seed=300 + hq, permute=True)
    tail, ttable, tlens, ks, vs = _tail_scenario(sc, tail_lens, 301 + hq)
    ws = hma.new_workspace(sc.desc, sc.B, copies=2)
    ref64, _ = orc.decode_attention_mixed(bf16_bits(sc.q), sc.k_wires[0], sc.v_wires[0], ks, vs, hkv)
    outs = {}
    for dt in (torch.float32, torch.bfloat16):
        out = torch.full((sc.B, hq, 128), float("nan"), dtype=dt, device="cuda")
        hma.hma_decode_attention_mixed(sc.cache, tail, 0, sc.q, out, sc.table, sc.ctx, ttable, tlens, 1.0 / np.sqrt(128.0), ws)
        torch.cuda.synchronize()
        outs[dt] = out
    check_attention(outs[torch.float32].cpu().numpy(), bf16_bits(outs[torch.bfloat16]), ref64)
    assert hma.hma_error_flags(sc.cache) == 0 and hma.hma_error_flags(tail) == 0
    # with empty tails the two-cache call equals the one-cache call up to summation order
    zero = torch.zeros_like(tlens)
    out = torch.empty((sc.B, hq, 128), dtype=torch.float32, device="cuda")
    hma.hma_decode_attention_mixed(sc.cache, tail, 0, sc.q, out, sc.table, sc.ctx, ttable, zero, 1.0 / np.sqrt(128.0), ws)
    torch.cuda.synchronize()
    assert np.abs(out.cpu().numpy() - sc.attention(0, torch.float32).cpu().numpy()).max() <= 2e-3
    assert not out[2].any()                                  # no tokens in either cache


def test_long_tails_short_prefixes_and_a_larger_batch():
    """Tails that several CTAs share (their partials arrive as several tiles per segment), prefixes that one warp holds
    entirely, sequences that live in one cache only; twice on the same workspace."""
    prefix_lens = [112, 3000, 0, 40, 0] + [100 + 13 * i for i in range(19)]
    tail_lens = [2100, 900, 700, 0, 0] + [(7 * i) % 50 for i in range(19)]
    sc = Scenario(prefix_lens, 16, 4, seed=320, permute=True)
    tail, ttable, tlens, ks, vs = _tail_scenario(sc, tail_lens, 321)
    ws = hma.new_workspace(sc.desc, sc.B, copies=2)
    ref64, _ = orc.decode_attention_mixed(bf16_bits(sc.q), sc.k_wires[0], sc.v_wires[0], ks, vs, 4)
    outs = []
    for rep in range(2):
        o32 = torch.full((sc.B, 16, 128), float("nan"), dtype=torch.float32, device="cuda")
        o16 = torch.full((sc.B, 16, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
        hma.hma_decode_attention_mixed(sc.cache, tail, 0, sc.q, o32, sc.table, sc.ctx, ttable, tlens, 1.0 / np.sqrt(128.0), ws)
        hma.hma_decode_attention_mixed(sc.cache, tail, 0, sc.q, o16, sc.table, sc.ctx, ttable, tlens, 1.0 / np.sqrt(128.0), ws)
        torch.cuda.synchronize()
        check_attention(o32.cpu().numpy(), bf16_bits(o16), ref64)
        outs.append(o32)
    assert torch.equal(outs[0], outs[1])                     # fixed orders everywhere: bitwise repeatable
    # with both launches' set-up taken from plans: the same bits
    pplan = hma.hma_decode_attention_plan(sc.cache, sc.table, sc.ctx)
    tplan = hma.hma_decode_attention_plan(tail, ttable, tlens)
    o32 = torch.full((sc.B, 16, 128), float("nan"), dtype=torch.float32, device="cuda")
    hma.hma_decode_attention_mixed_planned(sc.cache, tail, 0, sc.q, o32, sc.table, sc.ctx, ttable, tlens, 1.0 / np.sqrt(128.0), pplan, tplan, ws)
    torch.cuda.synchronize()
    assert torch.equal(o32, outs[0])
    hma.hma_decode_attention_mixed_planned(sc.cache, tail, 0, sc.q, o32, sc.table, sc.ctx, ttable, tlens, 1.0 / np.sqrt(128.0), tplan, pplan, ws)
    torch.cuda.synchronize()                                 # plans swapped: refused
    assert hma.hma_error_flags(tail) | hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_PLAN and torch.equal(o32, outs[0])
    assert not outs[0][4].any()                              # no tokens in either cache
    assert hma.hma_error_flags(sc.cache) == 0 and hma.hma_error_flags(tail) == 0
    # the ordinary one-cache call still finds the workspace's counters at zero
    ws1 = ws[:ws.numel() // 2]
    out = torch.empty((sc.B, 16, 128), dtype=torch.float32, device="cuda")
    hma.hma_decode_attention(sc.cache, 0, sc.q, out, sc.table, sc.ctx, 1.0 / np.sqrt(128.0), ws1)
    torch.cuda.synchronize()
    assert torch.equal(out, sc.attention(0, torch.float32))


def test_bf16_rows_ingest_round_trip_and_rejection():
    sc = Scenario([40], 8, 2, seed=310, fmt=hma.HMA_KV_BF16)
    k = torch.randn((2, 40, 128), generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    v = torch.randn((2, 40, 128), generator=torch.Generator().manual_seed(2)).to(torch.bfloat16)
    pages = sc.table[0, :3].contiguous()
    hma.hma_kv_ingest_layer(sc.cache, 0, k.cuda(), v.cuda(), hma.HMA_WIRE_BF16_ROWS, 0, 2, pages, 0, 40)
    for which, src in ((0, k), (1, v)):
        out = torch.zeros((40, 2, 128), dtype=torch.bfloat16, device="cuda")
        hma.hma_bfp8_dequant_bf16(sc.cache, 0, which, pages, 0, 40, out)
        torch.cuda.synchronize()
        assert torch.equal(out.cpu().transpose(0, 1), src)
    bfp8 = Scenario([40], 8, 2, seed=311)
    with pytest.raises(hma.HmaError) as e:                   # plain BF16 rows cannot enter a BFP8 cache
        hma.hma_kv_ingest_layer(bfp8.cache, 0, k.cuda(), v.cuda(), hma.HMA_WIRE_BF16_ROWS, 0, 2, pages, 0, 40)
    assert e.value.status == hma.HMA_ERR_INVALID_ARG
