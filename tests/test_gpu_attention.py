"""GPU parity, floating point: fused BFP8 paged decode attention against the fp64 oracle."""
import numpy as np
import pytest
import torch

from paper_2606_29986_b200 import hma, synth
from helpers import Scenario, bf16_bits, bf16_bits_to_f64, check_attention, parity_metrics

pytestmark = pytest.mark.gpu


def _run_and_check(sc, layer=0, sm_scale=None):
    ref64, _ = sc.oracle(layer, sm_scale)
    o32 = sc.attention(layer, torch.float32, sm_scale=sm_scale).cpu().numpy()
    o16 = bf16_bits(sc.attention(layer, torch.bfloat16, sm_scale=sm_scale))
    return check_attention(o32, o16, ref64), ref64, o32, o16


def test_workload_qwen3_4b_full():
    """Config 1 in full: 32 q / 8 kv heads, batch 4, context 1024, outlier channels, seed 0."""
    w = synth.WORKLOADS["qwen3-4b-b4-ctx1k"]
    lens = synth.context_lens(w["ctx"], w["batch"], 0)
    sc = Scenario(lens, w["hq"], w["hkv"], seed=0)
    (ma, rl, mb, rb), ref64, o32, o16 = _run_and_check(sc)
    print("config1 parity: f32 max-abs %.3e rel-L2 %.3e | bf16 max-abs %.3e rel-L2 %.3e" % (ma, rl, mb, rb))
    # floor: the oracle's own result rounded to BF16
    _, ref16 = sc.oracle()
    print("bf16 rounding floor: max-abs %.3e rel-L2 %.3e" % parity_metrics(bf16_bits_to_f64(ref16), ref64))
    assert hma.hma_error_flags(sc.cache) == 0


@pytest.mark.parametrize("hq,hkv", [(8, 8), (8, 4), (16, 4), (40, 8), (64, 8), (24, 8), (7, 1)])
def test_ragged_contexts_and_group_sizes(hq, hkv):
    lens = [1, 15, 16, 17, 31, 33, 0, 200, 48, 5]
    sc = Scenario(lens, hq, hkv, seed=hq * 13 + hkv, permute=True)
    _, ref64, o32, o16 = _run_and_check(sc)
    assert not o32[6].any() and not o16[6].any()          # empty context -> zeros
    # T = 1 returns V exactly
    from oracle import oracle as orc
    v = orc.decode_rowmajor_f64(sc.v_wires[0][0])
    G = hq // hkv
    for h in range(hq):
        assert np.array_equal(bf16_bits_to_f64(o16[0, h]), v[h // G, 0])


def test_simple_kernel_and_bf16_cache_agree_with_oracle():
    lens = [70, 16, 129, 0, 3]
    for fmt in (hma.HMA_KV_BFP8, hma.HMA_KV_BF16):
        sc = Scenario(lens, 32, 8, seed=21, permute=True, fmt=fmt)
        ref64, _ = sc.oracle()
        o32 = sc.attention(0, torch.float32, simple=True).cpu().numpy()
        o16 = bf16_bits(sc.attention(0, torch.bfloat16, simple=True))
        check_attention(o32, o16, ref64)
        if fmt == hma.HMA_KV_BF16:
            check_attention(sc.attention(0, torch.float32).cpu().numpy(), bf16_bits(sc.attention(0, torch.bfloat16)), ref64)


@pytest.mark.parametrize("hq,hkv", [(64, 8), (40, 8), (8, 8), (4, 1)])
def test_bf16_cache_tensor_core_path(hq, hkv):
    """The same values in a BF16 cache (filled by the decoding ingest) through the BF16 variant of the fused kernel."""
    lens = [1, 15, 16, 17, 33, 0, 700, 48, 5000]
    sc = Scenario(lens, hq, hkv, seed=hq + 3 * hkv, permute=True, fmt=hma.HMA_KV_BF16, fill=0xFF)
    _, ref64, o32, o16 = _run_and_check(sc)
    assert not o32[5].any()
    again = bf16_bits(sc.attention(0, torch.bfloat16))
    assert np.array_equal(again, o16)
    twin = Scenario(lens, hq, hkv, seed=hq + 3 * hkv, permute=True, fmt=hma.HMA_KV_BFP8)
    t32 = twin.attention(0, torch.float32).cpu().numpy()
    assert np.abs(t32 - o32).max() <= 5e-3           # BFP8 path and BF16 path see identical values
    assert hma.hma_error_flags(sc.cache) == 0


@pytest.mark.parametrize("fmt", [hma.HMA_KV_BFP8, hma.HMA_KV_BF16])
def test_interleaved_rotary_keys(fmt):
    """Keys cached in the prefill accelerator's interleaved rotary order, queries in half-split order (key re-layout)."""
    lens = [33, 700, 16, 0, 2100]
    sc = Scenario(lens, 40, 8, seed=91, permute=True, fmt=fmt, key_layout=hma.HMA_KEYS_INTERLEAVED)
    _, ref64, o32, _ = _run_and_check(sc)
    plain = Scenario(lens, 40, 8, seed=91, permute=True, fmt=fmt)
    assert np.abs(plain.attention(0, torch.float32).cpu().numpy() - o32).max() > 0.1      # the layout flag matters
    simple = sc.attention(0, torch.float32, simple=True).cpu().numpy()
    assert np.abs(simple - o32).max() <= 5e-3
    # the one-shot rebuild hands the keys over in half-split order; values are untouched
    from oracle import oracle as orc
    T = lens[1]
    pages = sc.table[1, :(T + 15) // 16].contiguous()
    for which, wires in ((0, sc.k_wires), (1, sc.v_wires)):
        out = torch.zeros((T, 8, 128), dtype=torch.bfloat16, device="cuda")
        hma.hma_bfp8_dequant_bf16(sc.cache, 0, which, pages, 0, T, out)
        torch.cuda.synchronize()
        want = orc.decode_rowmajor_bf16(wires[0][1])
        if which == 0:
            want = orc.relayout_keys_to_half_split(want)
        assert np.array_equal(bf16_bits(out).transpose(1, 0, 2), want), which


def test_long_context_many_splits_and_determinism():
    """One long sequence is cut across every CTA (split-K), short ones sit inside a single CTA."""
    lens = [6000, 40, 2500, 16]
    sc = Scenario(lens, 64, 8, seed=31, permute=True)
    _, ref64, o32, o16 = _run_and_check(sc)
    again = bf16_bits(sc.attention(0, torch.bfloat16))
    assert np.array_equal(again, o16)                      # fixed reduction order: bitwise repeatable
    simple = sc.attention(0, torch.float32, simple=True).cpu().numpy()
    assert np.abs(simple - o32).max() <= 5e-3


def test_page_permutation_and_tail_garbage_change_nothing():
    lens = [100, 37, 260]
    a = Scenario(lens, 32, 8, seed=41, permute=False, fill=0x00)
    b = Scenario(lens, 32, 8, seed=41, permute=True, fill=0xFF)     # other physical pages, 0xFF in every unwritten byte
    oa, ob = a.attention(0, torch.float32).cpu().numpy(), b.attention(0, torch.float32).cpu().numpy()
    assert np.array_equal(oa, ob)
    assert np.isfinite(ob).all()


def test_sm_scale_and_q_range():
    lens = [90, 33]
    sc = Scenario(lens, 16, 4, seed=51)
    _run_and_check(sc, sm_scale=0.3)
    # huge and tiny queries: the per-head power-of-two scaling keeps FP16 operands in range
    for scale in (3.0e4, 1.0e-6):
        q = (sc.q.float() * scale).to(torch.bfloat16)
        ref64, _ = sc.oracle(q=q, sm_scale=0.05 / scale)
        o32 = sc.attention(0, torch.float32, q=q, sm_scale=0.05 / scale).cpu().numpy()
        ma, rl = parity_metrics(o32, ref64)
        assert ma <= 1e-2 and rl <= 2e-3, (scale, ma, rl)


def test_wide_exponent_spread_in_v():
    """V blocks whose exponents differ by 2^40 between tokens: the running reference exponent must track them."""
    sc = Scenario([64], 8, 1, seed=61, extra_pages=0)
    kw, vw = sc.k_wires[0][0].copy(), sc.v_wires[0][0].copy()
    rng = np.random.default_rng(61)
    vw[0, :, :8] = rng.integers(90, 170, (64, 8)).astype(np.uint8)
    kw[0, :, :8] = rng.integers(120, 130, (64, 8)).astype(np.uint8)
    hma.hma_kv_ingest_layer(sc.cache, 0, torch.from_numpy(kw).cuda(), torch.from_numpy(vw).cuda(), hma.HMA_WIRE_ROWMAJOR, 0, 1,
                            sc.table[0, :4].contiguous(), 0, 64)
    sc.k_wires[0][0], sc.v_wires[0][0] = kw, vw
    ref64, _ = sc.oracle()
    o32 = sc.attention(0, torch.float32).cpu().numpy().astype(np.float64)
    # per 16-channel block the scale differs by many orders of magnitude: compare block by block, relatively
    for j in range(8):
        r, g = ref64[0, :, 16 * j:16 * j + 16], o32[0, :, 16 * j:16 * j + 16]
        assert np.sqrt(((g - r) ** 2).sum() / (r ** 2).sum()) <= 2e-3, j


def test_bad_page_id_is_skipped_and_flagged():
    sc = Scenario([64, 64], 8, 2, seed=71)
    good = sc.attention(0, torch.float32).cpu().numpy()
    assert hma.hma_error_flags(sc.cache) == 0
    tbl = sc.table.clone()
    tbl[1, 2] = sc.num_pages + 100
    saved, sc.table = sc.table, tbl
    out = sc.attention(0, torch.float32).cpu().numpy()
    assert hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_PAGE_ATTENTION
    assert np.isfinite(out).all() and np.array_equal(out[0], good[0])
    # the result equals attention over the remaining 48 tokens of sequence 1
    from oracle import oracle as orc
    keep = np.r_[0:32, 48:64]
    ref, _ = orc.decode_attention(bf16_bits(sc.q[1:2]), [sc.k_wires[0][1][:, keep]], [sc.v_wires[0][1][:, keep]], 2)
    assert parity_metrics(out[1:2], ref)[1] <= 2e-3
    sc.table = saved


def test_argument_errors():
    sc = Scenario([32], 8, 2, seed=81)
    out = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device="cuda")
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention(sc.cache, 0, sc.q, out, sc.table, sc.ctx, 0.1, small)
    assert e.value.status == hma.HMA_ERR_WORKSPACE_TOO_SMALL
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention(sc.cache, 3, sc.q, out, sc.table, sc.ctx, 0.1, sc.workspace)
    assert e.value.status == hma.HMA_ERR_INVALID_ARG
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention(sc.cache, 0, sc.q.view(-1)[1:].view(torch.bfloat16), out, sc.table, sc.ctx, 0.1, sc.workspace)
    assert e.value.status == hma.HMA_ERR_ALIGNMENT


def test_concurrent_ingest_on_a_side_stream_leaves_decode_untouched():
    """A new request's layers land in spare pages on a side stream while decode runs: decode output stays bitwise the
    same, and afterwards the new request attends and rebuilds correctly (section 3.2: transfer overlaps compute)."""
    from oracle import oracle as orc
    lens = [3000, 1500, 700, 4000]
    new_T = 1000
    sc = Scenario(lens, 32, 8, seed=111, permute=True, layers=2, extra_pages=(new_T + 15) // 16)
    quiet = [bf16_bits(sc.attention(l, torch.bfloat16)) for l in range(2)]
    kw = [synth.make_kv_wire(8, new_T, 7000 + l) for l in range(2)]
    vw = [synth.make_kv_wire(8, new_T, 7100 + l) for l in range(2)]
    kt = [[synth.rowmajor_to_tile32(w[2 * s:2 * s + 2].contiguous()).cuda() for s in range(4)] for w in kw]
    vt = [[synth.rowmajor_to_tile32(w[2 * s:2 * s + 2].contiguous()).cuda() for s in range(4)] for w in vw]
    spare = torch.from_numpy(np.ascontiguousarray(sc.spare)).cuda()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    outs = []
    for rep in range(6):
        for l in range(2):
            hma.hma_kv_ingest_layer_shards(sc.cache, l, kt[l], vt[l], hma.HMA_WIRE_TILE32, [0, 2, 4, 6], [2] * 4, spare, 0, new_T, side)
            out = torch.empty((len(lens), 32, 128), dtype=torch.bfloat16, device="cuda")
            hma.hma_decode_attention(sc.cache, l, sc.q, out, sc.table, sc.ctx, 1.0 / np.sqrt(128.0), sc.workspace)
            outs.append((l, out))
    torch.cuda.synchronize()
    for l, out in outs:
        assert np.array_equal(bf16_bits(out), quiet[l])
    assert hma.hma_error_flags(sc.cache) == 0
    # the request that arrived meanwhile joins the batch
    table = torch.full((1, spare.numel()), -1, dtype=torch.int32, device="cuda")
    table[0] = spare
    ctx = torch.tensor([new_T], dtype=torch.int32, device="cuda")
    q = synth.make_q(1, 32, 112).cuda()
    for l in range(2):
        out = torch.empty((1, 32, 128), dtype=torch.float32, device="cuda")
        hma.hma_decode_attention(sc.cache, l, q, out, table, ctx, 1.0 / np.sqrt(128.0), sc.workspace)
        torch.cuda.synchronize()
        ref64, _ = orc.decode_attention(bf16_bits(q), [kw[l].numpy()], [vw[l].numpy()], 8)
        ma, rl = parity_metrics(out.cpu().numpy(), ref64)
        assert ma <= 1e-2 and rl <= 2e-3


def test_context_longer_than_the_block_table_is_clamped_and_many_kv_heads():
    """context_lens beyond max_pages_per_seq * 16 are clamped to what the table can address; 16 kv heads work."""
    from oracle import oracle as orc
    sc = Scenario([64, 48], 32, 16, seed=121)
    ctx = torch.tensor([10_000, 48], dtype=torch.int32, device="cuda")       # the table has 4 pages per sequence
    out = torch.empty((2, 32, 128), dtype=torch.float32, device="cuda")
    hma.hma_decode_attention(sc.cache, 0, sc.q, out, sc.table, ctx, 1.0 / np.sqrt(128.0), sc.workspace)
    torch.cuda.synchronize()
    ref64, _ = sc.oracle()
    ma, rl = parity_metrics(out.cpu().numpy(), ref64)
    assert ma <= 1e-2 and rl <= 2e-3 and hma.hma_error_flags(sc.cache) == 0
    neg = torch.tensor([-5, 48], dtype=torch.int32, device="cuda")           # a negative length counts as empty
    hma.hma_decode_attention(sc.cache, 0, sc.q, out, sc.table, neg, 1.0 / np.sqrt(128.0), sc.workspace)
    torch.cuda.synchronize()
    assert not out[0].any() and parity_metrics(out[1:].cpu().numpy(), ref64[1:])[1] <= 2e-3
