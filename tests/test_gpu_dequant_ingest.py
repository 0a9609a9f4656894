"""GPU parity, bytes: flat and paged BFP8 -> BF16 reconstruction and the ingest scatter, bit-exact against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2606_29986_b200 import hma, synth
from helpers import Scenario, bf16_bits

pytestmark = pytest.mark.gpu


def test_flat_dequant_exhaustive_table():
    E = np.repeat(np.arange(256, dtype=np.uint8), 16)
    m = np.tile(np.arange(256, dtype=np.uint8), 256).reshape(-1, 16)
    out = torch.zeros(E.size * 16, dtype=torch.bfloat16, device="cuda")
    hma.hma_bfp8_dequant_blocks_bf16(torch.from_numpy(E).cuda(), torch.from_numpy(m).cuda(), E.size, out)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(out).reshape(-1, 16), orc.bfp8_decode_bf16(E, m))


def test_flat_dequant_random_ragged_sizes():
    rng = np.random.default_rng(0)
    for n in (1, 7, 255, 100003):
        E = rng.integers(0, 256, n).astype(np.uint8)
        m = rng.integers(0, 256, (n, 16)).astype(np.uint8)
        out = torch.zeros(n * 16 + 16, dtype=torch.bfloat16, device="cuda")
        hma.hma_bfp8_dequant_blocks_bf16(torch.from_numpy(E).cuda(), torch.from_numpy(m).cuda(), n, out)
        torch.cuda.synchronize()
        got = bf16_bits(out)
        assert np.array_equal(got[:n * 16].reshape(-1, 16), orc.bfp8_decode_bf16(E, m))
        assert not got[n * 16:].any()
    hma.hma_bfp8_dequant_blocks_bf16(None, None, 0, None)     # empty input is a no-op


def _dequant_all(sc, layer, which, b):
    T = int(sc.lens[b])
    out = torch.zeros((T, sc.hkv, 128), dtype=torch.bfloat16, device="cuda")
    if T:
        hma.hma_bfp8_dequant_bf16(sc.cache, layer, which, sc.table[b, :(T + 15) // 16].contiguous(), 0, T, out)
    torch.cuda.synchronize()
    return bf16_bits(out).transpose(1, 0, 2)          # -> [Hkv][T][128]


@pytest.mark.parametrize("fmt", [hma.HMA_KV_BFP8, hma.HMA_KV_BF16])
@pytest.mark.parametrize("layout,shards", [(hma.HMA_WIRE_ROWMAJOR, 1), (hma.HMA_WIRE_TILE32, 1), (hma.HMA_WIRE_TILE32, 4),
                                           (hma.HMA_WIRE_ROWMAJOR, 2)])
def test_ingest_then_paged_dequant_equals_oracle_decode(fmt, layout, shards):
    sc = Scenario([1, 15, 16, 17, 33, 100, 0, 64], 32, 8, seed=3, permute=True, fmt=fmt, wire_layout=layout, shards=shards, layers=2)
    for l in range(2):
        for b in range(sc.B):
            for which, wires in ((0, sc.k_wires), (1, sc.v_wires)):
                assert np.array_equal(_dequant_all(sc, l, which, b), orc.decode_rowmajor_bf16(wires[l][b])), (l, b, which)
    assert hma.hma_error_flags(sc.cache) == 0


@pytest.mark.parametrize("fmt", [hma.HMA_KV_BFP8, hma.HMA_KV_BF16])
@pytest.mark.parametrize("layout", [hma.HMA_WIRE_ROWMAJOR, hma.HMA_WIRE_TILE32])
def test_partial_range_ingest_keeps_other_bytes(fmt, layout):
    """Overwrite tokens [21, 21+45) of a 100-token sequence: those change, everything else is byte-identical."""
    sc = Scenario([100, 40], 16, 4, seed=5, permute=True, fmt=fmt, layers=1)
    before = [t.clone() for t in sc.cache.layers]
    t0, n = 21, 45
    new_k = synth.make_kv_wire(4, n, 991)
    new_v = synth.make_kv_wire(4, n, 992)
    first, last = t0 // 16, (t0 + n - 1) // 16
    pages = sc.table[0, first:last + 1].contiguous()
    kk, vv = (new_k, new_v) if layout == hma.HMA_WIRE_ROWMAJOR else (synth.rowmajor_to_tile32(new_k), synth.rowmajor_to_tile32(new_v))
    hma.hma_kv_ingest_layer(sc.cache, 0, kk.cuda(), vv.cuda(), layout, 0, 4, pages, t0, n)
    torch.cuda.synchronize()
    want_k, want_v = sc.k_wires[0][0].copy(), sc.v_wires[0][0].copy()
    want_k[:, t0:t0 + n], want_v[:, t0:t0 + n] = new_k.numpy(), new_v.numpy()
    assert np.array_equal(_dequant_all(sc, 0, 0, 0), orc.decode_rowmajor_bf16(want_k))
    assert np.array_equal(_dequant_all(sc, 0, 1, 0), orc.decode_rowmajor_bf16(want_v))
    assert np.array_equal(_dequant_all(sc, 0, 0, 1), orc.decode_rowmajor_bf16(sc.k_wires[0][1]))
    # pages not named in the call are untouched, byte for byte (including the 0xA5 fill of spare pages)
    rb = 4352 if fmt == hma.HMA_KV_BFP8 else 8192
    now = sc.cache.layers[0].view(sc.num_pages, -1).cpu().numpy()
    was = before[0].view(sc.num_pages, -1).cpu().numpy()
    touched = set(int(p) for p in pages.cpu().numpy())
    for p in range(sc.num_pages):
        if p not in touched:
            assert np.array_equal(now[p], was[p]), p
    assert now.shape[1] == 4 * rb
    # sub-range dequant (token_begin not page aligned) matches the same slice
    out = torch.zeros((n, 4, 128), dtype=torch.bfloat16, device="cuda")
    hma.hma_bfp8_dequant_bf16(sc.cache, 0, 1, pages, t0, n, out)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(out).transpose(1, 0, 2), orc.decode_rowmajor_bf16(new_v.numpy()))


@pytest.mark.parametrize("layout", [hma.HMA_WIRE_ROWMAJOR, hma.HMA_WIRE_TILE32])
def test_all_shards_in_one_launch_equal_shard_by_shard(layout):
    lens = [33, 100, 16, 1]
    a = Scenario(lens, 32, 8, seed=9, permute=True, wire_layout=layout, shards=4, fill=0x11)
    b = Scenario(lens, 32, 8, seed=9, permute=True, wire_layout=layout, shards=4, fill=0x11, one_launch=True)
    assert torch.equal(a.cache.layers[0], b.cache.layers[0])
    kw = torch.from_numpy(a.k_wires[0][0][:2]).cuda()
    with pytest.raises(hma.HmaError) as e:       # overlapping head ranges are refused
        hma.hma_kv_ingest_layer_shards(a.cache, 0, [kw, kw], [kw, kw], hma.HMA_WIRE_ROWMAJOR, [0, 1], [2, 2], a.table[0, :3].contiguous(), 0, 33)
    assert e.value.status == hma.HMA_ERR_INVALID_ARG


def test_paged_dequant_of_arbitrary_bytes_every_exponent():
    """Random wire bytes (every exponent 0..255, every element byte) through ingest and the paged rebuild."""
    rng = np.random.default_rng(12)
    T, H = 64, 2
    desc = hma.make_desc(1, 2, H, 6)
    cache = hma.KVCache(desc, "cuda", fill=0)
    pages = torch.tensor([4, 1, 5, 2], dtype=torch.int32, device="cuda")
    for trial in range(3):
        kw = rng.integers(0, 256, (H, T, 136)).astype(np.uint8)
        vw = rng.integers(0, 256, (H, T, 136)).astype(np.uint8)
        kw[0, :32, :8] = np.arange(256, dtype=np.uint8).reshape(32, 8)           # each exponent at least once
        vw[1, 32:, :8] = np.arange(256, dtype=np.uint8).reshape(32, 8)[::-1]
        hma.hma_kv_ingest_layer(cache, 0, torch.from_numpy(kw).cuda(), torch.from_numpy(vw).cuda(), hma.HMA_WIRE_ROWMAJOR, 0, H, pages, 0, T)
        for which, wire in ((0, kw), (1, vw)):
            out = torch.zeros((T, H, 128), dtype=torch.bfloat16, device="cuda")
            hma.hma_bfp8_dequant_bf16(cache, 0, which, pages, 0, T, out)
            torch.cuda.synchronize()
            assert np.array_equal(bf16_bits(out).transpose(1, 0, 2), orc.decode_rowmajor_bf16(wire))
    assert hma.hma_error_flags(cache) == 0


@pytest.mark.parametrize("fmt", [hma.HMA_KV_BFP8, hma.HMA_KV_BF16])
def test_whole_request_rebuild_in_one_launch(fmt):
    sc = Scenario([75, 16, 200], 16, 4, seed=14, permute=True, fmt=fmt, layers=3, key_layout=hma.HMA_KEYS_INTERLEAVED)
    for b, t0, n in ((0, 0, 75), (2, 37, 101)):
        first, last = t0 // 16, (t0 + n - 1) // 16
        pages = sc.table[b, first:last + 1].contiguous()
        out = torch.zeros((3, 2, n, 4, 128), dtype=torch.bfloat16, device="cuda")
        hma.hma_bfp8_rebuild_request(sc.cache, pages, t0, n, out)
        naive = torch.zeros_like(out)
        for l in range(3):
            for which in (0, 1):
                hma.hma_bfp8_dequant_bf16_naive(sc.cache, l, which, pages, t0, n, naive[l, which])
        torch.cuda.synchronize()
        assert torch.equal(naive, out)                     # the elementwise strawman produces the same bits
        got = bf16_bits(out)
        for l in range(3):
            wk = orc.relayout_keys_to_half_split(orc.decode_rowmajor_bf16(sc.k_wires[l][b][:, t0:t0 + n]))
            wv = orc.decode_rowmajor_bf16(sc.v_wires[l][b][:, t0:t0 + n])
            assert np.array_equal(got[l, 0].transpose(1, 0, 2), wk) and np.array_equal(got[l, 1].transpose(1, 0, 2), wv)


def test_gpu_encoder_is_bit_identical_to_the_oracle_encoder():
    rng = np.random.default_rng(15)
    x = (rng.standard_normal((3, 37, 128)) * 4.0 ** rng.integers(-6, 7, (3, 37, 1))).astype(np.float32)
    x[rng.random(x.shape) < 0.02] *= 20
    x[rng.random(x.shape) < 0.02] = 0.0
    x[0, 0, :16] = [1.0, 0.5, -0.25, 0.0, 127 / 64, 1 / 64, 1 / 128, 3 / 128, 255 / 128, -1 / 3, 0.1, -0.0, 0.75, 1e-3, -1.5, 0.3]
    x[0, 1, :] = 1e-41                       # FP32 subnormals
    x[0, 2, :] = 0
    x[0, 3, :16] = 2.0 ** -140
    x[0, 3, 0] = 3e38
    x[1, 0, :16] = 2.0 ** np.arange(-20, -4, dtype=np.float32)      # shifts beyond 24 bits
    sc = Scenario([16], 9, 3, seed=15)
    wire = torch.zeros((3, 37, 136), dtype=torch.uint8, device="cuda")
    hma.hma_bfp8_encode_rows(sc.cache, torch.from_numpy(x).cuda(), wire)
    torch.cuda.synchronize()
    assert np.array_equal(wire.cpu().numpy(), orc.encode_rowmajor(x))
    xb = torch.from_numpy(x).to(torch.bfloat16)
    hma.hma_bfp8_encode_rows(sc.cache, xb.cuda(), wire)
    torch.cuda.synchronize()
    assert np.array_equal(wire.cpu().numpy(), orc.encode_rowmajor(xb.float().numpy()))
    assert hma.hma_error_flags(sc.cache) == 0
    # a token made on the GPU joins the cache: encode its K, V rows and ingest them at the end of the sequence
    knew, vnew = torch.from_numpy(x[:, :1]).cuda().contiguous(), torch.from_numpy(x[:, 1:2]).cuda().contiguous()
    kw, vw = torch.zeros((3, 1, 136), dtype=torch.uint8, device="cuda"), torch.zeros((3, 1, 136), dtype=torch.uint8, device="cuda")
    hma.hma_bfp8_encode_rows(sc.cache, knew, kw)
    hma.hma_bfp8_encode_rows(sc.cache, vnew, vw)
    page = sc.spare[:1].copy()
    hma.hma_kv_ingest_layer(sc.cache, 0, kw, vw, hma.HMA_WIRE_ROWMAJOR, 0, 3, torch.from_numpy(page).cuda(), 16, 1)
    out = torch.zeros((1, 3, 128), dtype=torch.bfloat16, device="cuda")
    hma.hma_bfp8_dequant_bf16(sc.cache, 0, 0, torch.from_numpy(page).cuda(), 16, 1, out)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_bits(out).transpose(1, 0, 2), orc.decode_rowmajor_bf16(orc.encode_rowmajor(x[:, :1])))
    bad = torch.full((1, 128), float("inf"), device="cuda")
    hma.hma_bfp8_encode_rows(sc.cache, bad, kw[:1])
    assert hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_VALUE_ENCODE


def test_bfp8_cache_holds_the_wire_bytes_unchanged():
    """Ingest permutes positions only: the multiset of bytes of a fully written page equals that of its wire rows."""
    sc = Scenario([32], 8, 2, seed=6, layers=1, extra_pages=0)
    rec = sc.cache.layers[0].view(2, 2, 4352).cpu().numpy()          # [page][head][record]
    for p in range(2):
        for h in range(2):
            wire = np.concatenate([sc.k_wires[0][0][h, 16 * p:16 * p + 16].reshape(-1), sc.v_wires[0][0][h, 16 * p:16 * p + 16].reshape(-1)])
            assert np.array_equal(np.sort(rec[p, h]), np.sort(wire))


@pytest.mark.parametrize("layout,T", [(hma.HMA_WIRE_TILE32, 112), (hma.HMA_WIRE_TILE32, 75), (hma.HMA_WIRE_ROWMAJOR, 50)])
def test_whole_request_ingest_equals_layer_by_layer(layout, T):
    """hma_kv_ingest_request_shards (every layer in one call) leaves the cache that layer-by-layer ingest leaves."""
    L, H, shards = 3, 4, 2
    sc = Scenario([T], 8, H, seed=31, layers=L, wire_layout=layout, shards=shards, one_launch=True, permute=True)
    want = [t.clone() for t in sc.cache.layers]
    for t in sc.cache.layers:
        t.fill_(0xA5)
    hs = H // shards
    pages = sc.table[0, :(T + 15) // 16].contiguous()
    # [layer][tensor][shard] wire pieces in one allocation, a fixed stride between layers
    pieces = []
    for l in range(L):
        for w in (sc.k_wires[l][0], sc.v_wires[l][0]):
            for s in range(shards):
                x = torch.from_numpy(w[s * hs:(s + 1) * hs].copy())
                pieces.append(synth.rowmajor_to_tile32(x).reshape(-1) if layout == hma.HMA_WIRE_TILE32 else x.reshape(-1))
    n = pieces[0].numel()
    pad = (n + 15) // 16 * 16
    buf = torch.zeros((L, 2, shards, pad), dtype=torch.uint8, device="cuda")
    it = iter(pieces)
    for l in range(L):
        for t in range(2):
            for s in range(shards):
                buf[l, t, s, :n] = next(it).cuda()
    hma.hma_kv_ingest_request_shards(sc.cache, [buf[0, 0, s] for s in range(shards)], [buf[0, 1, s] for s in range(shards)],
                                     2 * shards * pad, layout, [s * hs for s in range(shards)], [hs] * shards, pages, 0, T)
    torch.cuda.synchronize()
    assert hma.hma_error_flags(sc.cache) == 0
    for l in range(L):
        assert torch.equal(sc.cache.layers[l], want[l]), l


def test_rowmajor_wire_needs_only_the_encoders_alignment():
    """hma_bfp8_encode_rows promises 8-byte aligned rows; a wire that starts 8 bytes off a 16-byte boundary is ingested as it is."""
    sc = Scenario([48], 8, 2, seed=21, layers=1)
    pages = sc.table[0, :3].contiguous()
    want = sc.cache.layers[0].clone()
    sc.cache.layers[0].fill_(0xA5)                  # the constructor's fill: pages nobody writes keep it
    kw, vw = sc.k_wires[0][0], sc.v_wires[0][0]
    def shifted(w):
        buf = torch.zeros(w.size + 16, dtype=torch.uint8, device="cuda")
        assert buf.data_ptr() % 16 == 0
        buf[8:8 + w.size] = torch.from_numpy(w.reshape(-1)).cuda()
        return buf[8:8 + w.size]
    hma.hma_kv_ingest_layer(sc.cache, 0, shifted(kw), shifted(vw), hma.HMA_WIRE_ROWMAJOR, 0, 2, pages, 0, 48)
    torch.cuda.synchronize()
    assert hma.hma_error_flags(sc.cache) == 0
    assert torch.equal(sc.cache.layers[0], want)
    with pytest.raises(hma.HmaError) as e:      # a tiled wire is moved in 16-byte pieces
        hma.hma_kv_ingest_layer(sc.cache, 0, shifted(kw), shifted(vw), hma.HMA_WIRE_TILE32, 0, 2, pages, 0, 48)
    assert e.value.status == hma.HMA_ERR_ALIGNMENT


def test_bad_arguments_and_bad_page_ids():
    sc = Scenario([40], 8, 2, seed=7, layers=1)
    kw = torch.from_numpy(sc.k_wires[0][0]).cuda()
    pages = sc.table[0, :3].contiguous()
    with pytest.raises(hma.HmaError) as e:
        hma.hma_kv_ingest_layer(sc.cache, 1, kw, kw, hma.HMA_WIRE_ROWMAJOR, 0, 2, pages, 0, 40)
    assert e.value.status == hma.HMA_ERR_INVALID_ARG
    with pytest.raises(hma.HmaError):
        hma.hma_kv_ingest_layer(sc.cache, 0, kw, kw, hma.HMA_WIRE_ROWMAJOR, 1, 2, pages, 0, 40)       # heads 1..2 of 2
    with pytest.raises(hma.HmaError):
        hma.hma_kv_ingest_layer(sc.cache, 0, kw, kw, 7, 0, 2, pages, 0, 40)
    with pytest.raises(hma.HmaError) as e:
        hma.hma_kv_ingest_layer(sc.cache, 0, kw.view(-1)[1:], kw, hma.HMA_WIRE_ROWMAJOR, 0, 2, pages, 0, 32)
    assert e.value.status == hma.HMA_ERR_ALIGNMENT
    # an out-of-range page id never traps: the page is skipped and a flag bit is raised
    before = sc.cache.layers[0].clone()
    bad = torch.tensor([sc.num_pages + 5, -1, int(pages[2])], dtype=torch.int32, device="cuda")
    hma.hma_kv_ingest_layer(sc.cache, 0, kw, kw, hma.HMA_WIRE_ROWMAJOR, 0, 2, bad, 0, 32)
    assert hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_PAGE_INGEST
    assert torch.equal(before, sc.cache.layers[0])
    out = torch.full((32, 2, 128), 1.0, dtype=torch.bfloat16, device="cuda")
    hma.hma_bfp8_dequant_bf16(sc.cache, 0, 0, bad, 0, 32, out)
    assert hma.hma_error_flags(sc.cache) == hma.HMA_FLAG_BAD_PAGE_DEQUANT
    assert not bf16_bits(out).any()
    assert hma.hma_error_flags(sc.cache) == 0
