"""Pins of the CPU oracle's BFP8 encode/decode, BF16 rounding and tile packer (no GPU)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2606_29986_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name, key):
    rows = []
    for line in open(os.path.join(GOLDEN, name)):
        line = line.strip()
        if line and not line.startswith("#") and line.split()[0] == key:
            rows.append(line.split()[1:])
    return rows


def _bf16_bits_to_float(bits):
    """BF16 bit patterns -> python floats through numpy's own IEEE float32 (independent of the oracle)."""
    return (np.asarray(bits, np.uint32) << 16).view(np.float32).astype(np.float64)


def test_golden_decode_bytes():
    rows = _golden("bfp8_blocks.txt", "decode")
    assert len(rows) >= 20
    for E, b, want in rows:
        m = np.zeros(16, np.uint8)
        m[3] = int(b, 16)
        got = orc.bfp8_decode_bf16(np.array([int(E, 16)], np.uint8), m)[0]
        assert got[3] == int(want, 16), (E, b, hex(got[3]), want)
        assert got[0] == 0          # m = 0, s = 0 -> +0 whatever E


def test_golden_encode_blocks():
    rows = _golden("bfp8_blocks.txt", "encode")
    assert len(rows) == 3
    for r in rows:
        k = r.index("->")
        x = np.array([float(v) for v in r[:k]], np.float32)
        want = [int(v, 16) for v in r[k + 1:]]
        e, m = orc.bfp8_encode(x)
        assert [int(e[0])] + [int(v) for v in m[0]] == want


def test_decode_table_exhaustive():
    """All 256 x 256 (E, byte) pairs: the BF16 bits, read back by numpy, are exactly m * 2^(E-133)."""
    E = np.repeat(np.arange(256, dtype=np.uint8), 16)                      # 16 blocks per exponent
    bytes_ = np.tile(np.arange(256, dtype=np.uint8), 256).reshape(-1, 16)  # each block 16 consecutive byte values
    bits = orc.bfp8_decode_bf16(E, bytes_).reshape(256, 256)
    vals = _bf16_bits_to_float(bits)
    f64 = orc.bfp8_decode_f64(E, bytes_).reshape(256, 256)
    for e in range(256):
        for b in (0, 1, 2, 63, 64, 65, 127, 128, 129, 191, 192, 255) if e not in (0, 1, 6, 7, 127, 254, 255) else range(256):
            m, s = b & 0x7F, b >> 7
            exact = math.ldexp(m, e - 133) * (-1.0 if s else 1.0)
            assert f64[e, b] == exact
            if e == 255 and m >= 64:
                assert bits[e, b] == (0xFF80 if s else 0x7F80)
            else:
                assert vals[e, b] == exact, (e, b)
            assert (bits[e, b] >> 15) == s                 # the sign survives, also for m = 0
    # vectorised check of every finite entry
    mm = (np.arange(256) & 0x7F).astype(np.float64) * np.where(np.arange(256) >= 128, -1.0, 1.0)
    exact = np.ldexp(mm[None, :], (np.arange(256)[:, None] - 133))
    finite = np.isfinite(vals)
    assert finite[:255].all()
    assert np.array_equal(vals[finite], exact[finite])
    assert np.array_equal(np.isinf(vals[255]), (np.arange(256) & 0x7F) >= 64)
    # E = 0 decodes to the BF16 subnormal with the same bits
    assert np.array_equal(bits[0], np.where(np.arange(256) >= 128, 0x8000, 0) | (np.arange(256) & 0x7F))


def test_f64_to_bf16_matches_library_rounding():
    """RNE against torch's float32 -> bfloat16 conversion (a library routine) on float32-exact inputs."""
    rng = np.random.default_rng(1)
    x = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(10.0) ** rng.integers(-30, 30, 20000).astype(np.float32),
        (np.arange(1, 4000, dtype=np.uint32) << 9).view(np.float32),          # float32/bf16 subnormal range, ties included
        np.array([0.0, -0.0, 1.0, 3.3895314e38, 3.4e38, -3.4e38, 1.00390625, 1.01171875, 2 ** -133, 2 ** -134, 1.5 * 2 ** -134], np.float32),
    ])
    x = x[np.isfinite(x)]
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([orc.f64_to_bf16(float(v)) for v in x], np.uint16)
    assert np.array_equal(got, want)
    for h in (0x0001, 0x007F, 0x0080, 0x3F80, 0x7F7F, 0x8001, 0xC2F7):
        assert orc.f64_to_bf16(orc.bf16_to_f64(h)) == h
        assert orc.bf16_to_f64(h) == float(_bf16_bits_to_float([h])[0])


def _representable_blocks(rng, n):
    E = rng.integers(7, 255, n).astype(np.uint8)      # below 7 the small elements are FP32 subnormals, which the encoder flushes
    m = rng.integers(0, 256, (n, 16)).astype(np.uint8)
    m[:, 0] = (m[:, 0] & 0x80) | 64 | (m[:, 0] & 0x3F)     # one element with its leading one at the top
    return E, m


def test_round_trip_on_representable_values():
    rng = np.random.default_rng(2)
    E, m = _representable_blocks(rng, 4000)
    x = orc.bfp8_decode_f64(E, m).astype(np.float32)         # exact: 7-bit significands
    E2, m2 = orc.bfp8_encode(x)
    assert np.array_equal(E2, E) and np.array_equal(m2, m)    # encode(decode(bytes)) == bytes
    assert np.array_equal(orc.bfp8_decode_f64(E2, m2).astype(np.float32), x)


def test_encode_invariants():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal((5000, 16)) * 10.0 ** rng.integers(-3, 4, (5000, 1))).astype(np.float32)
    x[rng.random(x.shape) < 0.02] *= 20
    x[rng.random(x.shape) < 0.02] = 0
    E, m = orc.bfp8_encode(x)
    fexp = (x.view(np.uint32) >> 23) & 0xFF
    assert np.array_equal(E, fexp.max(axis=1).astype(np.uint8))          # shared exponent = largest exponent field
    assert np.array_equal(m >> 7, (x.view(np.uint32) >> 31).astype(np.uint8))   # sign always copied
    dec = orc.bfp8_decode_f64(E, m)
    ulp = np.ldexp(1.0, E.astype(np.int64) - 133)[:, None]
    sat = (m & 0x7F) == 127
    assert (np.abs(dec - x)[~sat] <= 0.5 * ulp.repeat(16, 1)[~sat]).all()   # round to nearest
    assert (np.abs(dec - x)[sat] < ulp.repeat(16, 1)[sat]).all()            # saturation loses < 1 ulp
    E3, m3 = orc.bfp8_encode(dec.astype(np.float32))                          # idempotent
    assert np.array_equal(orc.bfp8_decode_f64(E3, m3), dec)
    assert ((m & 0x7F).max(axis=1) >= 64).all()                               # the largest element is normalised


def test_encode_special_inputs():
    sub = np.full(16, 1e-40, np.float32)
    e, m = orc.bfp8_encode(sub)
    assert e[0] == 0 and not m.any()                       # FP32 subnormals flush to zero
    with pytest.raises(ValueError):
        orc.bfp8_encode(np.array([np.inf] + [0] * 15, np.float32))
    far = np.zeros(16, np.float32)
    far[0], far[1], far[2] = 1.0, 2.0 ** -7, 2.0 ** -8 * 1.5
    e, m = orc.bfp8_encode(far)
    assert e[0] == 127 and list(m[0][:3]) == [0x40, 0x00, 0x00]    # 1/128 ties to even 0; 1.5/256 rounds to 0
    far[1] = 2.0 ** -7 * 1.0001
    assert orc.bfp8_encode(far)[1][0][1] == 1


def test_synth_encoder_matches_oracle_encoder():
    """The torch-op producer encode used to make inputs is bit-identical to the oracle's own encoder."""
    rng = np.random.default_rng(4)
    x = (rng.standard_normal((64, 9, 128)) * 4.0 ** rng.integers(-4, 5, (64, 9, 1))).astype(np.float32)
    x[rng.random(x.shape) < 0.01] *= 20
    x[rng.random(x.shape) < 0.01] = 0.0
    x[0, 0, :16] = [1.0, 0.5, -0.25, 0.0, 127 / 64, 1 / 64, 1 / 128, 3 / 128, 255 / 128, -1 / 3, 0.1, -0.0, 0.75, 1e-3, -1.5, 0.3]
    x[1, 1, :] = 1e-41
    x[2, 2, :] = 0
    x[3, 3, :16] = 2.0 ** -140
    x[3, 3, 0] = 3e38
    wire = synth.bfp8_encode(torch.from_numpy(x)).numpy()
    assert np.array_equal(wire, orc.encode_rowmajor(x.reshape(64, 9, 128)))
    w2 = synth.make_kv_wire(8, 40, seed=11).numpy()
    x2 = synth.make_kv_fp32(8, 40, seed=11).numpy()
    assert np.array_equal(w2, orc.encode_rowmajor(x2))
    # outlier channels really are there: 10 of 1024 (head, channel) pairs are ~20x larger
    big = np.sqrt((x2 ** 2).mean(axis=1)) > 8
    assert big.sum() == 10


def test_tile32_packer():
    rng = np.random.default_rng(5)
    for T, H in ((1, 1), (17, 2), (32, 1), (33, 3), (100, 8)):
        rm = rng.integers(0, 256, (H, T, 136)).astype(np.uint8)
        tiles = orc.pack_tile32(rm)
        assert tiles.size == H * ((T + 31) // 32) * 4 * 1088
        assert np.array_equal(orc.unpack_tile32(tiles, T, H), rm)
        assert np.array_equal(synth.rowmajor_to_tile32(torch.from_numpy(rm)).numpy().reshape(-1), tiles)
    # hand-indexed byte: token 17, channel 21 of head 0 -> tile (0,0), face 3, exponent byte 49, mantissa byte 853
    rm = np.zeros((1, 32, 136), np.uint8)
    rm[0, 17, 8 + 21] = 0xAB
    rm[0, 17, 21 // 16] = 0xCD
    tiles = orc.pack_tile32(rm)
    assert tiles[853] == 0xAB and tiles[49] == 0xCD and np.count_nonzero(tiles) == 2
    # token 40, channel 100 of head 1 (T = 64): tile row 1, tile col 3, r = 8, cc = 4 -> face 0
    rm = np.zeros((2, 64, 136), np.uint8)
    rm[1, 40, 8 + 100] = 0x11
    tiles = orc.pack_tile32(rm)
    base = ((1 * 2 + 1) * 4 + 3) * 1088
    assert tiles[base + 64 + 0 * 256 + 8 * 16 + 4] == 0x11 and np.count_nonzero(tiles) == 1


def test_paper_kv_byte_accounting():
    """136 bytes per (token, kv head, tensor) reproduces the sizes and the egress time the paper prints."""
    (kv,) = _golden("paper_kv_sizes.txt", "kv_size")
    f = dict(s.split("=") for s in kv)
    L, H, d, T = int(f["layers"]), int(f["kv_heads"]), int(f["head_dim"]), int(f["tokens"])
    assert orc.ROW_BYTES == d + d // orc.BLOCK
    bf16 = 2 * L * H * d * T * 2 / 1e9
    bfp8 = 2 * L * H * T * orc.ROW_BYTES / 1e9
    assert abs(bf16 - float(f["bf16_gb"])) <= float(f["rel_tol"]) * float(f["bf16_gb"])
    assert abs(bfp8 - float(f["bfp8_gb"])) <= float(f["rel_tol"]) * float(f["bfp8_gb"])
    (eg,) = _golden("paper_kv_sizes.txt", "egress")
    f = dict(s.split("=") for s in eg)
    nbytes = 2 * int(f["layers"]) * int(f["kv_heads"]) * int(f["tokens"]) * orc.ROW_BYTES
    ms = nbytes * 8 / (float(f["gbit_per_s"]) * 1e9) * 1e3
    assert abs(ms - float(f["ms"])) <= float(f["abs_tol_ms"])
    wire = orc.encode_rowmajor(np.ones((2, 3, 128), np.float32))
    assert wire.nbytes == 2 * 3 * orc.ROW_BYTES
