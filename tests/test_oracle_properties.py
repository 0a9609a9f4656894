"""Property tests of the CPU oracle with hypothesis (no GPU): the BFP8 codec on arbitrary finite inputs, the tile packer on
arbitrary bytes, attention invariants on arbitrary wire bytes."""
import math

import numpy as np
from hypothesis import given, settings, strategies as st
from hypothesis.extra import numpy as hnp

from oracle import oracle as orc

finite32 = st.floats(min_value=-float(2.0 ** 127), max_value=float(2.0 ** 127), allow_nan=False, allow_infinity=False, width=32)


@settings(max_examples=200, deadline=None)
@given(hnp.arrays(np.float32, 16, elements=finite32))
def test_block_encode_properties(x):
    E, m = orc.bfp8_encode(x)
    E, m = int(E[0]), m[0]
    fields = (x.view(np.uint32) >> 23) & 0xFF
    assert E == fields.max()                                           # shared exponent = largest exponent field
    assert np.array_equal(m >> 7, (x.view(np.uint32) >> 31).astype(np.uint8))
    dec = orc.bfp8_decode_f64(np.array([E], np.uint8), m)[0]
    ulp = math.ldexp(1.0, E - 133)
    xs = np.where(fields == 0, 0.0, x.astype(np.float64))             # FP32 subnormals flush to zero
    mag = m & 0x7F
    assert (np.abs(dec - xs)[mag < 127] <= 0.5 * ulp).all()            # round to nearest
    assert (np.abs(dec - xs)[mag == 127] < ulp).all()                  # saturation
    if E > 0:
        assert mag.max() >= 64                                         # the largest element keeps its leading one
    # order is preserved among elements of equal sign (monotone rounding)
    pos = np.argsort(xs)
    assert (np.diff(dec[pos]) >= 0).all()
    # decode to BF16 is exact and re-encoding the decoded block is the identity on bytes (when E is in normal range)
    bf = orc.bfp8_decode_bf16(np.array([E], np.uint8), m)[0]
    back = (bf.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    if E < 255:
        assert np.array_equal(back, dec)
    if 7 <= E < 255 and mag.max() >= 64:
        E2, m2 = orc.bfp8_encode(dec.astype(np.float32))
        assert int(E2[0]) == E and np.array_equal(m2[0] & 0x7F, mag)


@settings(max_examples=300, deadline=None)
@given(st.floats(allow_nan=False, allow_infinity=False, width=64))
def test_bf16_rounding_is_nearest_even(x):
    h = orc.f64_to_bf16(x)
    v = orc.bf16_to_f64(h)
    if math.isinf(v):
        assert abs(x) >= (2 - 2 ** -8) * 2.0 ** 127                    # overflow threshold: max finite + half an ulp
        return
    # neighbours in BF16: v is at least as close to x as either of them, ties go to the even pattern
    mag = h & 0x7FFF
    lo = orc.bf16_to_f64((h & 0x8000) | (mag - 1)) if mag > 0 else -orc.bf16_to_f64(0x0001) * (1 if not (h & 0x8000) else -1)
    hi = orc.bf16_to_f64((h & 0x8000) | (mag + 1)) if mag < 0x7F7F else math.copysign(math.inf, v if v else 1.0)
    d = abs(x - v)
    for nb in (lo, hi):
        if math.isfinite(nb):
            assert d <= abs(x - nb)
            if d == abs(x - nb) and nb != v:
                assert (h & 1) == 0


@settings(max_examples=50, deadline=None)
@given(st.integers(1, 70), st.integers(1, 3), st.integers(0, 2 ** 32 - 1))
def test_tile_packer_is_a_byte_permutation(T, H, seed):
    rm = np.random.default_rng(seed).integers(0, 256, (H, T, 136)).astype(np.uint8)
    tiles = orc.pack_tile32(rm)
    assert np.array_equal(orc.unpack_tile32(tiles, T, H), rm)
    # padding is zero and every wire byte appears exactly once
    assert np.array_equal(np.sort(tiles[tiles.nonzero()]), np.sort(rm[rm.nonzero()]))


@settings(max_examples=25, deadline=None)
@given(st.integers(1, 40), st.integers(0, 2 ** 32 - 1))
def test_attention_invariants_on_arbitrary_bytes(T, seed):
    rng = np.random.default_rng(seed)
    kw = rng.integers(0, 256, (2, T, 136)).astype(np.uint8)
    vw = rng.integers(0, 256, (2, T, 136)).astype(np.uint8)
    kw[:, :, :8] = rng.integers(110, 135, (2, T, 8))                   # keep scores and values in a sane range
    vw[:, :, :8] = rng.integers(110, 135, (2, T, 8))
    q = (rng.standard_normal((1, 4, 128)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    o, _, p = orc.decode_attention(q, [kw], [vw], 2, want_probs=True)
    assert abs(p.sum() - 1) < 1e-12 and (p >= 0).all()
    v = orc.decode_rowmajor_f64(vw)
    for h in range(4):                                                 # outputs are convex combinations of the values
        assert (o[0, h] <= v[h // 2].max(axis=0) + 1e-9).all() and (o[0, h] >= v[h // 2].min(axis=0) - 1e-9).all()
    perm = rng.permutation(T)                                          # token order does not matter
    o2, _ = orc.decode_attention(q, [kw[:, perm]], [vw[:, perm]], 2)
    assert np.allclose(o, o2, rtol=1e-12, atol=1e-12 * np.abs(v).max())
    o3, _ = orc.decode_attention(q, [np.concatenate([kw, kw], 1)], [np.concatenate([vw, vw], 1)], 2)   # duplicating every token too
    assert np.allclose(o, o3, rtol=1e-12, atol=1e-12 * np.abs(v).max())
