"""Pins of the CPU oracle's fp64 decode attention (no GPU): closed forms, a float64 library routine, brute force."""
import math

import numpy as np
import torch

from oracle import oracle as orc
from paper_2606_29986_b200 import synth


def _np_values(wire):
    """Independent numpy decode of ROWMAJOR wire bytes [H][T][136] -> float64 [H][T][128]."""
    E = wire[:, :, :8].astype(np.int64).repeat(16, axis=2)
    b = wire[:, :, 8:].astype(np.int64)
    return np.ldexp((b & 0x7F).astype(np.float64), E - 133) * np.where(b >= 128, -1.0, 1.0)


def _bf16_to_f64(bits):
    return (np.asarray(bits, np.uint32) << 16).view(np.float32).astype(np.float64)


def _case(B, Hq, Hkv, lens, seed):
    q = synth.make_q(B, Hq, seed).view(torch.int16).numpy().view(np.uint16)
    kw = [synth.make_kv_wire(Hkv, int(t), synth.sequence_seed(seed, 0, b, 0)).numpy() for b, t in enumerate(lens)]
    vw = [synth.make_kv_wire(Hkv, int(t), synth.sequence_seed(seed, 0, b, 1)).numpy() for b, t in enumerate(lens)]
    return q, kw, vw


def test_softmax_rows_sum_to_one_and_weights_match_definition():
    q, kw, vw = _case(2, 8, 2, [57, 9], 1)
    _, _, p = orc.decode_attention(q, kw, vw, 2, want_probs=True)
    assert p.shape == (57,) and abs(p.sum() - 1.0) < 1e-12 and (p > 0).all()
    s = (_np_values(kw[0])[0] @ _bf16_to_f64(q[0, 0])) / math.sqrt(128)
    w = np.exp(s - s.max())
    assert np.allclose(p, w / w.sum(), rtol=1e-12, atol=0)


def test_single_key_returns_v_exactly():
    q, kw, vw = _case(3, 8, 4, [1, 1, 1], 2)
    o64, o16 = orc.decode_attention(q, kw, vw, 4)
    for b in range(3):
        v = _np_values(vw[b])                       # [Hkv][1][128]
        for h in range(8):
            assert np.array_equal(o64[b, h], v[h // 2, 0])
            assert np.array_equal(_bf16_to_f64(o16[b, h]), v[h // 2, 0])   # BFP8 values are BF16-exact


def test_zero_query_gives_mean_of_v():
    q, kw, vw = _case(2, 4, 2, [33, 16], 3)
    q[:] = 0
    o64, _ = orc.decode_attention(q, kw, vw, 2)
    for b in range(2):
        v = _np_values(vw[b])
        for h in range(4):
            assert np.allclose(o64[b, h], v[h // 2].mean(axis=0), rtol=1e-13, atol=1e-15)


def test_group_heads_with_equal_query_agree_and_empty_context_is_zero():
    q, kw, vw = _case(2, 8, 2, [20, 0], 4)
    q[0, 1:4] = q[0, 0]
    o64, o16 = orc.decode_attention(q, kw, vw, 2)
    for h in (1, 2, 3):
        assert np.array_equal(o64[0, h], o64[0, 0])
    assert not np.array_equal(o64[0, 4], o64[0, 0])
    assert not o64[1].any() and not o16[1].any()


def test_against_float64_library_attention():
    """torch scaled_dot_product_attention in float64 on CPU over independently decoded K, V."""
    for (B, Hq, Hkv, lens, seed) in ((2, 8, 2, [40, 40], 5), (1, 10, 2, [77], 6), (3, 8, 8, [16, 16, 16], 7)):
        q, kw, vw = _case(B, Hq, Hkv, lens, seed)
        o64, o16 = orc.decode_attention(q, kw, vw, Hkv, sm_scale=0.11)
        G = Hq // Hkv
        for b in range(B):
            K = torch.from_numpy(_np_values(kw[b])).repeat_interleave(G, dim=0)      # [Hq][T][128]
            V = torch.from_numpy(_np_values(vw[b])).repeat_interleave(G, dim=0)
            Q = torch.from_numpy(_bf16_to_f64(q[b]))[:, None, :]
            ref = torch.nn.functional.scaled_dot_product_attention(Q[None], K[None], V[None], scale=0.11)[0, :, 0].numpy()
            assert np.allclose(o64[b], ref, rtol=1e-10, atol=1e-12)
            want16 = torch.from_numpy(ref).to(torch.float32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
            # double rounding through float32 can differ from the direct RNE only on near-ties: allow 1 ulp on <0.1 %
            diff = (o16[b].astype(np.int32) - want16.astype(np.int32))
            assert np.abs(diff).max() <= 1 and (diff != 0).mean() < 1e-3


def test_brute_force_tiny():
    """Pure-python loops, exact rational-free float arithmetic in a different evaluation order."""
    q, kw, vw = _case(2, 4, 2, [5, 3], 8)
    o64, _ = orc.decode_attention(q, kw, vw, 2, sm_scale=0.25)
    for b, T in enumerate([5, 3]):
        for h in range(4):
            g = h // 2
            qv = [float(x) for x in _bf16_to_f64(q[b, h])]
            scores = []
            for t in range(T):
                row = kw[b][g, t]
                acc = 0.0
                for d in range(128):
                    byte = int(row[8 + d])
                    val = math.ldexp(byte & 0x7F, int(row[d // 16]) - 133)
                    acc += qv[d] * (-val if byte & 0x80 else val)
                scores.append(0.25 * acc)
            mx = max(scores)
            w = [math.exp(s - mx) for s in scores]
            tot = sum(w)
            for d in range(0, 128, 7):
                o = 0.0
                for t in range(T):
                    row = vw[b][g, t]
                    byte = int(row[8 + d])
                    val = math.ldexp(byte & 0x7F, int(row[d // 16]) - 133)
                    o += (w[t] / tot) * (-val if byte & 0x80 else val)
                assert abs(o - o64[b, h, d]) <= 1e-13 * max(1.0, abs(o))


def test_softmax_shift_invariance_and_scale():
    """Adding a constant to every key along q leaves the output unchanged; sm_scale = 0 gives the mean."""
    q, kw, vw = _case(1, 2, 1, [24], 9)
    o_a, _ = orc.decode_attention(q, kw, vw, 1, sm_scale=0.0)
    v = _np_values(vw[0])
    assert np.allclose(o_a[0, 0], v[0].mean(axis=0), rtol=1e-13, atol=1e-15)
    o_b, _ = orc.decode_attention(q, kw, vw, 1, sm_scale=1e3)    # near-argmax
    s = _np_values(kw[0])[0] @ _bf16_to_f64(q[0, 0])
    assert np.allclose(o_b[0, 0], v[0, int(np.argmax(s))], rtol=0, atol=1e-6 * np.abs(v).max()) or np.sort(s)[-1] - np.sort(s)[-2] < 0.02


def test_key_relayout_matches_the_two_rotary_conventions():
    """The interleaved -> half-split map is pinned by RoPE itself: rotating pairs (2i, 2i+1) and then re-laying out
    equals re-laying out and then rotating pairs (i, i+64) with the same angles."""
    idx = [orc.half_split_index(c) for c in range(128)]
    assert sorted(idx) == list(range(128))                                   # a permutation
    assert idx[:4] == [0, 64, 1, 65] and idx[126:] == [63, 127]
    rng = np.random.default_rng(10)
    x = rng.standard_normal((3, 128))
    theta = rng.uniform(0, 2 * np.pi, 64)
    c, s = np.cos(theta), np.sin(theta)
    inter = np.empty_like(x)                                                  # RoPE in interleaved convention
    inter[:, 0::2] = x[:, 0::2] * c - x[:, 1::2] * s
    inter[:, 1::2] = x[:, 0::2] * s + x[:, 1::2] * c
    xs = orc.relayout_keys_to_half_split(x)
    half = np.empty_like(x)                                                   # RoPE in half-split convention
    half[:, :64] = xs[:, :64] * c - xs[:, 64:] * s
    half[:, 64:] = xs[:, :64] * s + xs[:, 64:] * c
    assert np.allclose(orc.relayout_keys_to_half_split(inter), half, rtol=0, atol=1e-14)


def test_attention_with_interleaved_keys_equals_attention_in_one_layout():
    q, kw, vw = _case(2, 8, 2, [37, 12], 11)
    o_int, _ = orc.decode_attention(q, kw, vw, 2, keys_interleaved=True)       # q is half-split, keys interleaved
    q_int = np.empty_like(q)                                                   # the same queries brought to the keys' order
    for c in range(128):
        q_int[..., c] = q[..., orc.half_split_index(c)]
    o_same, _ = orc.decode_attention(q_int, kw, vw, 2)
    assert np.array_equal(o_int, o_same)
    o_plain, _ = orc.decode_attention(q, kw, vw, 2)
    assert not np.allclose(o_int, o_plain)                                     # and the flag does change the result


def test_mixed_prefix_and_bf16_tail():
    """BFP8 prefix + BF16 tail: equals the plain oracle when the tail is empty or when the tail holds the BF16 decode of
    BFP8 bytes, and equals float64 library attention over the concatenated values."""
    q, kw, vw = _case(2, 8, 2, [21, 7], 12)
    empty = [np.zeros((2, 0, 128), np.uint16)] * 2
    o_plain, b_plain = orc.decode_attention(q, kw, vw, 2, sm_scale=0.2)
    o_mix, b_mix = orc.decode_attention_mixed(q, kw, vw, empty, empty, 2, sm_scale=0.2)
    assert np.array_equal(o_plain, o_mix) and np.array_equal(b_plain, b_mix)
    # split every sequence: the first part stays BFP8, the rest is handed over as its exact BF16 decode
    cut = [9, 0]
    kp = [w[:, :c] for w, c in zip(kw, cut)]
    vp = [w[:, :c] for w, c in zip(vw, cut)]
    kt = [orc.decode_rowmajor_bf16(w[:, c:]) for w, c in zip(kw, cut)]
    vt = [orc.decode_rowmajor_bf16(w[:, c:]) for w, c in zip(vw, cut)]
    o_split, _ = orc.decode_attention_mixed(q, kp, vp, kt, vt, 2, sm_scale=0.2)
    assert np.allclose(o_split, o_plain, rtol=1e-13, atol=1e-15)
    # a genuinely BF16 tail (values BFP8 cannot hold) against the float64 library routine
    rng = np.random.default_rng(13)
    tails = [(rng.standard_normal((2, s, 128)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16) for s in (5, 12)]
    tails_v = [(rng.standard_normal((2, s, 128)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16) for s in (5, 12)]
    o_m, _ = orc.decode_attention_mixed(q, kw, vw, tails, tails_v, 2, sm_scale=0.2)
    for b in range(2):
        K = np.concatenate([_np_values(kw[b]), _bf16_to_f64(tails[b])], axis=1)
        V = np.concatenate([_np_values(vw[b]), _bf16_to_f64(tails_v[b])], axis=1)
        Kt = torch.from_numpy(K).repeat_interleave(4, dim=0)
        Vt = torch.from_numpy(V).repeat_interleave(4, dim=0)
        Q = torch.from_numpy(_bf16_to_f64(q[b]))[:, None, :]
        ref = torch.nn.functional.scaled_dot_product_attention(Q[None], Kt[None], Vt[None], scale=0.2)[0, :, 0].numpy()
        assert np.allclose(o_m[b], ref, rtol=1e-10, atol=1e-12)
