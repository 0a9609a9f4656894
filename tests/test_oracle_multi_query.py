"""Pins of the oracle's multi-query decode attention (no GPU): it must reduce to the single-query oracle on truncated
contexts, agree with float64 library attention under an explicit causal mask, and obey the closed forms."""
import math

import numpy as np
import torch

from oracle import oracle as orc
from paper_2606_29986_b200 import synth


def _np_values(wire):
    E = wire[:, :, :8].astype(np.int64).repeat(16, axis=2)
    b = wire[:, :, 8:].astype(np.int64)
    return np.ldexp((b & 0x7F).astype(np.float64), E - 133) * np.where(b >= 128, -1.0, 1.0)


def _bf16_to_f64(bits):
    return (np.asarray(bits, np.uint32) << 16).view(np.float32).astype(np.float64)


def _case(B, q_len, Hq, Hkv, lens, seed):
    q = synth.make_q(B * q_len, Hq, seed).view(torch.int16).numpy().view(np.uint16).reshape(B, q_len, Hq, 128)
    kw = [synth.make_kv_wire(Hkv, int(t), synth.sequence_seed(seed, 0, b, 0)).numpy() for b, t in enumerate(lens)]
    vw = [synth.make_kv_wire(Hkv, int(t), synth.sequence_seed(seed, 0, b, 1)).numpy() for b, t in enumerate(lens)]
    return q, kw, vw


def test_one_query_token_is_plain_decode_attention():
    q, kw, vw = _case(3, 1, 8, 2, [40, 1, 17], 11)
    m64, m16 = orc.decode_attention_multi(q, kw, vw, 2)
    s64, s16 = orc.decode_attention(q[:, 0], kw, vw, 2)
    assert np.array_equal(m64[:, 0], s64) and np.array_equal(m16[:, 0], s16)


def test_query_i_equals_single_query_attention_over_the_truncated_context():
    """Query i sees exactly the first T - (q_len - 1 - i) tokens: the same numbers as the (separately pinned)
    single-query oracle run on the wire bytes cut to that length."""
    lens, q_len = [37, 4, 16, 3], 4
    q, kw, vw = _case(4, q_len, 8, 4, lens, 12)
    m64, m16 = orc.decode_attention_multi(q, kw, vw, 4, sm_scale=0.11)
    for b, T in enumerate(lens):
        for i in range(q_len):
            vis = T - (q_len - 1 - i)
            if vis <= 0:
                assert not m64[b, i].any() and not m16[b, i].any()       # a query that sees nothing: zeros
                continue
            s64, s16 = orc.decode_attention(q[b:b + 1, i], [kw[b][:, :vis]], [vw[b][:, :vis]], 4, sm_scale=0.11)
            assert np.allclose(m64[b, i], s64[0], rtol=1e-13, atol=1e-300)
            assert np.array_equal(m16[b, i], s16[0])


def test_agrees_with_float64_library_attention_under_a_causal_mask():
    lens, q_len, Hq, Hkv = [29, 8], 3, 8, 2
    q, kw, vw = _case(2, q_len, Hq, Hkv, lens, 13)
    m64, _ = orc.decode_attention_multi(q, kw, vw, Hkv)
    G = Hq // Hkv
    for b, T in enumerate(lens):
        K = torch.from_numpy(_np_values(kw[b])).repeat_interleave(G, dim=0)          # [Hq][T][128]
        V = torch.from_numpy(_np_values(vw[b])).repeat_interleave(G, dim=0)
        Q = torch.from_numpy(_bf16_to_f64(q[b])).permute(1, 0, 2)                     # [Hq][q_len][128]
        mask = torch.zeros((q_len, T), dtype=torch.bool)
        for i in range(q_len):
            mask[i, :T - (q_len - 1 - i)] = True
        ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, attn_mask=mask, scale=1.0 / math.sqrt(128))
        assert np.allclose(m64[b], ref.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_closed_forms_first_query_of_a_two_token_context_returns_v0_and_zero_queries_give_prefix_means():
    q, kw, vw = _case(1, 2, 4, 2, [2], 14)
    m64, m16 = orc.decode_attention_multi(q, kw, vw, 2)
    v = _np_values(vw[0])
    for h in range(4):
        assert np.array_equal(m64[0, 0, h], v[h // 2, 0])                 # query 0 sees only token 0: its V exactly
        assert np.array_equal(_bf16_to_f64(m16[0, 0, h]), v[h // 2, 0])
    q, kw, vw = _case(1, 3, 4, 2, [20], 15)
    q[:] = 0
    m64, _ = orc.decode_attention_multi(q, kw, vw, 2)
    v = _np_values(vw[0])
    for i in range(3):
        for h in range(4):
            assert np.allclose(m64[0, i, h], v[h // 2, :20 - (2 - i)].mean(axis=0), rtol=1e-13, atol=1e-15)
