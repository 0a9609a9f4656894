"""GPU parity of hma_decode_attention_multi (several query tokens per sequence, causal inside the new tokens) against
the oracle's multi-query attention."""
import numpy as np
import pytest
import torch

from paper_2606_29986_b200 import hma, synth
from helpers import Scenario, bf16_bits, check_attention

pytestmark = pytest.mark.gpu
SCALE = 1.0 / np.sqrt(128.0)


def _run(sc, q, dtype):
    out = torch.full(q.shape, float("nan"), dtype=dtype, device="cuda")
    ws = hma.new_workspace(sc.desc, q.shape[0] * q.shape[1])
    hma.hma_decode_attention_multi(sc.cache, 0, q, out, sc.table, sc.ctx, SCALE, ws)
    torch.cuda.synchronize()
    return out


@pytest.mark.parametrize("q_len,hq,hkv,fmt", [(2, 64, 8, hma.HMA_KV_BFP8), (4, 32, 8, hma.HMA_KV_BFP8), (3, 40, 8, hma.HMA_KV_BFP8),
                                              (2, 8, 8, hma.HMA_KV_BFP8), (4, 64, 8, hma.HMA_KV_BF16)])
def test_multi_query_parity(q_len, hq, hkv, fmt):
    from oracle import oracle as orc
    lens = [700, 33, 16, 17, 2, 1, 0, 2100, 48]           # includes contexts shorter than q_len: some queries see nothing
    sc = Scenario(lens, hq, hkv, seed=500 + q_len + hq, permute=True, fmt=fmt)
    q = synth.make_q(len(lens) * q_len, hq, 77).cuda().view(len(lens), q_len, hq, 128)
    ref64, _ = orc.decode_attention_multi(bf16_bits(q), sc.k_wires[0], sc.v_wires[0], hkv)
    o32, o16 = _run(sc, q, torch.float32), _run(sc, q, torch.bfloat16)
    n = len(lens) * q_len
    check_attention(o32.cpu().numpy().reshape(n, hq, 128), bf16_bits(o16).reshape(n, hq, 128), ref64.reshape(n, hq, 128))
    for b, T in enumerate(lens):                           # rows of queries that see no token are zero
        for i in range(q_len):
            if T - (q_len - 1 - i) <= 0:
                assert not o32[b, i].any()
    assert torch.equal(_run(sc, q, torch.bfloat16), o16)   # bitwise repeatable
    assert hma.hma_error_flags(sc.cache) == 0


def test_one_query_token_is_the_plain_call():
    sc = Scenario([900, 40, 0, 16], 32, 8, seed=510, permute=True)
    plain = sc.attention(0, torch.float32)
    multi = _run(sc, sc.q.view(4, 1, 32, 128), torch.float32)
    assert torch.equal(multi.view(4, 32, 128), plain)


def test_multi_query_limits():
    sc = Scenario([64] * 300, 8, 8, seed=511)
    q = torch.zeros((300, 4, 8, 128), dtype=torch.bfloat16, device="cuda")          # 1200 rows > 1024
    out = torch.zeros_like(q)
    with pytest.raises(hma.HmaError) as e:
        hma.hma_decode_attention_multi(sc.cache, 0, q, out, sc.table, sc.ctx, 0.1, hma.new_workspace(sc.desc, 1024))
    assert e.value.status == hma.HMA_ERR_UNSUPPORTED_SHAPE
