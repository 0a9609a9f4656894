"""Seeded random small workloads: every supported group size, ragged and empty contexts, both cache formats, both key
layouts, permuted pages, random softmax scales; GPU against the oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2606_29986_b200 import hma
from helpers import Scenario, bf16_bits, check_attention

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("case", range(16))
def test_random_small_workload(case):
    rng = np.random.default_rng(1000 + case)
    hkv = int(rng.choice([1, 2, 3, 4, 8]))
    G = int(rng.integers(1, 9))
    B = int(rng.integers(1, 7))
    lens = [int(v) for v in rng.choice([0, 1, 2, 15, 16, 17, 31, 32, 33, 47, 64, 100, 130, 257, 300], B)]
    fmt = hma.HMA_KV_BF16 if rng.random() < 0.3 else hma.HMA_KV_BFP8
    layout = hma.HMA_WIRE_TILE32 if rng.random() < 0.5 else hma.HMA_WIRE_ROWMAJOR
    keyl = hma.HMA_KEYS_INTERLEAVED if rng.random() < 0.3 else hma.HMA_KEYS_AS_QUERIES
    sc = Scenario(lens, G * hkv, hkv, seed=2000 + case, permute=bool(rng.random() < 0.7), fmt=fmt, wire_layout=layout,
                  key_layout=keyl, fill=int(rng.integers(0, 256)), layers=2)
    scale = float(rng.uniform(0.02, 0.3))
    for layer in (0, 1):
        ref64, _ = sc.oracle(layer, scale)
        o32 = sc.attention(layer, torch.float32, sm_scale=scale).cpu().numpy()
        o16 = bf16_bits(sc.attention(layer, torch.bfloat16, sm_scale=scale))
        check_attention(o32, o16, ref64)
        for b, T in enumerate(lens):
            if T == 0:
                assert not o32[b].any()
        simple = sc.attention(layer, torch.float32, simple=True, sm_scale=scale).cpu().numpy()
        assert np.abs(simple - o32).max() <= 5e-3
    assert hma.hma_error_flags(sc.cache) == 0
