"""Seeded synthetic inputs for the BFP8 decode-attention path.

This module is shared by the tests, the benchmark and the smoke check.  It holds
no arithmetic of the decode-side path (no BFP8 decode, no attention); it only
draws random tensors, shapes and block tables, and turns FP32 draws into the raw
BFP8 wire bytes a prefill accelerator would ship (the producer's job, paper
section 3.1).  It imports neither the CUDA binding nor the CPU oracle.

The workloads stand in for the paper's ShareGPT / LongBench / arXiv traces
(Table 2), which are not available offline: shapes follow Qwen3 attention
geometry, values are N(0,1) with 1 % of (kv head, channel) pairs scaled x20, the
channel-outlier structure typical of post-RoPE keys.
"""
import math

import numpy as np
import torch

HEAD_DIM = 128
PAGE_TOKENS = 16
BLOCK = 16
ROW_BYTES = 136          # 8 exponent bytes + 128 mantissa bytes per (token, kv head)
TILE_BYTES = 1088        # one 32x32 tile: 64 exponent bytes + 1024 mantissa bytes

# name -> geometry of the five benchmark workloads
WORKLOADS = {
    "qwen3-4b-b4-ctx1k": dict(hq=32, hkv=8, batch=4, layers=1, ctx=("uniform", 1024), permute=False),
    "qwen3-8b-b64-ctx4k": dict(hq=32, hkv=8, batch=64, layers=36, ctx=("uniform", 4096), permute=False),
    "qwen3-14b-b128-lognormal": dict(hq=40, hkv=8, batch=128, layers=40,
                                     ctx=("lognormal", 2048, 0.8, 256, 8192), permute=True),
    "qwen3-32b-b32-ctx8k": dict(hq=64, hkv=8, batch=32, layers=64, ctx=("uniform", 8192), permute=False),
    "qwen3-32b-b256-trace": dict(hq=64, hkv=8, batch=256, layers=16,
                                 ctx=("lognormal", 4096, 0.8, 512, 32768), permute=True),
}


def context_lens(spec, batch, seed=0):
    """Context length of each sequence (int32 numpy array)."""
    if spec[0] == "uniform":
        return np.full(batch, spec[1], np.int32)
    _, median, sigma, lo, hi = spec
    rng = np.random.default_rng(seed)
    t = np.exp(math.log(median) + sigma * rng.standard_normal(batch))
    return np.clip(np.rint(t), lo, hi).astype(np.int32)


def pages_of(ctx):
    return (np.asarray(ctx, np.int64) + PAGE_TOKENS - 1) // PAGE_TOKENS


def block_table(ctx, permute, seed=0, extra_pages=0):
    """Block table int32 [B][max_pages] (unused entries -1) and the number of physical pages.

    Physical pages are handed out in sequence order, or as one seeded random
    permutation of all pages when `permute` is set."""
    npg = pages_of(ctx)
    total = int(npg.sum())
    ids = np.arange(total + extra_pages, dtype=np.int32)
    if permute:
        ids = np.random.default_rng(seed + 7919).permutation(ids).astype(np.int32)
    table = np.full((len(ctx), max(int(npg.max()), 1)), -1, np.int32)
    o = 0
    for b, n in enumerate(npg):
        table[b, :n] = ids[o:o + n]
        o += int(n)
    return table, total + extra_pages, ids[total:]


def make_q(batch, hq, seed=0, device="cpu"):
    """Q ~ N(0,1) rounded to BF16, [B][Hq][128]."""
    if torch.device(device).type == "cpu":
        q = torch.from_numpy(np.random.default_rng(seed + 104729).standard_normal(
            (batch, hq, HEAD_DIM)).astype(np.float32))
        return q.to(torch.bfloat16)
    g = torch.Generator(device=device)
    g.manual_seed(seed + 104729)
    return torch.randn((batch, hq, HEAD_DIM), generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)


def outlier_channels(hkv, seed):
    """The (kv head, channel) pairs whose values are scaled x20: 1 % of hkv*128, without replacement."""
    n = int(round(0.01 * hkv * HEAD_DIM))
    flat = np.random.default_rng(seed + 15485863).choice(hkv * HEAD_DIM, size=n, replace=False)
    return np.stack([flat // HEAD_DIM, flat % HEAD_DIM], axis=1)


def make_kv_fp32(hkv, tokens, seed, device="cpu", outlier_scale=20.0, channel_seed=None):
    """One tensor (K or V) of one sequence: FP32 [Hkv][tokens][128], N(0,1) with outlier channels.

    `channel_seed` picks the outlier channels; sequences of one layer share it (outlier channels
    are a property of the layer, not of the sequence).  It defaults to `seed`."""
    if torch.device(device).type == "cpu":
        x = torch.from_numpy(np.random.default_rng(seed).standard_normal(
            (hkv, tokens, HEAD_DIM)).astype(np.float32))
    else:
        g = torch.Generator(device=device)
        g.manual_seed(seed)
        x = torch.randn((hkv, tokens, HEAD_DIM), generator=g, device=device, dtype=torch.float32)
    for h, c in outlier_channels(hkv, seed if channel_seed is None else channel_seed):
        x[int(h), :, int(c)] *= outlier_scale
    return x


def bfp8_encode(x):
    """FP32 tensor [..., 128] -> ROWMAJOR BFP8 wire bytes uint8 [..., 136] (producer-side encode).

    Blocks of 16 consecutive channels share the largest FP32 exponent field of the
    block; each 24-bit significand is shifted to that exponent and rounded to
    nearest-even onto 7 bits, saturating at 127; the sign bit is copied."""
    assert x.dtype == torch.float32 and x.shape[-1] == HEAD_DIM
    bits = x.contiguous().view(torch.int32)
    lead = bits.shape[:-1]
    bits = bits.reshape(-1, HEAD_DIM // BLOCK, BLOCK)
    e = (bits >> 23) & 0xFF
    if bool((e == 0xFF).any()):
        raise ValueError("NaN/Inf cannot be BFP8-encoded")
    E = e.max(dim=-1, keepdim=True).values
    sig = (bits & 0x7FFFFF) | 0x800000
    sh = torch.clamp(17 + (E - e), max=30)
    quo = sig >> sh
    rem = sig & ((1 << sh) - 1)
    half = 1 << (sh - 1)
    quo = quo + ((rem > half) | ((rem == half) & ((quo & 1) == 1))).to(torch.int32)
    quo = torch.where(e == 0, torch.zeros_like(quo), torch.clamp(quo, max=127))
    byte = (((bits >> 31) & 1) << 7) | quo
    out = torch.empty((bits.shape[0], ROW_BYTES), dtype=torch.uint8, device=x.device)
    out[:, :HEAD_DIM // BLOCK] = E.squeeze(-1).to(torch.uint8)
    out[:, HEAD_DIM // BLOCK:] = byte.reshape(-1, HEAD_DIM).to(torch.uint8)
    return out.reshape(*lead, ROW_BYTES)


def make_kv_wire(hkv, tokens, seed, device="cpu", channel_seed=None):
    """ROWMAJOR wire bytes [Hkv][tokens][136] of one tensor of one sequence."""
    return bfp8_encode(make_kv_fp32(hkv, tokens, seed, device, channel_seed=channel_seed))


def rowmajor_to_tile32(wire):
    """ROWMAJOR [heads][tokens][136] -> TILE32 bytes [heads][ceil(T/32)][4][1088] (pure byte movement).

    A tile covers 32 tokens x 32 channels as four 16x16 faces ordered (row half,
    column half); exponents first (face*16 + row%16), then mantissas
    (64 + face*256 + (row%16)*16 + col%16).  Padding rows are zero."""
    H, T, _ = wire.shape
    tr = (T + 31) // 32
    pad = torch.zeros((H, tr * 32, ROW_BYTES), dtype=torch.uint8, device=wire.device)
    pad[:, :T] = wire
    ex = pad[:, :, :8].reshape(H, tr, 2, 16, 4, 2)             # head, tile row, row half, r, tile col, col half
    mt = pad[:, :, 8:].reshape(H, tr, 2, 16, 4, 2, 16)
    out = torch.empty((H, tr, 4, TILE_BYTES), dtype=torch.uint8, device=wire.device)
    out[..., :64] = ex.permute(0, 1, 4, 2, 5, 3).reshape(H, tr, 4, 64)
    out[..., 64:] = mt.permute(0, 1, 4, 2, 5, 3, 6).reshape(H, tr, 4, 1024)
    return out


def channel_seed(base_seed, layer, which):
    """Seed of the outlier-channel choice of tensor `which` (0 = K, 1 = V) in a layer."""
    return (base_seed * 1000003 + layer) * 2 + which + 900001


def sequence_seed(base_seed, layer, b, which):
    """Seed of tensor `which` (0 = K, 1 = V) of sequence b in a layer."""
    return ((base_seed * 1000003 + layer) * 100003 + b) * 2 + which + 1
