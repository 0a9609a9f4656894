"""ctypes binding of the CPU oracle (hma_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import
this module.  It imports nothing from the CUDA package.  All arrays are numpy.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hma_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

ROW_BYTES = 136      # 8 exponent bytes + 128 mantissa bytes per (token, kv head)
HEAD_DIM = 128
BLOCK = 16


def build(force=False):
    """Compile the oracle with gcc if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.orc_f64_to_bf16.restype = ctypes.c_uint16
        _lib.orc_f64_to_bf16.argtypes = [ctypes.c_double]
        _lib.orc_bf16_to_f64.restype = ctypes.c_double
        _lib.orc_bf16_to_f64.argtypes = [ctypes.c_uint16]
        _lib.orc_bfp8_encode.restype = ctypes.c_int64
        _lib.orc_tile32_bytes.restype = ctypes.c_int64
        _lib.orc_tile32_bytes.argtypes = [ctypes.c_int64, ctypes.c_int32]
        _lib.orc_num_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def f64_to_bf16(x):
    return int(lib().orc_f64_to_bf16(float(x)))


def bf16_to_f64(h):
    return float(lib().orc_bf16_to_f64(int(h)))


def bfp8_encode(x):
    """x: float32 array whose size is a multiple of 16 -> (exps uint8 [n_blocks], mants uint8 [n_blocks,16])."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    assert x.size % BLOCK == 0
    nb = x.size // BLOCK
    exps = np.empty(nb, np.uint8)
    mants = np.empty((nb, BLOCK), np.uint8)
    bad = lib().orc_bfp8_encode(_p(x), ctypes.c_int64(nb), _p(exps), _p(mants))
    if bad:
        raise ValueError("%d NaN/Inf inputs cannot be BFP8-encoded" % bad)
    return exps, mants


def bfp8_decode_f64(exps, mants):
    exps = np.ascontiguousarray(exps, np.uint8).reshape(-1)
    mants = np.ascontiguousarray(mants, np.uint8).reshape(-1, BLOCK)
    assert mants.shape[0] == exps.size
    out = np.empty((exps.size, BLOCK), np.float64)
    lib().orc_bfp8_decode_f64(_p(exps), _p(mants), ctypes.c_int64(exps.size), _p(out))
    return out


def bfp8_decode_bf16(exps, mants):
    exps = np.ascontiguousarray(exps, np.uint8).reshape(-1)
    mants = np.ascontiguousarray(mants, np.uint8).reshape(-1, BLOCK)
    assert mants.shape[0] == exps.size
    out = np.empty((exps.size, BLOCK), np.uint16)
    lib().orc_bfp8_decode_bf16(_p(exps), _p(mants), ctypes.c_int64(exps.size), _p(out))
    return out


def encode_rowmajor(x):
    """x: float32 [heads][tokens][128] -> ROWMAJOR wire bytes uint8 [heads][tokens][136]."""
    x = np.ascontiguousarray(x, np.float32)
    H, T, D = x.shape
    assert D == HEAD_DIM
    exps, mants = bfp8_encode(x)
    wire = np.empty((H, T, ROW_BYTES), np.uint8)
    wire[:, :, :8] = exps.reshape(H, T, 8)
    wire[:, :, 8:] = mants.reshape(H, T, HEAD_DIM)
    return wire


def decode_rowmajor_bf16(wire):
    """ROWMAJOR wire bytes [heads][tokens][136] -> BF16 bit patterns uint16 [heads][tokens][128]."""
    wire = np.ascontiguousarray(wire, np.uint8)
    H, T, _ = wire.shape
    exps = np.ascontiguousarray(wire[:, :, :8])
    mants = np.ascontiguousarray(wire[:, :, 8:])
    return bfp8_decode_bf16(exps, mants).reshape(H, T, HEAD_DIM)


def decode_rowmajor_f64(wire):
    wire = np.ascontiguousarray(wire, np.uint8)
    H, T, _ = wire.shape
    exps = np.ascontiguousarray(wire[:, :, :8])
    mants = np.ascontiguousarray(wire[:, :, 8:])
    return bfp8_decode_f64(exps, mants).reshape(H, T, HEAD_DIM)


def tile32_bytes(n_tokens, heads):
    return int(lib().orc_tile32_bytes(n_tokens, heads))


def pack_tile32(rowmajor):
    """ROWMAJOR [heads][tokens][136] -> TILE32 wire bytes (flat uint8)."""
    rowmajor = np.ascontiguousarray(rowmajor, np.uint8)
    H, T, _ = rowmajor.shape
    out = np.empty(tile32_bytes(T, H), np.uint8)
    lib().orc_pack_tile32(_p(rowmajor), ctypes.c_int64(T), ctypes.c_int32(H), _p(out))
    return out


def unpack_tile32(tiles, n_tokens, heads):
    tiles = np.ascontiguousarray(tiles, np.uint8).reshape(-1)
    assert tiles.size == tile32_bytes(n_tokens, heads)
    out = np.empty((heads, n_tokens, ROW_BYTES), np.uint8)
    lib().orc_unpack_tile32(_p(tiles), ctypes.c_int64(n_tokens), ctypes.c_int32(heads), _p(out))
    return out


def decode_attention(q_bf16, k_wires, v_wires, num_kv_heads, sm_scale=None, want_probs=False, keys_interleaved=False):
    """fp64 decode attention over ROWMAJOR wire bytes.

    q_bf16  : uint16 [B][Hq][128] (BF16 bit patterns)
    k_wires : list of B uint8 arrays [Hkv][T_b][136] (T_b may be 0)
    v_wires : same for V
    returns (out_f64 [B][Hq][128], out_bf16 uint16 [B][Hq][128]) and, if want_probs,
    the softmax weights of (sequence 0, head 0).
    """
    q_bf16 = np.ascontiguousarray(q_bf16, np.uint16)
    B, Hq, D = q_bf16.shape
    assert D == HEAD_DIM and Hq % num_kv_heads == 0 and len(k_wires) == B == len(v_wires)
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(HEAD_DIM)
    lens = np.array([w.shape[1] for w in k_wires], np.int32)
    offs = np.zeros(B, np.int64)
    sizes = [num_kv_heads * int(t) * ROW_BYTES for t in lens]
    offs[1:] = np.cumsum(sizes)[:-1]
    for w, v, t in zip(k_wires, v_wires, lens):
        assert w.shape == (num_kv_heads, t, ROW_BYTES) == v.shape
    kcat = np.concatenate([np.ascontiguousarray(w, np.uint8).reshape(-1) for w in k_wires] + [np.zeros(1, np.uint8)])
    vcat = np.concatenate([np.ascontiguousarray(w, np.uint8).reshape(-1) for w in v_wires] + [np.zeros(1, np.uint8)])
    out64 = np.empty((B, Hq, D), np.float64)
    out16 = np.empty((B, Hq, D), np.uint16)
    probs = np.zeros(max(int(lens[0]), 1), np.float64) if want_probs else None
    lib().orc_decode_attention(_p(q_bf16), _p(kcat), _p(vcat), _p(offs), _p(lens),
                               ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(num_kv_heads),
                               ctypes.c_double(sm_scale), ctypes.c_int32(1 if keys_interleaved else 0), _p(out64), _p(out16),
                               _p(probs) if want_probs else None)
    if want_probs:
        return out64, out16, probs[:int(lens[0])]
    return out64, out16


def decode_attention_mixed(q_bf16, k_wires, v_wires, k_tails, v_tails, num_kv_heads, sm_scale=None):
    """fp64 decode attention over BFP8 prefixes followed by BF16 tails.

    k_wires, v_wires : list of B uint8 arrays [Hkv][T_b][136]
    k_tails, v_tails : list of B uint16 arrays [Hkv][S_b][128] (BF16 bit patterns), S_b may be 0
    returns (out_f64, out_bf16)."""
    q_bf16 = np.ascontiguousarray(q_bf16, np.uint16)
    B, Hq, D = q_bf16.shape
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(HEAD_DIM)
    lens = np.array([w.shape[1] for w in k_wires], np.int32)
    tl = np.array([t.shape[1] for t in k_tails], np.int32)
    offs = np.zeros(B, np.int64)
    offs[1:] = np.cumsum([num_kv_heads * int(t) * ROW_BYTES for t in lens])[:-1]
    toffs = np.zeros(B, np.int64)
    toffs[1:] = np.cumsum([num_kv_heads * int(t) * HEAD_DIM for t in tl])[:-1]
    kcat = np.concatenate([np.ascontiguousarray(w, np.uint8).reshape(-1) for w in k_wires] + [np.zeros(1, np.uint8)])
    vcat = np.concatenate([np.ascontiguousarray(w, np.uint8).reshape(-1) for w in v_wires] + [np.zeros(1, np.uint8)])
    ktc = np.concatenate([np.ascontiguousarray(t, np.uint16).reshape(-1) for t in k_tails] + [np.zeros(1, np.uint16)])
    vtc = np.concatenate([np.ascontiguousarray(t, np.uint16).reshape(-1) for t in v_tails] + [np.zeros(1, np.uint16)])
    out64 = np.empty((B, Hq, D), np.float64)
    out16 = np.empty((B, Hq, D), np.uint16)
    lib().orc_decode_attention_mixed(_p(q_bf16), _p(kcat), _p(vcat), _p(offs), _p(lens), _p(ktc), _p(vtc), _p(toffs), _p(tl),
                                     ctypes.c_int32(B), ctypes.c_int32(Hq), ctypes.c_int32(num_kv_heads),
                                     ctypes.c_double(sm_scale), _p(out64), _p(out16))
    return out64, out16


def decode_attention_multi(q_bf16, k_wires, v_wires, num_kv_heads, sm_scale=None):
    """fp64 decode attention with q_len query tokens per sequence (the last q_len cached tokens are the new tokens;
    query i sees tokens t < T - (q_len - 1 - i)).

    q_bf16 : uint16 [B][q_len][Hq][128]; k_wires, v_wires as in decode_attention.
    returns (out_f64 [B][q_len][Hq][128], out_bf16)."""
    q_bf16 = np.ascontiguousarray(q_bf16, np.uint16)
    B, q_len, Hq, D = q_bf16.shape
    assert D == HEAD_DIM and Hq % num_kv_heads == 0 and len(k_wires) == B == len(v_wires)
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(HEAD_DIM)
    lens = np.array([w.shape[1] for w in k_wires], np.int32)
    offs = np.zeros(B, np.int64)
    offs[1:] = np.cumsum([num_kv_heads * int(t) * ROW_BYTES for t in lens])[:-1]
    kcat = np.concatenate([np.ascontiguousarray(w, np.uint8).reshape(-1) for w in k_wires] + [np.zeros(1, np.uint8)])
    vcat = np.concatenate([np.ascontiguousarray(w, np.uint8).reshape(-1) for w in v_wires] + [np.zeros(1, np.uint8)])
    out64 = np.empty((B, q_len, Hq, D), np.float64)
    out16 = np.empty((B, q_len, Hq, D), np.uint16)
    lib().orc_decode_attention_multi(_p(q_bf16), _p(kcat), _p(vcat), _p(offs), _p(lens), ctypes.c_int32(B), ctypes.c_int32(q_len),
                                     ctypes.c_int32(Hq), ctypes.c_int32(num_kv_heads), ctypes.c_double(sm_scale), _p(out64), _p(out16))
    return out64, out16


def half_split_index(c):
    """Half-split position of interleaved-order channel c (the key re-layout of section 3.3)."""
    lib().orc_half_split_index.restype = ctypes.c_int32
    return int(lib().orc_half_split_index(ctypes.c_int32(int(c))))


def relayout_keys_to_half_split(x):
    """x[..., 128] in interleaved rotary order -> the same values in half-split order."""
    x = np.asarray(x)
    out = np.empty_like(x)
    for c in range(HEAD_DIM):
        out[..., half_split_index(c)] = x[..., c]
    return out


def num_threads():
    return int(lib().orc_num_threads())
