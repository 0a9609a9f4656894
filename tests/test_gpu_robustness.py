"""GPU tests of what surrounds the arithmetic: workspace reuse, guard bytes around every buffer the library writes,
the exponent-range flag, and a drill of the bounded device-side wait (no fault and no hang is ever provoked)."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2606_29986_b200 import hma, synth
from helpers import Scenario, bf16_bits, parity_metrics

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
SCALE = 1.0 / np.sqrt(128.0)


def _attend(sc, ws, dtype=torch.float32):
    out = torch.full((sc.B, sc.hq, 128), float("nan"), dtype=dtype, device="cuda")
    hma.hma_decode_attention(sc.cache, 0, sc.q, out, sc.table, sc.ctx, SCALE, ws)
    torch.cuda.synchronize()
    return out


def test_one_workspace_serves_calls_of_any_shape_and_is_left_clean():
    """The arrival counters at the head of the workspace are zero again after every call, so one zero-filled
    workspace can be handed to calls of different batches and head counts, in any order."""
    a = Scenario([6000, 40, 2500, 16, 0, 777], 64, 8, seed=201, permute=True)      # segments shared by many CTAs
    b = Scenario([300] * 40, 32, 8, seed=202)                                      # many short segments
    c = Scenario([33, 5000], 8, 1, seed=203, permute=True)
    want = [_attend(s, s.workspace) for s in (a, b, c)]
    big = hma.new_workspace(b.desc, 64)                                            # large enough for all three
    assert big.numel() >= max(s.workspace.numel() for s in (a, b, c))
    for s, w in list(zip((a, b, c), want)) * 2 + [(a, want[0])]:
        got = _attend(s, big)
        assert torch.equal(got, w)
        assert not big[:1024 * 64 * 4].any()                                       # the counter region at the head of the workspace
    # a workspace that was never zero-filled is the caller's error, but it must not hang or fault: garbage counters
    # only mean that segments shared between CTAs may stay unmerged
    dirty = torch.full_like(big, 0x7F)
    _attend(c, dirty)
    assert hma.hma_error_flags(c.cache) == 0


def test_guard_bytes_around_everything_the_library_writes():
    """Sentinels before and after the workspace, the outputs, the dequant output and the cache layer stay intact
    through ingest, attention (both output types), the built-in-scratch variant, dequant and the probes."""
    lens = [700, 33, 16, 0, 2100]
    hq, hkv, G = 32, 8, 256
    table, num_pages, _ = synth.block_table(np.asarray(lens, np.int32), True, 5, 2)
    desc = hma.make_desc(1, hq, hkv, num_pages)
    layer_bytes = hma.hma_cache_layer_bytes(desc)

    def guarded(nbytes):
        buf = torch.full((nbytes + 2 * G,), 0xC3, dtype=torch.uint8, device="cuda")
        return buf, buf[G:G + nbytes]

    def intact(buf, nbytes):
        return bool((buf[:G] == 0xC3).all()) and bool((buf[G + nbytes:] == 0xC3).all())

    # the cache layer itself lives between guards: hma_cache_create takes the pointer
    import ctypes
    lbuf, layer = guarded(layer_bytes)
    handle = ctypes.c_void_p()
    ptrs = (ctypes.c_void_p * 1)(layer.data_ptr())
    assert hma.lib().hma_cache_create(ctypes.byref(desc), ptrs, ctypes.byref(handle)) == 0

    class C:      # the shape the binding expects
        pass
    cache = C()
    cache.handle, cache.desc = handle, desc
    tbl, ctx = torch.from_numpy(table).cuda(), torch.tensor(lens, dtype=torch.int32, device="cuda")
    wires = []
    for b, T in enumerate(lens):
        if not T:
            wires.append(None)
            continue
        kw, vw = synth.make_kv_wire(hkv, T, 900 + b), synth.make_kv_wire(hkv, T, 950 + b)
        wires.append((kw, vw))
        kb, kview = guarded(kw.numel())
        vb, vview = guarded(vw.numel())
        kview.copy_(kw.reshape(-1).cuda())
        vview.copy_(vw.reshape(-1).cuda())
        hma.hma_kv_ingest_layer(cache, 0, kview, vview, hma.HMA_WIRE_ROWMAJOR, 0, hkv, tbl[b, :(T + 15) // 16].contiguous(), 0, T)
        torch.cuda.synchronize()
        assert intact(kb, kw.numel()) and intact(vb, vw.numel())
    assert intact(lbuf, layer_bytes)
    ws_bytes = hma.hma_decode_attention_workspace_bytes(desc, len(lens))
    wbuf, ws = guarded((ws_bytes + 255) // 256 * 256)
    ws.zero_()
    q = synth.make_q(len(lens), hq, 7).cuda()
    for dtype, esz in ((torch.float32, 4), (torch.bfloat16, 2)):
        n = len(lens) * hq * 128 * esz
        obuf, oview = guarded(n)
        out = oview.view(dtype).view(len(lens), hq, 128)
        hma.hma_decode_attention(cache, 0, q, out, tbl, ctx, SCALE, ws)
        hma.hma_decode_attention_static(cache, 0, q, out, tbl, ctx, SCALE)
        hma.hma_kv_read_probe(cache, 0, tbl, ctx, ws)
        hma.hma_attention_alu_probe(cache, 0, tbl, ctx, ws)
        torch.cuda.synchronize()
        assert intact(obuf, n) and intact(wbuf, ws.numel()) and intact(lbuf, layer_bytes)
        assert torch.isfinite(out.float()).all()
    T = lens[4]
    dbuf, dview = guarded(T * hkv * 128 * 2)
    deq = dview.view(torch.bfloat16).view(T, hkv, 128)
    from oracle import oracle as orc
    for which in (0, 1):
        hma.hma_bfp8_dequant_bf16(cache, 0, which, tbl[4, :(T + 15) // 16].contiguous(), 0, T, deq)
        torch.cuda.synchronize()
        assert intact(dbuf, T * hkv * 128 * 2)
        assert np.array_equal(bf16_bits(deq).transpose(1, 0, 2), orc.decode_rowmajor_bf16(wires[4][which].numpy()))
    assert hma.hma_error_flags(cache) == 0
    hma.lib().hma_cache_destroy(handle)


def test_block_exponents_beyond_the_supported_range_raise_a_flag():
    """V block exponents above 250, and K exponents that overflow fp32 scores, are outside the kernel's range: the
    call returns, HMA_FLAG_EXPONENT_RANGE is set, sequences that do not contain such blocks are unaffected."""
    sc = Scenario([64, 48], 8, 1, seed=301, extra_pages=0)
    good = sc.attention(0, torch.float32).cpu().numpy()
    assert hma.hma_error_flags(sc.cache) == 0
    for tensor in ("v", "k"):
        kw, vw = sc.k_wires[0][0].copy(), sc.v_wires[0][0].copy()
        if tensor == "v":
            vw[0, 5, 3] = 253                     # one V block of token 5 with exponent 253
        else:
            kw[0, :, :8] = 254                    # every K block of the sequence: scores overflow
        hma.hma_kv_ingest_layer(sc.cache, 0, torch.from_numpy(kw).cuda(), torch.from_numpy(vw).cuda(), hma.HMA_WIRE_ROWMAJOR, 0, 1,
                                sc.table[0, :4].contiguous(), 0, 64)
        out = sc.attention(0, torch.float32).cpu().numpy()
        assert hma.hma_error_flags(sc.cache) & hma.HMA_FLAG_EXPONENT_RANGE, tensor
        assert np.array_equal(out[1], good[1])    # the other sequence is untouched
    # an exponent of exactly 250 is still inside the range and exact enough
    kw, vw = sc.k_wires[0][0].copy(), sc.v_wires[0][0].copy()
    vw[0, :, 3] = 250
    hma.hma_kv_ingest_layer(sc.cache, 0, torch.from_numpy(kw).cuda(), torch.from_numpy(vw).cuda(), hma.HMA_WIRE_ROWMAJOR, 0, 1,
                            sc.table[0, :4].contiguous(), 0, 64)
    out = sc.attention(0, torch.float32).cpu().numpy().astype(np.float64)
    assert hma.hma_error_flags(sc.cache) == 0
    from oracle import oracle as orc
    ref, _ = orc.decode_attention(bf16_bits(sc.q), [kw, sc.k_wires[0][1]], [vw, sc.v_wires[0][1]], 1)
    blk = slice(48, 64)
    assert np.sqrt(((out[0, :, blk] - ref[0, :, blk]) ** 2).sum() / (ref[0, :, blk] ** 2).sum()) <= 2e-3


_DRILL = r"""
import json, sys
import numpy as np, torch
sys.path.insert(0, %r)
sys.path.insert(0, %r)
from paper_2606_29986_b200 import hma
from helpers import Scenario
sc = Scenario([4000, 4000, 4000, 4000], 8, 1, seed=401)
scale = 1.0 / np.sqrt(128.0)
def run():
    out = torch.zeros((4, 8, 128), dtype=torch.float32, device="cuda")
    hma.hma_decode_attention(sc.cache, 0, sc.q, out, sc.table, sc.ctx, scale, sc.workspace)
    torch.cuda.synchronize()
    return out
good = run()
assert hma.hma_error_flags(sc.cache) == 0
assert hma.lib().hma_trace_arm_timeout_drill(10, 1000) == 0          # record 10: the first pages of sequence 0
bad = run()
flags = hma.hma_error_flags(sc.cache)
hma.hma_decode_attention_workspace_init(sc.workspace)                 # as the header asks after a timeout
again = run()
print(json.dumps({"flags": flags, "finite": bool(torch.isfinite(bad).all()), "far_rows_equal": bool(torch.equal(bad[2:], good[2:])),
                  "recovered": bool(torch.equal(again, good)), "flags_after": hma.hma_error_flags(sc.cache)}))
"""


def test_bounded_wait_runs_out_and_the_kernel_returns():
    """Drill of the device-side bounded wait, in a child process with the instrumented build: one record's arrival
    barrier expects 16 bytes more than its copy delivers, so the copy lands, the wait gives up after 1000 polls, the
    kernel returns, HMA_FLAG_WAIT_TIMEOUT is readable, rows of untouched sequences are bit-identical, and after
    re-zeroing the workspace the same call is right again."""
    from paper_2606_29986_b200 import build
    env = dict(os.environ, HMA_LIBRARY=build.build(trace=True))
    res = subprocess.run([sys.executable, "-c", _DRILL % (ROOT, os.path.join(ROOT, "tests"))], env=env, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0, res.stderr[-3000:]
    r = json.loads(res.stdout.strip().splitlines()[-1])
    assert r["flags"] & hma.HMA_FLAG_WAIT_TIMEOUT, r
    assert r["finite"] and r["far_rows_equal"] and r["recovered"] and r["flags_after"] == 0, r
