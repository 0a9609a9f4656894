#!/usr/bin/env python
"""Benchmark of the decode-side BFP8 KV path (one JSON line on stdout).

A step is one decode pass of the whole batch: for every layer one hma_decode_attention call
(fused BFP8 paged attention + cross-split reduction) on the main stream while, for the
Qwen3-32B workload, one new 8192-token request's raw BFP8 bytes are ingested layer by layer
on a side stream (hma_kv_ingest_layer_shards, TILE32 wire, 4 producer shards).  `value` is decode
tokens per second (batch / step time) with every input resident in HBM; `e2e` repeats the
step with Q, the arriving wire bytes and the outputs in pinned host memory.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
"""
import argparse
import json
import os
import shutil
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2606_29986_b200 import synth  # noqa: E402

DEFAULT_WORKLOAD = "qwen3-32b-b32-ctx8k"
BFP8_ROW = 272      # bytes per (token, kv head): K 136 + V 136
BF16_ROW = 512
# DRAM bytes per launch of the attention kernel as one ncu capture of this workload counted them
# (dram__bytes_read.sum + dram__bytes_write.sum); None where no capture exists.
NCU_TRAFFIC_BYTES = {"qwen3-32b-b32-ctx8k": 575_000_000}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        exe = shutil.which("nvidia-smi")
        if not exe:
            return
        self.proc = subprocess.Popen([exe, "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                      "--format=csv,noheader,nounits", "-lms", "20"],
                                     stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["not recorded: nvidia-smi absent"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ----------------------------------------------------------------------------- workload on the GPU
class Workload:
    def __init__(self, name, device, seed=0, with_bf16=True, with_ingest=True, layers=None):
        from paper_2606_29986_b200 import hma
        self.hma, self.name, self.device = hma, name, device
        w = synth.WORKLOADS[name]
        self.hq, self.hkv, self.B, self.L = w["hq"], w["hkv"], w["batch"], layers or w["layers"]
        self.lens = synth.context_lens(w["ctx"], self.B, seed)
        self.sum_t = int(self.lens.sum())
        self.ingest_tokens = 8192 if (with_ingest and name == DEFAULT_WORKLOAD) else 0
        extra = (self.ingest_tokens + 15) // 16
        table, self.num_pages, spare = synth.block_table(self.lens, w["permute"], seed, extra)
        self.table = torch.from_numpy(table).to(device)
        self.ctx = torch.from_numpy(self.lens).to(device)
        self.spare = torch.from_numpy(np.ascontiguousarray(spare)).to(device)
        self.sm_scale = 1.0 / np.sqrt(128.0)
        self.caches = {"bfp8": hma.KVCache(hma.make_desc(self.L, self.hq, self.hkv, self.num_pages, hma.HMA_KV_BFP8), device)}
        if with_bf16:
            self.caches["bf16"] = hma.KVCache(hma.make_desc(self.L, self.hq, self.hkv, self.num_pages, hma.HMA_KV_BF16), device)
        self.q = [synth.make_q(self.B, self.hq, seed + l, device) for l in range(self.L)]
        self.out = torch.empty((self.L, self.B, self.hq, 128), dtype=torch.bfloat16, device=device)
        self.workspace = hma.new_workspace(self.caches["bfp8"].desc, self.B, device)
        self.sample_wires = {}       # (layer, b) -> (k_wire, v_wire) numpy: wire bytes of a few sequences, for the parity tests
        keep = {(0, 0), (self.L - 1, self.B - 1), (0, int(np.argmin(self.lens))), (self.L - 1, int(np.argmax(self.lens)))}
        for l in range(self.L):
            for b in range(self.B):
                T = int(self.lens[b])
                kw = synth.make_kv_wire(self.hkv, T, synth.sequence_seed(seed, l, b, 0), device, synth.channel_seed(seed, l, 0))
                vw = synth.make_kv_wire(self.hkv, T, synth.sequence_seed(seed, l, b, 1), device, synth.channel_seed(seed, l, 1))
                pages = self.table[b, :(T + 15) // 16].contiguous()
                for c in self.caches.values():
                    hma.hma_kv_ingest_layer(c, l, kw, vw, hma.HMA_WIRE_ROWMAJOR, 0, self.hkv, pages, 0, T)
                if (l, b) in keep:
                    self.sample_wires[(l, b)] = (kw.cpu().numpy(), vw.cpu().numpy())
            torch.cuda.synchronize(device)
        # the arriving request: TILE32 wire, 4 shards x (hkv/4) heads, every layer, K and V
        # decode and the arriving request's ingest run on two streams of equal priority (measured: giving either one
        # a higher priority makes the step slower, because the favoured kernel's CTAs then sit on freed SMs waiting)
        self.side = torch.cuda.Stream(device)
        self.main = torch.cuda.Stream(device)
        if self.ingest_tokens:
            hs = self.hkv // 4
            one = synth.rowmajor_to_tile32(synth.make_kv_wire(hs, self.ingest_tokens, 4242, device)).reshape(-1)
            self.shard_bytes = one.numel()
            self.wire_dev = torch.empty((self.L, 2, 4, self.shard_bytes), dtype=torch.uint8, device=device)
            for l in range(self.L):
                for t in range(2):
                    for s in range(4):
                        seed_ls = 4242 + ((l * 2 + t) * 4 + s)
                        self.wire_dev[l, t, s] = synth.rowmajor_to_tile32(
                            synth.make_kv_wire(hs, self.ingest_tokens, seed_ls, device)).reshape(-1)
            self.wire_host = torch.empty(self.wire_dev.shape, dtype=torch.uint8, pin_memory=True)
            self.wire_host.copy_(self.wire_dev)
            self.wire_stage = torch.empty((2,) + tuple(self.wire_dev.shape[1:]), dtype=torch.uint8, device=device)
        self.q_host = torch.empty((self.L, self.B, self.hq, 128), dtype=torch.bfloat16, pin_memory=True)
        for l in range(self.L):
            self.q_host[l].copy_(self.q[l])
        self.out_host = torch.empty(self.out.shape, dtype=torch.bfloat16, pin_memory=True)
        self.q_stage = torch.empty((self.L, self.B, self.hq, 128), dtype=torch.bfloat16, device=device)
        torch.cuda.synchronize(device)

    def kv_bytes_per_layer(self, fmt):
        return self.sum_t * self.hkv * (BFP8_ROW if fmt == "bfp8" else BF16_ROW)

    def _ingest_all(self, wire, stream, staged=False, layers=None):
        """Ingest every layer of the arriving request on `stream`.  With `staged`, each layer's pinned host bytes are
        first copied to a device staging buffer by the copy engine (same stream), then scattered from there."""
        hma = self.hma
        hs = self.hkv // 4
        if layers is None:
            todo = range(self.L)
        else:       # `layers` layers per step, continuing where the previous step stopped (a request arriving over many steps)
            todo = [(self._ingest_next + i) % self.L for i in range(layers)]
            self._ingest_next = (self._ingest_next + layers) % self.L
        for l in todo:
            src = wire[l]
            if staged:
                with torch.cuda.stream(stream):
                    self.wire_stage[l & 1].copy_(wire[l], non_blocking=True)
                src = self.wire_stage[l & 1]
            hma.hma_kv_ingest_layer_shards(self.caches["bfp8"], l, [src[0, s] for s in range(4)], [src[1, s] for s in range(4)],
                                           hma.HMA_WIRE_TILE32, [s * hs for s in range(4)], [hs] * 4, self.spare, 0,
                                           self.ingest_tokens, stream)

    _ingest_next = 0

    def plan_for(self, fmt):
        """The plan buffer of a cache (allocated once); hma_decode_attention_plan refills it at the start of every step."""
        if not hasattr(self, "plans"):
            self.plans = {}
        if fmt not in self.plans:
            self.plans[fmt] = self.hma.hma_decode_attention_plan(self.caches[fmt], self.table, self.ctx)
        return self.plans[fmt]

    def step(self, fmt="bfp8", ingest=True, host=False, staged=True, ingest_layers=None, planned=True):
        """One decode pass over all layers (+ the concurrent ingest).  Everything is enqueued; nothing syncs.  With `planned`
        the kernel's set-up is computed once per step (hma_decode_attention_plan, inside the step) and every layer's call
        reads it; without, every call works it out again (hma_decode_attention)."""
        hma = self.hma
        main = torch.cuda.current_stream(self.device)
        do_ingest = ingest and self.ingest_tokens and fmt == "bfp8"
        if do_ingest:
            self.side.wait_stream(main)
            self._ingest_all(self.wire_host if host else self.wire_dev, self.side, staged=host and staged, layers=ingest_layers)
        cache = self.caches[fmt]
        if planned:
            plan = hma.hma_decode_attention_plan(cache, self.table, self.ctx, plan=self.plan_for(fmt), stream=main)
        for l in range(self.L):
            q = self.q[l]
            if host:
                self.q_stage[l].copy_(self.q_host[l], non_blocking=True)
                q = self.q_stage[l]
            if planned:
                hma.hma_decode_attention_planned(cache, l, q, self.out[l], self.table, self.ctx, self.sm_scale, plan, self.workspace, main)
            else:
                hma.hma_decode_attention(cache, l, q, self.out[l], self.table, self.ctx, self.sm_scale, self.workspace, main)
            if host:
                self.out_host[l].copy_(self.out[l], non_blocking=True)
        if do_ingest:
            main.wait_stream(self.side)

    def time_steps(self, steps, warmup, **kw):
        for _ in range(warmup):
            self.step(**kw)
        torch.cuda.synchronize(self.device)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(self.device)
        e0.record()
        for _ in range(steps):
            self.step(**kw)
        e1.record()
        torch.cuda.synchronize(self.device)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1) / 1e3) / steps      # seconds per step

    def time_calls(self, kinds, passes, fmt="bfp8"):
        """Duration of single calls, CUDA events around every call on its stream.  `kinds` lists what to time
        ("attn": hma_decode_attention_planned with the step's plan, "attn_self": hma_decode_attention, "probe": hma_kv_read_probe, "alu": hma_attention_alu_probe, "hbm": a plain
        contiguous read of the layer's bytes); the kinds are interleaved call by call, layer after layer, so that
        every kind sees the same clocks and the same cold L2.  Returns kind -> (mean, median, min) in seconds."""
        cache = self.caches[fmt]
        if not hasattr(self, "sink"):
            self.sink = torch.zeros(1, dtype=torch.int32, device=self.device)
        evs = {k: [] for k in kinds}
        plan = self.plan_for(fmt)
        self.hma.hma_decode_attention_plan(cache, self.table, self.ctx, plan=plan)
        for r in range(passes):
            for l in range(self.L):
                for kind in kinds:
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    if kind == "alu":
                        self.hma.hma_attention_alu_probe(cache, l, self.table, self.ctx, self.workspace)
                    elif kind == "probe":
                        self.hma.hma_kv_read_probe(cache, l, self.table, self.ctx, self.workspace)
                    elif kind == "hbm":
                        self.hma.hma_hbm_read_probe(cache.layers[l], self.sink)
                    elif kind == "attn_self":
                        self.hma.hma_decode_attention(cache, l, self.q[l], self.out[l], self.table, self.ctx, self.sm_scale, self.workspace)
                    else:
                        self.hma.hma_decode_attention_planned(cache, l, self.q[l], self.out[l], self.table, self.ctx, self.sm_scale, plan,
                                                              self.workspace)
                    b.record()
                    evs[kind].append((a, b))
        torch.cuda.synchronize(self.device)
        res = {}
        for kind in kinds:
            t = np.array([a.elapsed_time(b) for a, b in evs[kind]]) / 1e3
            res[kind] = (float(t.mean()), float(np.median(t)), float(t.min()))
        return res

    def time_alternating(self, variants, rounds=4, steps=4):
        """Seconds per step of several step() variants measured in alternation (variant 0, 1, .., 0, 1, ..), so that all see
        the same clocks: under its power cap the GPU runs a long sequence of steps up to 10 % slower than a short one, which
        would otherwise be charged to whichever variant is timed later.  Returns the mean over the rounds per variant."""
        for kw in variants:
            self.step(**kw)
        torch.cuda.synchronize(self.device)
        tot = [0.0] * len(variants)
        for _ in range(rounds):
            for i, kw in enumerate(variants):
                tot[i] += self.time_steps(steps, 0, **kw)
        return [t / rounds for t in tot]

    def time_layer_calls(self, fmt, reps, probe=False):
        """Average duration of one hma_decode_attention call (or of one probe call), back to back."""
        kind = "alu" if probe == "alu" else "probe" if probe else "attn"
        return self.time_calls([kind], reps, fmt)[kind]

    def time_ingest(self, reps=5):
        """GPU time of the ingest alone (device-resident wire, every layer of the arriving request), replayed from a CUDA
        graph so that host launch overhead does not count; seconds per layer."""
        s = torch.cuda.Stream(self.device)
        s.wait_stream(torch.cuda.current_stream(self.device))
        with torch.cuda.stream(s):
            self._ingest_all(self.wire_dev, s)
            torch.cuda.synchronize(self.device)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                self._ingest_all(self.wire_dev, s)
            g.replay()
            torch.cuda.synchronize(self.device)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            torch.cuda.synchronize(self.device)
            # the same harness around the plainest kernel with the same byte counts: one launch per layer that reads the
            # layer's wire bytes and writes as many to a buffer of its own
            dst = torch.empty_like(self.wire_dev)
            nbytes = self.wire_dev[0].numel()

            def copies():
                for l in range(self.L):
                    self.hma.hma_hbm_copy_probe(self.wire_dev[l], nbytes, dst[l], nbytes, s)
            copies()
            torch.cuda.synchronize(self.device)
            gc = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gc, stream=s):
                copies()
            gc.replay()
            torch.cuda.synchronize(self.device)
            c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            c0.record()
            for _ in range(reps):
                gc.replay()
            c1.record()
            torch.cuda.synchronize(self.device)
            self.copy_probe_layer_s = c0.elapsed_time(c1) / 1e3 / reps / self.L
            del dst
            # every layer of the request in one call (hma_kv_ingest_request_shards): the same bytes in one launch
            hs = self.hkv // 4
            w = self.wire_dev

            def whole():
                self.hma.hma_kv_ingest_request_shards(self.caches["bfp8"], [w[0, 0, i] for i in range(4)], [w[0, 1, i] for i in range(4)],
                                                      2 * 4 * self.shard_bytes, self.hma.HMA_WIRE_TILE32, [i * hs for i in range(4)],
                                                      [hs] * 4, self.spare, 0, self.ingest_tokens, s)
            whole()
            torch.cuda.synchronize(self.device)
            c0.record()
            for _ in range(reps):
                whole()
            c1.record()
            torch.cuda.synchronize(self.device)
            self.ingest_request_s = c0.elapsed_time(c1) / 1e3 / reps
        torch.cuda.current_stream(self.device).wait_stream(s)
        return e0.elapsed_time(e1) / 1e3 / reps / self.L

    def time_mixed(self, tail_tokens=64, reps=3):
        """hma_decode_attention_mixed: the BFP8 cache as prefix plus a BF16 cache holding `tail_tokens` decode-side tokens per
        sequence (plain BF16 rows); mean seconds per call."""
        hma = self.hma
        lens = np.full(self.B, tail_tokens, np.int32)
        table, num_pages, _ = synth.block_table(lens, True, 99)
        tail = hma.KVCache(hma.make_desc(self.L, self.hq, self.hkv, num_pages, hma.HMA_KV_BF16), self.device)
        ttable, tlens = torch.from_numpy(table).to(self.device), torch.from_numpy(lens).to(self.device)
        g = torch.Generator(device=self.device)
        g.manual_seed(99)
        rows = torch.randn((self.hkv, tail_tokens, 128), generator=g, device=self.device).to(torch.bfloat16)
        for l in range(self.L):
            for b in range(self.B):
                hma.hma_kv_ingest_layer(tail, l, rows, rows, hma.HMA_WIRE_BF16_ROWS, 0, self.hkv, ttable[b].contiguous(), 0, tail_tokens)
        ws = hma.new_workspace(self.caches["bfp8"].desc, self.B, self.device, copies=2)
        pplan = hma.hma_decode_attention_plan(self.caches["bfp8"], self.table, self.ctx)
        tplan = hma.hma_decode_attention_plan(tail, ttable, tlens)

        def run():          # two plans per pass over the layers, then planned calls
            hma.hma_decode_attention_plan(self.caches["bfp8"], self.table, self.ctx, plan=pplan)
            hma.hma_decode_attention_plan(tail, ttable, tlens, plan=tplan)
            for l in range(self.L):
                hma.hma_decode_attention_mixed_planned(self.caches["bfp8"], tail, l, self.q[l], self.out[l], self.table, self.ctx, ttable,
                                                       tlens, self.sm_scale, pplan, tplan, ws)
        run()
        torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize(self.device)
        return e0.elapsed_time(e1) / 1e3 / reps / self.L

    def time_pcie(self, reps=3):
        """Host-to-device copy rate of this machine: the arriving request's pinned wire bytes (or 1 GiB of pinned memory)
        copied to a device buffer by the copy engine, best of `reps`; GB/s."""
        src = self.wire_host.view(-1) if self.ingest_tokens else torch.empty(1 << 30, dtype=torch.uint8, pin_memory=True)
        dst = torch.empty(src.numel(), dtype=torch.uint8, device=self.device)
        best = 1e30
        for _ in range(reps + 1):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dst.copy_(src, non_blocking=True)
            e1.record()
            torch.cuda.synchronize(self.device)
            best = min(best, e0.elapsed_time(e1) / 1e3)
        return src.numel() / best / 1e9

    def time_multi_query(self, q_len, reps=3):
        """hma_decode_attention_planned with q_len query tokens per sequence (the last q_len cached tokens; the planned form of
        hma_decode_attention_multi): mean seconds per call, the pass's one plan launch included."""
        hma = self.hma
        q = synth.make_q(self.B * q_len, self.hq, 4321, self.device).view(self.B, q_len, self.hq, 128)
        out = torch.empty_like(q)
        ws = hma.new_workspace(self.caches["bfp8"].desc, self.B * q_len, self.device)

        plan = hma.hma_decode_attention_plan(self.caches["bfp8"], self.table, self.ctx, q_len=q_len)

        def run():          # one plan per pass over the layers, as in step()
            hma.hma_decode_attention_plan(self.caches["bfp8"], self.table, self.ctx, q_len=q_len, plan=plan)
            for l in range(self.L):
                hma.hma_decode_attention_planned(self.caches["bfp8"], l, q, out, self.table, self.ctx, self.sm_scale, plan, ws)
        run()
        torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize(self.device)
        return e0.elapsed_time(e1) / 1e3 / reps / self.L

    def time_rebuild(self, reps=3):
        """One-shot BFP8 -> BF16 rebuild of one whole request (sequence 0: every layer, K and V): seconds, bytes moved."""
        T = int(self.lens[0])
        pages = self.table[0, :(T + 15) // 16].contiguous()
        out = torch.empty((self.L, 2, T, self.hkv, 128), dtype=torch.bfloat16, device=self.device)
        cache = self.caches["bfp8"]

        def run():
            self.hma.hma_bfp8_rebuild_request(cache, pages, 0, T, out)
        run()
        torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record()
        torch.cuda.synchronize(self.device)
        elems = 2 * self.L * T * self.hkv * 128
        fused = e0.elapsed_time(e1) / 1e3 / reps
        # the elementwise strawman, layer by layer and tensor by tensor
        def naive():
            for l in range(self.L):
                for which in (0, 1):
                    self.hma.hma_bfp8_dequant_bf16_naive(cache, l, which, pages, 0, T, out[l, which])
        naive()
        torch.cuda.synchronize(self.device)
        e0.record()
        naive()
        e1.record()
        torch.cuda.synchronize(self.device)
        self.naive_rebuild_s = e0.elapsed_time(e1) / 1e3
        # the plainest kernel with the same byte counts: reads 17 bytes for every 32 it writes, from one layer's cache
        src = cache.layers[0]
        rd = min(int(elems * 17 // 16), src.numel()) // 16 * 16
        wr_bytes = rd * 32 // 17 // 16 * 16
        dst = out.view(-1)
        self.hma.hma_hbm_copy_probe(src, rd, dst, wr_bytes)
        torch.cuda.synchronize(self.device)
        e0.record()
        for _ in range(reps):
            self.hma.hma_hbm_copy_probe(src, rd, dst, wr_bytes)
        e1.record()
        torch.cuda.synchronize(self.device)
        # scaled to the rebuild's bytes when one layer's cache is smaller than what the rebuild reads
        self.copy_probe_rebuild_s = e0.elapsed_time(e1) / 1e3 / reps * (elems * (17 / 16 + 2)) / (rd + wr_bytes)
        return fused, elems * (17 / 16 + 2), elems

# ----------------------------------------------------------------------------- ranks
def world():
    return int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0"))


def barrier():
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        torch.distributed.barrier()


def max_over_ranks(x):
    """Largest value of x over all ranks (the step time of the slowest rank)."""
    if torch.distributed.is_available() and torch.distributed.is_initialized():
        dev = "cuda" if torch.distributed.get_backend() == "nccl" else "cpu"
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        return float(t.item())
    return x


def aggregate_value(tokens_per_rank, seconds_per_step, n_ranks):
    """Whole-job tokens/s: every rank decodes its own batch (no data-path collective), time = slowest rank."""
    return tokens_per_rank * n_ranks / seconds_per_step


# ----------------------------------------------------------------------------- CPU oracle timing
def time_oracle(name, n_seq, seed=0, repeats=1):
    """Seconds the CPU oracle needs for one layer of `n_seq` sequences of the workload; returns (seconds, threads, tokens)."""
    from oracle import oracle as orc
    w = synth.WORKLOADS[name]
    lens = synth.context_lens(w["ctx"], w["batch"], seed)[:n_seq]
    q = synth.make_q(n_seq, w["hq"], seed).view(torch.int16).numpy().view(np.uint16)
    kw = [synth.make_kv_wire(w["hkv"], int(t), synth.sequence_seed(seed, 0, b, 0), channel_seed=synth.channel_seed(seed, 0, 0)).numpy() for b, t in enumerate(lens)]
    vw = [synth.make_kv_wire(w["hkv"], int(t), synth.sequence_seed(seed, 0, b, 1), channel_seed=synth.channel_seed(seed, 0, 1)).numpy() for b, t in enumerate(lens)]
    orc.decode_attention(q[:1], [kw[0][:, :64]], [vw[0][:, :64]], w["hkv"])      # load the library
    best = 1e30
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.decode_attention(q, kw, vw, w["hkv"])
        best = min(best, time.perf_counter() - t0)
    return best, orc.num_threads(), int(lens.sum())


def reference_arm(args):
    """The CPU oracle as it stands, on the host cores: each step is one layer of one sequence of the workload."""
    ws, rank, _ = world()
    if rank != 0:
        return
    name = args.workload
    w = synth.WORKLOADS[name]
    n_seq = 1
    for _ in range(args.warmup):
        time_oracle(name, n_seq)
    t = []
    threads = 1
    for _ in range(args.steps):
        sec, threads, toks = time_oracle(name, n_seq)
        t.append(sec)
    sec = float(np.mean(t))
    # one layer of n_seq sequences took `sec`; a decode token needs all layers
    value = n_seq / (sec * w["layers"])
    line = {"impl": "reference", "metric": "decode_attn_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "sample": "1 sequence x 1 layer per step, scaled to %d layers" % w["layers"]},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                             "sample": "layer 0 of sequence 0 (%d tokens, %d q heads) per step; tokens/s = 1 / (t * %d layers)" % (toks, w["hq"], w["layers"])},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-bf16", action="store_true", help="skip the BF16-KV comparison run")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--layers", type=int, default=None, help="development only: build fewer layers than the workload has")
    ap.add_argument("--kernel-only", action="store_true", help="development only: print per-call kernel timing and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        reference_arm(args)
        return

    ws, rank, local = world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library has no CPU fallback")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if ws > 1:
        torch.distributed.init_process_group("nccl", device_id=device)
    from paper_2606_29986_b200 import hma
    hma.lib()

    wl = Workload(args.workload, device, with_bf16=not args.no_bf16, layers=args.layers)
    torch.cuda.synchronize(device)
    torch.cuda.set_stream(wl.main)          # everything timed below is enqueued on the high-priority stream
    peak, peak_kind = measured_peak()


    sampler = ClockSampler(local)      # started early: nvidia-smi needs a moment before its first sample
    sampler.start()
    time.sleep(0.3)
    # per-call duration of the dominant kernel (decode attention), CUDA events around each call
    # (back to back, as inside a decode pass), then the two read ceilings interleaved with it call by call
    wl.time_layer_calls("bfp8", 1)
    call_mean, call_med, call_min = wl.time_layer_calls("bfp8", 5)
    wl.time_calls(["attn", "attn_self", "probe", "hbm"], 1)
    ceil = wl.time_calls(["attn", "attn_self", "probe", "hbm"], 5)
    self_mean, self_med, self_min = ceil["attn_self"]
    probe_mean, probe_med, probe_min = ceil["probe"]
    hbm_mean, hbm_med, hbm_min = ceil["hbm"]
    inter_mean, inter_med, inter_min = ceil["attn"]
    if args.kernel_only:
        wl.time_layer_calls("bfp8", 1, probe="alu")
        alu_mean = wl.time_layer_calls("bfp8", 3, probe="alu")[0]
        res = {"alu_probe_us_per_call": alu_mean * 1e6, "workload": args.workload, "layers_built": wl.L, "bfp8_us_per_call": [call_mean * 1e6, call_med * 1e6, call_min * 1e6],
               "bfp8_gbs": wl.kv_bytes_per_layer("bfp8") / call_mean / 1e9, "probe_us_per_call": [probe_mean * 1e6, probe_med * 1e6, probe_min * 1e6],
               "probe_gbs": wl.kv_bytes_per_layer("bfp8") / probe_med / 1e9,
               "bfp8_us_per_call_interleaved": [inter_mean * 1e6, inter_med * 1e6, inter_min * 1e6],
               "hbm_read_us": [hbm_mean * 1e6, hbm_med * 1e6, hbm_min * 1e6],
               "hbm_read_gbs": wl.caches["bfp8"].layers[0].numel() / hbm_med / 1e9}
        if "bf16" in wl.caches:
            wl.time_layer_calls("bf16", 1)
            m, md, mn = wl.time_layer_calls("bf16", 2)
            res.update({"bf16_us_per_call": [m * 1e6, md * 1e6, mn * 1e6], "bf16_gbs": wl.kv_bytes_per_layer("bf16") / m / 1e9})
        sampler.stop()
        print(json.dumps(res))
        return

    sec = wl.time_steps(args.steps, args.warmup)
    clocks = sampler.stop()
    n0 = hma.hma_launch_count()
    wl.step()
    launches = hma.hma_launch_count() - n0          # kernels of this library per step
    torch.cuda.synchronize(device)

    sec_decode_only = wl.time_steps(args.steps, args.warmup, ingest=False)
    # what the plan buys: steps with one plan per step against steps whose every call sets itself up, in alternation
    alt_planned, alt_self = wl.time_alternating([dict(ingest=False), dict(ingest=False, planned=False)])
    # the ingest's cost to decode, each pair measured in alternation (same clocks for both sides)
    alt_ingest, alt_plain = wl.time_alternating([dict(), dict(ingest=False)]) if wl.ingest_tokens else (sec, sec)
    # the same request arriving at the rate of the paper's 100 Gb link (92.3 Gb/s measured, section 3.2): layers per step
    paced = {}
    if wl.ingest_tokens:
        layer_bytes = 2 * 4 * wl.shard_bytes
        per_step = max(1, int(round(92.3e9 / 8 * sec_decode_only / layer_bytes)))
        sec_paced = wl.time_steps(args.steps, args.warmup, ingest_layers=per_step)
        alt_paced, alt_plain2 = wl.time_alternating([dict(ingest_layers=per_step), dict(ingest=False)])
        paced = {"layers_per_step": per_step, "link_gbit_s": 92.3, "ms_per_step": sec_paced * 1e3,
                 "tokens_per_s": aggregate_value(wl.B, sec_paced, ws), "slowdown_vs_decode_only": alt_paced / alt_plain2 - 1.0,
                 "how": "slowdown from steps with and without the paced ingest timed in alternation (4 rounds of 4 steps each)"}
    sec_e2e = wl.time_steps(max(2, args.steps // 4), 3, host=True)
    sec_e2e_mapped = wl.time_steps(max(2, args.steps // 4), 3, host=True, staged=False) if wl.ingest_tokens else sec_e2e
    pcie_gbs = wl.time_pcie()
    e2e_paced = {}
    if wl.ingest_tokens:
        # end to end at the paper's operating point: the request's bytes arrive from the host at the link's rate
        sec_e2e_paced = wl.time_steps(max(2, args.steps // 4), 3, host=True, ingest_layers=paced["layers_per_step"])
        e2e_paced = {"layers_per_step": paced["layers_per_step"], "ms_per_step": sec_e2e_paced * 1e3,
                     "tokens_per_s": aggregate_value(wl.B, sec_e2e_paced, ws),
                     "h2d_bytes_per_step": wl.L * wl.B * wl.hq * 128 * 2 + paced["layers_per_step"] * 2 * 4 * wl.shard_bytes,
                     "slowdown_vs_decode_only_resident_inputs": sec_e2e_paced / sec_decode_only - 1.0}
    extra = {}
    if "bf16" in wl.caches:
        k = max(5, args.steps // 4)
        sec_bf16 = wl.time_steps(k, 3, fmt="bf16", ingest=False)
        extra["bf16_kv"] = {"tokens_per_s": aggregate_value(wl.B, sec_bf16, ws), "ms_per_step": sec_bf16 * 1e3,
                            "kv_gbs": wl.kv_bytes_per_layer("bf16") * wl.L / sec_bf16 / 1e9, "steps": k,
                            "bfp8_speedup": sec_bf16 / sec_decode_only}
        alt_bf16, alt_bfp8 = wl.time_alternating([dict(fmt="bf16", ingest=False), dict(ingest=False)], rounds=3, steps=3)
        extra["bf16_kv"]["bfp8_speedup_alternating"] = alt_bf16 / alt_bfp8

    t_rb, rb_bytes, rb_elems = wl.time_rebuild()
    extra["rebuild_request"] = {"ms": t_rb * 1e3, "tokens": int(wl.lens[0]), "layers": wl.L, "gbs": rb_bytes / t_rb / 1e9,
                                "frac_of_peak": rb_bytes / t_rb / 1e9 / peak, "calls": 1,
                                "naive_elementwise_ms": wl.naive_rebuild_s * 1e3, "fused_speedup_over_naive": wl.naive_rebuild_s / t_rb,
                                "copy_probe_ms": wl.copy_probe_rebuild_s * 1e3, "frac_of_copy_probe": wl.copy_probe_rebuild_s / t_rb,
                                "copy_probe": "hma_hbm_copy_probe: a plain streaming kernel that reads 17 bytes for every 32 it writes, same byte counts",
                                "what": "hma_bfp8_rebuild_request: one request, K and V, all layers, one launch (1.0625 B in + 2 B out per element)"}
    if wl.ingest_tokens:
        t_ing = wl.time_ingest()
        layer_bytes = 2 * 4 * wl.shard_bytes
        extra["ingest_alone"] = {"us_per_layer": t_ing * 1e6, "gbs_read_plus_write": 2 * layer_bytes / t_ing / 1e9,
                                 "frac_of_peak": 2 * layer_bytes / t_ing / 1e9 / peak,
                                 "copy_probe_us_per_layer": wl.copy_probe_layer_s * 1e6, "frac_of_copy_probe": wl.copy_probe_layer_s / t_ing,
                                 "whole_request_one_call": {"ms": wl.ingest_request_s * 1e3, "gbs_read_plus_write": 2 * layer_bytes * wl.L / wl.ingest_request_s / 1e9,
                                                            "frac_of_peak": 2 * layer_bytes * wl.L / wl.ingest_request_s / 1e9 / peak,
                                                            "what": "hma_kv_ingest_request_shards: every layer of the same request in one launch"},
                                 "copy_probe": "hma_hbm_copy_probe in the same harness: one plain launch per layer that reads the layer's wire bytes and writes as many",
                                 "what": "hma_kv_ingest_layer_shards, one 8192-token layer (4 shards, TILE32), device-resident wire, CUDA-graph replay"}
    t_mixed = wl.time_mixed()
    extra["mixed_prefix_tail"] = {"us_per_call": t_mixed * 1e6, "tail_tokens_per_sequence": 64,
                                  "what": "hma_decode_attention_mixed_planned: BFP8 prefix cache + BF16 cache with 64 decode-side tokens per sequence (two plans per pass)",
                                  "overhead_vs_prefix_only": t_mixed / call_mean - 1.0}
    mq = {"what": "hma_decode_attention_planned with q_len query tokens per sequence over the same cache (speculative / chunked decode; "
                  "the planned form of hma_decode_attention_multi, one plan per pass over the layers); "
                  "tokens/s counts query tokens, attention only, all layers"}
    base_call = wl.time_multi_query(1)
    for q_len in (1, 2, 4):
        t = base_call if q_len == 1 else wl.time_multi_query(q_len)
        mq["q_len_%d" % q_len] = {"us_per_call": t * 1e6, "tokens_per_s": wl.B * q_len / (t * wl.L), "per_token_speedup": q_len * base_call / t}
    extra["multi_query"] = mq
    kv_step = wl.kv_bytes_per_layer("bfp8") * wl.L
    value = aggregate_value(wl.B, sec, ws)
    achieved = wl.kv_bytes_per_layer("bfp8") / call_mean / 1e9
    q_bytes = wl.L * wl.B * wl.hq * 128 * 2
    wire_bytes = int(wl.wire_host.numel()) if wl.ingest_tokens else 0
    line = {
        "metric": "decode_attn_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": ws, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bfp8 bytes (u8) -> f16 mma operands, f32 accumulate", "data": "synthetic",
        "config": {"workload": args.workload, "q_heads": wl.hq, "kv_heads": wl.hkv, "batch_per_gpu": wl.B, "layers": wl.L,
                   "sum_context": wl.sum_t, "page_tokens": 16, "kv_format": "bfp8", "parallelism": "replicas only",
                   "layers_built": wl.L, "concurrent_ingest_tokens": wl.ingest_tokens, "l2": "inputs_larger_than_l2 (%.0f MB per layer, %d distinct layers)"
                   % (wl.kv_bytes_per_layer("bfp8") / 1e6, wl.L)},
        "kv_gbs": kv_step * ws / sec / 1e9,
        "kv_gbs_frac_of_8000": kv_step / sec / 1e9 / 8000.0,
        "clocks": clocks,
        "e2e": {"value": aggregate_value(wl.B, sec_e2e, ws), "unit": "tokens/s", "ms_per_step": sec_e2e * 1e3,
                "h2d_bytes_per_step": q_bytes + wire_bytes, "d2h_bytes_per_step": q_bytes,
                "ingest_source": "pinned host -> device staging (copy engine) -> hma_kv_ingest_layer",
                "ms_per_step_mapped_reads": sec_e2e_mapped * 1e3,
                "pcie_h2d_gbs_measured": pcie_gbs,
                "h2d_gbs": (q_bytes + wire_bytes) / sec_e2e / 1e9,
                "frac_of_pcie": (q_bytes + wire_bytes) / sec_e2e / 1e9 / pcie_gbs,
                "at_link_rate": e2e_paced},
        "gpu_launches": int(launches * args.steps),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": "of " + peak_kind, "frac_of_8000": achieved / 8000.0,
                     "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                     "probe_gbs": wl.kv_bytes_per_layer("bfp8") / probe_med / 1e9,
                     "frac_of_probe": probe_med / inter_med,
                     "hbm_read_gbs": wl.caches["bfp8"].layers[0].numel() / hbm_med / 1e9,
                     "frac_of_hbm_read": (wl.kv_bytes_per_layer("bfp8") / inter_med) / (wl.caches["bfp8"].layers[0].numel() / hbm_med),
                     "ceilings": {"what": "hma_decode_attention_planned, hma_decode_attention (sets itself up in every call), "
                                          "hma_kv_read_probe (same records, no arithmetic) and hma_hbm_read_probe "
                                          "(plain contiguous read of the layer) interleaved call by call, 5 passes over all layers; "
                                          "[mean, median, min] us per call",
                                  "attention_us": [inter_mean * 1e6, inter_med * 1e6, inter_min * 1e6],
                                  "attention_self_planned_us": [self_mean * 1e6, self_med * 1e6, self_min * 1e6],
                                  "kv_read_probe_us": [probe_mean * 1e6, probe_med * 1e6, probe_min * 1e6],
                                  "hbm_read_us": [hbm_mean * 1e6, hbm_med * 1e6, hbm_min * 1e6]},
                     "kernel": "hma_decode_attention_planned (attn_kernel<6,0,1>: attention and cross-split reduction in one launch, set-up "
                               "read from the step's plan; one hma_decode_attention_plan launch per step is inside the timed steps)",
                     "bytes_per_launch": wl.kv_bytes_per_layer("bfp8"), "us_per_launch_mean": call_mean * 1e6,
                     "us_per_launch_median": call_med * 1e6, "us_per_launch_min": call_min * 1e6},
        "decode_only": {"tokens_per_s": aggregate_value(wl.B, sec_decode_only, ws), "ms_per_step": sec_decode_only * 1e3,
                        "kv_gbs": kv_step / sec_decode_only / 1e9, "slowdown_from_ingest": alt_ingest / alt_plain - 1.0,
                        "how": "ms_per_step from its own run of the timed steps; the slowdown from steps with and without the ingest "
                               "timed in alternation (4 rounds of 4 steps each)"},
        "ingest_paced_at_link_rate": paced,
        "plan": {"what": "decode pass (no ingest) with one hma_decode_attention_plan per step + planned calls, against the same pass "
                         "with hma_decode_attention (every call repeats the set-up); timed in alternation, 4 rounds of 4 steps each",
                 "ms_per_step_planned": alt_planned * 1e3, "ms_per_step_self_planned": alt_self * 1e3, "speedup": alt_self / alt_planned},
    }
    line.update(extra)
    if rank == 0 and ws == 1 and not args.no_cpu:
        n_seq = wl.B
        t, threads, toks = time_oracle(args.workload, n_seq)
        line["cpu_baseline"] = {"value": n_seq / (t * wl.L), "unit": "tokens/s", "cores": threads, "kind": "oracle",
                                "kv_gbs": toks * wl.hkv * BFP8_ROW / t / 1e9, "seconds": t,
                                "sample": "layer 0 of all %d sequences (%d tokens x %d q heads); tokens/s = %d / (t x %d layers)"
                                % (n_seq, toks, wl.hq, n_seq, wl.L)}
    if rank == 0 and ws == 1 and not args.no_cpu:
        # the oracle's BFP8 -> BF16 decode beside the library's rebuild (elements per second)
        from oracle import oracle as orc
        wire = synth.make_kv_wire(wl.hkv, 8192, 99).numpy()
        orc.decode_rowmajor_bf16(wire[:, :64])
        t0 = time.perf_counter()
        orc.decode_rowmajor_bf16(wire)
        t_dec = time.perf_counter() - t0
        rb = extra["rebuild_request"]
        line["cpu_baseline"]["dequant"] = {"oracle_elements_per_s": wire.shape[0] * wire.shape[1] * 128 / t_dec, "oracle_threads": 1,
                                           "oracle_sample": "one tensor of one layer of one 8192-token request (%d elements)" % (wire.shape[0] * wire.shape[1] * 128),
                                           "gpu_elements_per_s": rb_elems / (rb["ms"] / 1e3), "gpu_call": "hma_bfp8_rebuild_request"}
    if rank == 0:
        print(json.dumps(line))
    if ws > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
