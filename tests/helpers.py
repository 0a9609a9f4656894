"""Shared scaffolding of the GPU parity tests: build a paged cache from seeded wire bytes through the C ABI."""
import numpy as np
import torch

from paper_2606_29986_b200 import hma, synth


def bf16_bits(t):
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def bf16_bits_to_f64(bits):
    return (np.asarray(bits, np.uint32) << 16).view(np.float32).astype(np.float64)


class Scenario:
    """A batch of sequences with seeded BFP8 wire bytes, ingested into a paged cache on the GPU."""

    def __init__(self, lens, hq, hkv, seed=0, permute=False, fmt=hma.HMA_KV_BFP8, wire_layout=hma.HMA_WIRE_ROWMAJOR,
                 shards=1, layers=1, extra_pages=3, fill=0xA5, device="cuda", one_launch=False, key_layout=0):
        self.lens = np.asarray(lens, np.int32)
        self.B, self.hq, self.hkv, self.layers = len(lens), hq, hkv, layers
        self.seed = seed
        self.table_np, self.num_pages, self.spare = synth.block_table(self.lens, permute, seed, extra_pages)
        self.key_layout = key_layout
        self.desc = hma.make_desc(layers, hq, hkv, self.num_pages, fmt, key_layout=key_layout)
        self.cache = hma.KVCache(self.desc, device, fill=fill)
        self.table = torch.from_numpy(self.table_np).to(device)
        self.ctx = torch.from_numpy(self.lens).to(device)
        self.q = synth.make_q(self.B, hq, seed).to(device)
        self.k_wires = [[None] * self.B for _ in range(layers)]
        self.v_wires = [[None] * self.B for _ in range(layers)]
        for l in range(layers):
            for b, T in enumerate(self.lens):
                T = int(T)
                kw = synth.make_kv_wire(hkv, T, synth.sequence_seed(seed, l, b, 0), channel_seed=synth.channel_seed(seed, l, 0))
                vw = synth.make_kv_wire(hkv, T, synth.sequence_seed(seed, l, b, 1), channel_seed=synth.channel_seed(seed, l, 1))
                self.k_wires[l][b], self.v_wires[l][b] = kw.numpy(), vw.numpy()
                if T == 0:
                    continue
                pages = self.table[b, :(T + 15) // 16].contiguous()
                hs = hkv // shards
                kss, vss = [], []
                for s in range(shards):
                    ks, vs = kw[s * hs:(s + 1) * hs].contiguous(), vw[s * hs:(s + 1) * hs].contiguous()
                    if wire_layout == hma.HMA_WIRE_TILE32:
                        ks, vs = synth.rowmajor_to_tile32(ks), synth.rowmajor_to_tile32(vs)
                    kss.append(ks.to(device))
                    vss.append(vs.to(device))
                    if not one_launch:
                        hma.hma_kv_ingest_layer(self.cache, l, kss[-1], vss[-1], wire_layout, s * hs, hs, pages, 0, T)
                if one_launch:      # every shard of the layer in a single call
                    hma.hma_kv_ingest_layer_shards(self.cache, l, kss, vss, wire_layout, [s * hs for s in range(shards)],
                                                   [hs] * shards, pages, 0, T)
        torch.cuda.synchronize()
        self.workspace = hma.new_workspace(self.desc, self.B, device)

    def attention(self, layer=0, out_dtype=torch.bfloat16, simple=False, sm_scale=None, q=None):
        q = self.q if q is None else q
        sm_scale = 1.0 / np.sqrt(128.0) if sm_scale is None else sm_scale
        out = torch.full((self.B, self.hq, 128), float("nan"), dtype=out_dtype, device=q.device)
        if simple:
            hma.hma_decode_attention_simple(self.cache, layer, q, out, self.table, self.ctx, sm_scale)
        else:
            hma.hma_decode_attention(self.cache, layer, q, out, self.table, self.ctx, sm_scale, self.workspace)
        torch.cuda.synchronize()
        return out

    def oracle(self, layer=0, sm_scale=None, q=None):
        from oracle import oracle as orc
        q = self.q if q is None else q
        return orc.decode_attention(bf16_bits(q), self.k_wires[layer], self.v_wires[layer], self.hkv, sm_scale,
                                    keys_interleaved=bool(self.key_layout))


def parity_metrics(got, ref64):
    """max-abs and relative-L2 error of a float array against the fp64 oracle."""
    got = np.asarray(got, np.float64)
    err = got - ref64
    return float(np.abs(err).max()), float(np.sqrt((err ** 2).sum() / max((ref64 ** 2).sum(), 1e-300)))


def check_attention(out_f32, out_bf16, ref64):
    """The parity bar.  F32 output: max-abs <= 1e-2 and rel-L2 <= 2e-3 against the fp64 oracle, literally.
    BF16 output: bit-for-bit the round-to-nearest-even of that F32 output (so the only extra error is the output
    format's own rounding), |err| <= 1e-2 + 2^-8 |ref| everywhere, max-abs <= 1e-2 literally on the elements small
    enough for BF16 to resolve that (|ref| < 2), and rel-L2 <= 2e-3 literally wherever the oracle's own result
    rounded to BF16 meets that bar, else within 5 % of that rounding floor (BF16 keeps 8 significant bits: on long
    contexts with outlier channels the floor alone is 1.3e-3 .. 2.4e-3)."""
    ma, rl = parity_metrics(out_f32, ref64)
    assert ma <= 1e-2 and rl <= 2e-3, ("f32 output", ma, rl)
    want16 = torch.from_numpy(np.ascontiguousarray(out_f32, np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(np.asarray(out_bf16, np.uint16), want16), "bf16 output is not the RNE of the f32 output"
    got = bf16_bits_to_f64(out_bf16)
    err = np.abs(got - ref64)
    mb, rb = parity_metrics(got, ref64)
    assert (err <= 1e-2 + 2.0 ** -8 * np.abs(ref64)).all(), ("bf16 output bound", (err - 2.0 ** -8 * np.abs(ref64)).max())
    small = np.abs(ref64) < 2.0
    assert not small.any() or err[small].max() <= 1e-2, ("bf16 max-abs where BF16 resolves it", err[small].max())
    floor16 = torch.from_numpy(np.ascontiguousarray(ref64)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    _, floor = parity_metrics(bf16_bits_to_f64(floor16), ref64)
    assert rb <= (2e-3 if floor <= 1.9e-3 else 1.05 * floor), ("bf16 rel-L2", rb, "rounding floor", floor)
    return ma, rl, mb, rb


def parity_sample(wl):
    """Outputs of the sequences a bench.Workload kept wire bytes of, against the oracle on those bytes, in the
    full-size launch configuration that bench.py times (one plan, then planned calls); the call that plans for itself
    must give the same bits.  The bar (max-abs 1e-2, rel-L2 2e-3) is taken on the F32 output; the BF16 output
    must be exactly its rounding; the BF16 numbers and the oracle's own BF16 rounding floor are returned beside it."""
    from oracle import oracle as orc
    res = []
    out32 = torch.empty((wl.B, wl.hq, 128), dtype=torch.float32, device=wl.device)
    self32 = torch.empty_like(out32)
    c = wl.caches["bfp8"]
    plan = hma.hma_decode_attention_plan(c, wl.table, wl.ctx, plan=wl.plan_for("bfp8"))     # as at the start of a bench step
    for (l, b), (kw, vw) in sorted(wl.sample_wires.items()):
        hma.hma_decode_attention_planned(c, l, wl.q[l], out32, wl.table, wl.ctx, wl.sm_scale, plan, wl.workspace)
        hma.hma_decode_attention_planned(c, l, wl.q[l], wl.out[l], wl.table, wl.ctx, wl.sm_scale, plan, wl.workspace)
        hma.hma_decode_attention(c, l, wl.q[l], self32, wl.table, wl.ctx, wl.sm_scale, wl.workspace)
        torch.cuda.synchronize(wl.device)
        qb = bf16_bits(wl.q[l][b:b + 1])
        ref64, ref16 = orc.decode_attention(qb, [kw], [vw], wl.hkv, wl.sm_scale)
        ref = ref64[0]
        rel = lambda x: float(np.sqrt(((x - ref) ** 2).sum() / (ref ** 2).sum()))
        g32 = out32[b].cpu().numpy().astype(np.float64)
        g16 = wl.out[l][b].float().cpu().numpy().astype(np.float64)
        res.append({"layer": l, "seq": b, "context": int(wl.lens[b]),
                    "f32_max_abs": float(np.abs(g32 - ref).max()), "f32_rel_l2": rel(g32),
                    "bf16_max_abs": float(np.abs(g16 - ref).max()), "bf16_rel_l2": rel(g16),
                    "bf16_is_rne_of_f32": bool(torch.equal(out32[b].to(torch.bfloat16), wl.out[l][b])),
                    "planned_equals_self_planned": bool(torch.equal(out32.view(torch.int32), self32.view(torch.int32))),
                    "bf16_floor_rel_l2": rel(bf16_bits_to_f64(ref16[0]))})
    return res
