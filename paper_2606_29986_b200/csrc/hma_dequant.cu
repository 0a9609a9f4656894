// Stand-alone BFP8 -> BF16 reconstruction (section 3.3: block-float decode to BF16, bit-exact).
#include <cuda_fp16.h>

#include "hma_common.cuh"

namespace hma {

// Four elements of one block -> four BF16 bit patterns, bit-exact for every (E, byte) pair.
// The byte s<<7|m is first spread to the 16-bit pattern s<<15|m (the integer-only decode of section 3.3).
// Common exponents (every result a normal BF16 number, no overflow): 0x4300|m is the BF16 number 128 + m, and one
// packed BF16 fused multiply-add (128 + m) * 2^(E-133) - 2^(E-126) leaves m * 2^(E-133) exactly, two elements at a
// time; the sign bit is put back with one logic instruction, so m = 0 keeps its sign.
// Other exponents: the pattern is the FP16 subnormal +-m * 2^-24; widening to fp32 and multiplying by 2^(E-109) (one
// factor while it is a normal fp32 number, two exact power-of-two factors above that) gives m * 2^(E-133) exactly
// (fp32 subnormals and overflow to Inf included); its upper 16 bits are the BF16 value.
// exponents for which the packed BF16 path below is exact: every result a normal BF16 number, no overflow
__device__ __forceinline__ bool bf16_path_ok(uint32_t E) { return E - 20u <= 216u; }
// 2^(E-133) in both halves of a BF16 pair
__device__ __forceinline__ uint32_t bf16_scale2(uint32_t E) { return (E - 6u) * 0x00800080u; }
// two elements whose bytes were spread to the halfwords b<<8|b -> two BF16 values (bf16_path_ok exponents only)
__device__ __forceinline__ uint32_t dequant2_bf16(uint32_t h, uint32_t sc)
{
    uint32_t r;
    const uint32_t off = sc + 0x83808380u;                    // -2^(E-126) in both halves
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(r) : "r"((h & 0x007F007Fu) | 0x43004300u), "r"(sc), "r"(off));
    return r | (h & 0x80008000u);
}

__device__ __forceinline__ uint2 dequant4(uint32_t w, uint32_t E)
{
    uint32_t h01, h23;
    asm("prmt.b32 %0, %1, 0, 0x1100;" : "=r"(h01) : "r"(w));
    asm("prmt.b32 %0, %1, 0, 0x3322;" : "=r"(h23) : "r"(w));
    if (bf16_path_ok(E)) {
        const uint32_t sc = bf16_scale2(E);
        return make_uint2(dequant2_bf16(h01, sc), dequant2_bf16(h23, sc));
    }
    h01 &= 0x807F807Fu;
    h23 &= 0x807F807Fu;
    const float2 f01 = __half22float2(*reinterpret_cast<const __half2 *>(&h01));
    const float2 f23 = __half22float2(*reinterpret_cast<const __half2 *>(&h23));
    uint32_t b0, b1, b2, b3;
    if (E <= 236u) {
        // 2^(E-109) is a normal fp32 number: one exact multiplication (results below 2^-126 are exact subnormals)
        const float sc = __uint_as_float((E + 18u) << 23);
        b0 = __float_as_uint(f01.x * sc); b1 = __float_as_uint(f01.y * sc);
        b2 = __float_as_uint(f23.x * sc); b3 = __float_as_uint(f23.y * sc);
    } else {
        const float s1 = __uint_as_float(((E >> 1) + 73u) << 23);           // 2^(floor(E/2) - 54)
        const float s2 = __uint_as_float(((E - (E >> 1)) + 72u) << 23);     // 2^(ceil(E/2) - 55)
        b0 = __float_as_uint((f01.x * s1) * s2); b1 = __float_as_uint((f01.y * s1) * s2);
        b2 = __float_as_uint((f23.x * s1) * s2); b3 = __float_as_uint((f23.y * s1) * s2);
    }
    return make_uint2(__byte_perm(b0, b1, 0x7632), __byte_perm(b2, b3, 0x7632));
}

// Flat blocks: two threads per block, 8 elements each; 8-byte loads, 16-byte stores, both coalesced.
__global__ void __launch_bounds__(256) dequant_blocks_kernel(const uint8_t *__restrict__ exps,
                                                             const uint8_t *__restrict__ mants, int64_t n_blocks,
                                                             uint16_t *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // index of an 8-element half block
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < 2 * n_blocks; i += stride) {
        const uint32_t E = exps[i >> 1];
        const uint2 m = *reinterpret_cast<const uint2 *>(mants + i * 8);
        const uint2 lo = dequant4(m.x, E), hi = dequant4(m.y, E);
        *reinterpret_cast<uint4 *>(out + i * 8) = make_uint4(lo.x, lo.y, hi.x, hi.y);
    }
}

// One CTA per (logical page of the request, kv head): the K or V half record is staged in shared memory, then each
// thread rebuilds 8 consecutive channels of one token at a time and stores 16 bytes.  (One CTA per page covering all
// heads was measured slower: too few threads in flight for a copy-like kernel.)
// With `layers` set, blockIdx.z = 2 * layer + which selects the layer and the tensor, and the output is
// [num_layers][2][n_tokens][Hkv][128]: the whole request in one launch.
__global__ void __launch_bounds__(128) dequant_paged_kernel(CacheView cv, int which, const int32_t *__restrict__ page_ids,
                                                            int64_t token_begin, int64_t n_tokens,
                                                            uint16_t *__restrict__ out, void *const *__restrict__ layers)
{
    if (layers) {
        cv.layer = (uint8_t *)layers[blockIdx.z >> 1];
        which = blockIdx.z & 1;
        out += (int64_t)blockIdx.z * n_tokens * cv.num_kv_heads * kHeadDim;
    }
    __shared__ __align__(16) uint8_t recs[1][kBf16Half];
    const int64_t first_page = token_begin / kPageTokens;
    const int64_t lp = first_page + blockIdx.x;
    const int32_t pid = page_ids[blockIdx.x];
    const bool bad = pid < 0 || pid >= cv.num_pages;
    const int half = cv.format == HMA_KV_BFP8 ? kBfp8Half : kBf16Half;
    const bool relayout = which == 0 && cv.key_layout == HMA_KEYS_INTERLEAVED;
    if (bad && threadIdx.x == 0) atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_DEQUANT);
    {
        const int h0 = blockIdx.y;
        constexpr int nh = 1;
        if (!bad) {
            const int per = half / 16;                                  // 16-byte pieces per head
            for (int i = threadIdx.x; i < nh * per; i += blockDim.x) {
                const int hh = i / per, o = (i - hh * per) * 16;
                const uint8_t *src = cv.layer + ((int64_t)pid * cv.num_kv_heads + h0 + hh) * (int64_t)(2 * half) + (int64_t)which * half;
                *reinterpret_cast<uint4 *>(&recs[hh][o]) = *reinterpret_cast<const uint4 *>(src + o);
            }
        }
        __syncthreads();
        for (int item = threadIdx.x; item < kPageTokens * 16; item += blockDim.x) {
            const int tok = item >> 4, c0 = (item & 15) * 8;             // channels c0 .. c0+7 of token tok: half a block
            const int64_t gt = lp * kPageTokens + tok;
            if (gt < token_begin || gt >= token_begin + n_tokens) continue;
            const uint8_t *rec = recs[0];
            uint2 lo = make_uint2(0u, 0u), hi = lo;                     // channels c0..c0+3 and c0+4..c0+7 as BF16 pairs
            if (!bad) {
                // `rec` holds one half record: offsets below are relative to the start of that half
                if (cv.format == HMA_KV_BFP8) {
                    uint32_t w0, w1, E;
                    if (which == 0) {
                        E = rec[bfp8_k_exp_off(tok, c0 >> 4)];
                        const uint8_t *p = rec + bfp8_k_el_off(tok, c0);           // four channels are one word, the next four 16 bytes on
                        w0 = *reinterpret_cast<const uint32_t *>(p);
                        w1 = *reinterpret_cast<const uint32_t *>(p + 16);
                    } else {
                        // consecutive channels of a token sit 64 bytes apart, at the token's byte position
                        const uint8_t *p = rec + (bfp8_v_el_off(tok, c0) - kBfp8Half);
                        E = rec[bfp8_v_exp_off(tok, c0 >> 4) - kBfp8Half];
                        w0 = p[0] | (p[64] << 8) | (p[128] << 16) | ((uint32_t)p[192] << 24);
                        w1 = p[256] | (p[320] << 8) | (p[384] << 16) | ((uint32_t)p[448] << 24);
                    }
                    lo = dequant4(w0, E);
                    hi = dequant4(w1, E);
                } else if (which == 0) {
                    const uint8_t *p = rec + bf16_k_el_off(tok, c0);               // four channels are 8 bytes, the next four 16 bytes on
                    lo = *reinterpret_cast<const uint2 *>(p);
                    hi = *reinterpret_cast<const uint2 *>(p + 16);
                } else {
                    uint32_t e[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) e[k] = *reinterpret_cast<const uint16_t *>(rec + bf16_v_el_off(tok, c0 + k) - kBf16Half);
                    lo = make_uint2(e[0] | (e[1] << 16), e[2] | (e[3] << 16));
                    hi = make_uint2(e[4] | (e[5] << 16), e[6] | (e[7] << 16));
                }
            }
            uint16_t *row = out + ((gt - token_begin) * cv.num_kv_heads + blockIdx.y) * kHeadDim;
            if (relayout) {
                // keys cached with rotary pairs interleaved leave in half-split order (section 3.3, key re-layout):
                // cached channels c0, c0+2, .. go to c0/2 .., cached channels c0+1, c0+3, .. to 64 + c0/2 ..
                *reinterpret_cast<uint2 *>(row + (c0 >> 1)) =
                    make_uint2((lo.x & 0xFFFFu) | (lo.y << 16), (hi.x & 0xFFFFu) | (hi.y << 16));
                *reinterpret_cast<uint2 *>(row + 64 + (c0 >> 1)) =
                    make_uint2((lo.x >> 16) | (lo.y & 0xFFFF0000u), (hi.x >> 16) | (hi.y & 0xFFFF0000u));
            } else {
                *reinterpret_cast<uint4 *>(row + c0) = make_uint4(lo.x, lo.y, hi.x, hi.y);
            }
        }
    }
}

// ---------------------------------------------------------------- the streaming rebuild of BFP8 pages
// One CTA per SM, sixteen warps, and every warp is a worker of its own: it walks (layer, page, kv head) records with a
// private three-deep ring of 4352-byte slots that it feeds itself (one bulk async copy per record, one mbarrier per
// slot), so no CTA-wide barrier sits between a record's arrival and its stores.  K: a lane takes 8 channels of a token
// (two words of the record, one exponent) and stores 16 bytes, a warp's store covering two whole 256-byte rows.
// V: a word of the record holds four tokens of one channel, so a lane takes four channels, transposes the bytes in
// registers and writes an 8-byte piece for each of the four tokens.  Bit-exact like the kernels above (same dequant4).
constexpr int kRebuildWarps = 16;
constexpr int kRebuildDepth = 3;
constexpr int kRebuildThreads = kRebuildWarps * 32;
constexpr uint32_t kRebuildSpin = 1u << 22;
constexpr int kRebuildSmem = kRebuildWarps * kRebuildDepth * (kBfp8Record + 8);

struct RebuildArgs {
    void *const *layers;          // device array of layer pointers (NULL: cv.layer is the only layer)
    const int32_t *page_ids;
    int64_t token_begin, n_tokens;
    uint16_t *out_k, *out_v;      // rows [n_tokens][Hkv][128] of layer 0 (NULL: tensor not wanted)
    int64_t layer_stride;         // elements between consecutive layers of one tensor
    int32_t n_layers, n_pages;
};

__device__ __forceinline__ uint32_t rb_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool rb_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 1000;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

// One record -> its K and V rows.  kPlain: a good page, all sixteen tokens wanted, every exponent takes the packed
// BF16 path (the caller checked); otherwise bad pages give zeros, tokens outside [t_lo, t_hi) are skipped and every
// block picks its decode by its exponent.
template <bool kPlain>
__device__ __forceinline__ void rebuild_record(const RebuildArgs &a, const uint8_t *rec, bool relayout, int64_t base_el,
                                               int64_t row_elems, int lane, bool ok, int t_lo, int t_hi)
{
    if (a.out_k) {
        uint16_t *out0 = a.out_k + base_el;
        const int c0 = (lane & 15) * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            // lane = 8-channel group + 16 * (token & 1): a warp's store covers two whole rows
            const int tok = 2 * i + (lane >> 4);
            uint2 lo = make_uint2(0u, 0u), hi = lo;
            if (kPlain || ok) {
                const uint32_t E = rec[bfp8_k_exp_off(tok, c0 >> 4)];
                const uint8_t *p = rec + bfp8_k_el_off(tok, c0);
                const uint32_t w0 = *reinterpret_cast<const uint32_t *>(p), w1 = *reinterpret_cast<const uint32_t *>(p + 16);
                if (kPlain) {
                    const uint32_t sc = bf16_scale2(E);
                    lo = make_uint2(dequant2_bf16(__byte_perm(w0, 0u, 0x1100u), sc), dequant2_bf16(__byte_perm(w0, 0u, 0x3322u), sc));
                    hi = make_uint2(dequant2_bf16(__byte_perm(w1, 0u, 0x1100u), sc), dequant2_bf16(__byte_perm(w1, 0u, 0x3322u), sc));
                } else {
                    lo = dequant4(w0, E);
                    hi = dequant4(w1, E);
                }
            }
            if (!kPlain && (tok < t_lo || tok >= t_hi)) continue;
            uint16_t *row = out0 + tok * row_elems;
            if (relayout) {
                // keys cached with rotary pairs interleaved leave in half-split order (section 3.3, key re-layout)
                __stcs(reinterpret_cast<uint2 *>(row + (c0 >> 1)), make_uint2((lo.x & 0xFFFFu) | (lo.y << 16), (hi.x & 0xFFFFu) | (hi.y << 16)));
                __stcs(reinterpret_cast<uint2 *>(row + 64 + (c0 >> 1)), make_uint2((lo.x >> 16) | (lo.y & 0xFFFF0000u), (hi.x >> 16) | (hi.y & 0xFFFF0000u)));
            } else {
                __stcs(reinterpret_cast<uint4 *>(row + c0), make_uint4(lo.x, lo.y, hi.x, hi.y));      // streaming: written once, read by somebody else
            }
        }
    }
    if (a.out_v) {
        // V: a lane takes channels ch0 .. ch0+3 of tokens 2tq, 2tq+1, 2tq+8, 2tq+9 (the four bytes of its words).
        // Lanes differ in tq and in which quad of a 32-channel span they hold (two-way bank conflicts at most; every
        // store instruction covers whole 64-byte pieces of four output rows); the loop walks the four spans.
        uint16_t *out0 = a.out_v + base_el;
        const int tq = lane & 3;
        const uint8_t *vb = rec + kBfp8Half;
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const int j = 2 * jj + ((lane >> 2) & 1), cb0 = 8 * ((lane >> 3) & 1) + 4 * (lane >> 4), ch0 = 16 * j + cb0;
            uint32_t w[4] = {0u, 0u, 0u, 0u}, e4 = 0u;
            if (kPlain || ok) {
                const uint8_t *p = vb + 128 + (j >> 1) * 512 + ((cb0 & 7) * 4 + tq) * 16 + ((j & 1) * 2 + (cb0 >> 3)) * 4;
#pragma unroll
                for (int i = 0; i < 4; ++i) w[i] = *reinterpret_cast<const uint32_t *>(p + 64 * i);       // channel ch0 + i, four tokens
                e4 = *reinterpret_cast<const uint32_t *>(vb + tq * 32 + j * 4);                           // exponents of the four tokens, block j
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // byte k of the four words = channels ch0 .. ch0+3 of token 2tq + (k & 1) + 8 (k >> 1); one byte
                // permutation per channel pair picks the two bytes and spreads each over a halfword
                const int tok = 2 * tq + (k & 1) + 8 * (k >> 1);
                const uint32_t sel = (uint32_t)(k | (k << 4) | ((4 + k) << 8) | ((4 + k) << 12));
                const uint32_t h01 = __byte_perm(w[0], w[1], sel), h23 = __byte_perm(w[2], w[3], sel);
                const uint32_t E = (e4 >> (8 * k)) & 0xFFu;
                uint2 r = make_uint2(0u, 0u);
                if (kPlain) {
                    const uint32_t sc = bf16_scale2(E);
                    r = make_uint2(dequant2_bf16(h01, sc), dequant2_bf16(h23, sc));
                } else if (ok) {
                    r = dequant4(__byte_perm(h01, h23, 0x6420u), E);
                }
                if (!kPlain && (tok < t_lo || tok >= t_hi)) continue;
                __stcs(reinterpret_cast<uint2 *>(out0 + tok * row_elems + ch0), r);
            }
        }
    }
}

__global__ void __launch_bounds__(kRebuildThreads, 1) rebuild_stream_kernel(CacheView cv, RebuildArgs a)
{
    extern __shared__ __align__(128) uint8_t rb_smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    uint8_t *ring = rb_smem + (size_t)warp * kRebuildDepth * kBfp8Record;
    uint64_t *bars = reinterpret_cast<uint64_t *>(rb_smem + (size_t)kRebuildWarps * kRebuildDepth * kBfp8Record) + warp * kRebuildDepth;
    const uint32_t Hkv = (uint32_t)cv.num_kv_heads, n_pages = (uint32_t)a.n_pages;
    const uint32_t n_items = (uint32_t)a.n_layers * n_pages * Hkv;       // item = (layer, page, head), head fastest (the launcher keeps it below 2^31)
    const uint32_t n_workers = gridDim.x * kRebuildWarps;
    const uint32_t first = blockIdx.x * kRebuildWarps + warp;            // neighbouring warps take neighbouring heads: together they complete output rows
    if (lane == 0) {
        for (int s = 0; s < kRebuildDepth; ++s) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(rb_smem_u32(bars + s)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    // the whole record, or only the half that is wanted
    const int off = a.out_k ? 0 : kBfp8Half, bytes = (a.out_k && a.out_v) ? kBfp8Record : kBfp8Half;
    auto split = [&](uint32_t item, uint32_t &l, uint32_t &pg, uint32_t &h) {
        const uint32_t lp = item / Hkv;
        h = item - lp * Hkv;
        l = lp / n_pages;
        pg = lp - l * n_pages;
    };
    auto load = [&](uint32_t item, int slot) {      // lane 0 only
        uint32_t l, pg, h;
        split(item, l, pg, h);
        const int32_t pid = a.page_ids[pg];
        const uint32_t bar = rb_smem_u32(bars + slot);
        if (pid < 0 || pid >= cv.num_pages) {       // nothing to fetch: the consumer sees the same page id and writes zeros
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
            return;
        }
        const uint8_t *base = a.layers ? (const uint8_t *)a.layers[l] : cv.layer;
        const uint8_t *src = base + ((int64_t)pid * Hkv + h) * (int64_t)kBfp8Record + off;
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                         rb_smem_u32(ring + slot * kBfp8Record) + off),
                     "l"(src), "r"(bytes), "r"(bar)
                     : "memory");
    };
    if (lane == 0)
        for (int s = 0; s < kRebuildDepth; ++s) {
            const uint64_t item = first + (uint64_t)s * n_workers;
            if (item < n_items) load((uint32_t)item, s);
        }
    const bool relayout = cv.key_layout == HMA_KEYS_INTERLEAVED;
    const int64_t first_page = a.token_begin / kPageTokens;
    const int64_t row_elems = (int64_t)Hkv * kHeadDim;
    int slot = 0;
    uint32_t parity = 0;
    bool gave_up = false;
    for (uint64_t it64 = first; it64 < n_items; it64 += n_workers) {
        const uint32_t item = (uint32_t)it64;
        {
            const uint32_t bar = rb_smem_u32(bars + slot);
            uint32_t spins = 0;
            bool here = rb_try_wait(bar, parity);
            while (!here && ++spins < kRebuildSpin) here = rb_try_wait(bar, parity);
            gave_up = __any_sync(0xFFFFFFFFu, !here);
        }
        if (gave_up) break;
        uint32_t l, pg, h;
        split(item, l, pg, h);
        const int32_t pid = a.page_ids[pg];
        const bool ok = pid >= 0 && pid < cv.num_pages;
        if (!ok && lane == 0) atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_DEQUANT);
        const uint8_t *rec = ring + slot * kBfp8Record;
        // tokens [t_lo, t_hi) of this page belong to the request; rel = request row of the page's first slot
        const int64_t rel = (first_page + pg) * kPageTokens - a.token_begin;
        const int t_lo = rel < 0 ? (int)-rel : 0;
        const int t_hi = (a.n_tokens - rel) < kPageTokens ? (int)(a.n_tokens - rel) : kPageTokens;
        const int64_t base_el = (int64_t)l * a.layer_stride + rel * row_elems + (int64_t)h * kHeadDim;
        // The common case (a good page, all sixteen tokens wanted, every exponent in the range of the packed BF16
        // path) runs without a single test per element; anything else takes the general path.
        bool plain = ok && t_lo == 0 && t_hi == kPageTokens;
        if (plain) {
            bool in_range = true;
            if (a.out_k) {
                const uint32_t e = *reinterpret_cast<const uint32_t *>(rec + 4 * lane);
#pragma unroll
                for (int i = 0; i < 4; ++i) in_range &= bf16_path_ok((e >> (8 * i)) & 0xFFu);
            }
            if (a.out_v) {
                const uint32_t e = *reinterpret_cast<const uint32_t *>(rec + kBfp8Half + 4 * lane);
#pragma unroll
                for (int i = 0; i < 4; ++i) in_range &= bf16_path_ok((e >> (8 * i)) & 0xFFu);
            }
            plain = __all_sync(0xFFFFFFFFu, in_range);
        }
        if (plain) rebuild_record<true>(a, rec, relayout, base_el, row_elems, lane, true, 0, kPageTokens);
        else rebuild_record<false>(a, rec, relayout, base_el, row_elems, lane, ok, t_lo, t_hi);
        __syncwarp();                                  // every lane is done with the slot
        if (lane == 0) {
            const uint64_t next = it64 + (uint64_t)kRebuildDepth * n_workers;
            if (next < n_items) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                load((uint32_t)next, slot);
            }
        }
        if (++slot == kRebuildDepth) { slot = 0; parity ^= 1u; }
    }
    if (gave_up && lane == 0) {
        atomicOr(cv.flags, HMA_FLAG_WAIT_TIMEOUT);
        // copies still in flight target this CTA's shared memory: give them a bounded time to land before leaving
        for (int s = 0; s < kRebuildDepth; ++s)
            for (uint32_t spins = 0; spins < (1u << 16) && !rb_try_wait(rb_smem_u32(bars + s), 0) && !rb_try_wait(rb_smem_u32(bars + s), 1); ++spins) {}
    }
}

// The elementwise strawman of section 3.3: one thread per output element, byte
// loads straight from the cache, integer bit assembly, two-byte stores.  Kept only as the comparison point.
__global__ void __launch_bounds__(256) dequant_naive_kernel(CacheView cv, int which, const int32_t *__restrict__ page_ids,
                                                            int64_t token_begin, int64_t n_tokens, uint16_t *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_tokens * cv.num_kv_heads * kHeadDim) return;
    const int ch = (int)(i % kHeadDim), h = (int)((i / kHeadDim) % cv.num_kv_heads);
    const int64_t gt = token_begin + i / ((int64_t)kHeadDim * cv.num_kv_heads);
    const int tok = (int)(gt % kPageTokens);
    const int32_t pid = page_ids[gt / kPageTokens - token_begin / kPageTokens];
    uint32_t bits = 0;
    if (pid >= 0 && pid < cv.num_pages) {
        const uint8_t *rec = cv.layer + ((int64_t)pid * cv.num_kv_heads + h) * (int64_t)record_bytes(cv.format);
        if (cv.format == HMA_KV_BFP8)
            bits = which == 0 ? bfp8_to_bf16_bits(rec[bfp8_k_exp_off(tok, ch >> 4)], rec[bfp8_k_el_off(tok, ch)])
                              : bfp8_to_bf16_bits(rec[bfp8_v_exp_off(tok, ch >> 4)], rec[bfp8_v_el_off(tok, ch)]);
        else
            bits = *reinterpret_cast<const uint16_t *>(rec + (which == 0 ? bf16_k_el_off(tok, ch) : bf16_v_el_off(tok, ch)));
    } else {
        atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_DEQUANT);
    }
    const int oc = which == 0 ? key_channel_of_query(ch, cv.key_layout) : ch;
    out[(i / kHeadDim) * kHeadDim + oc] = (uint16_t)bits;
}

}  // namespace hma

static hma_status_t launch_rebuild(const hma::CacheView &cv, const hma::RebuildArgs &a, void *stream)
{
    int dev = 0, n_sm = 0;
    HMA_CUDA_OK(cudaGetDevice(&dev));
    HMA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    const int64_t items = (int64_t)a.n_layers * a.n_pages * cv.num_kv_heads;
    if (items > 0x7FFFFFFF) return HMA_ERR_INVALID_ARG;
    HMA_CUDA_OK(cudaFuncSetAttribute(hma::rebuild_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, hma::kRebuildSmem));
    // one CTA per SM at most, every warp walking its share of the records
    const int64_t want = (items + hma::kRebuildWarps - 1) / hma::kRebuildWarps;
    hma::rebuild_stream_kernel<<<(unsigned)(want < n_sm ? want : n_sm), hma::kRebuildThreads, hma::kRebuildSmem, (cudaStream_t)stream>>>(cv, a);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_bfp8_dequant_blocks_bf16(const uint8_t *exps, const uint8_t *mants, int64_t n_blocks,
                                                     void *out_bf16, void *stream)
{
    if (n_blocks < 0 || (n_blocks > 0 && (!exps || !mants || !out_bf16))) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)mants & 15u) || ((uintptr_t)out_bf16 & 15u)) return HMA_ERR_ALIGNMENT;
    if (n_blocks == 0) return HMA_OK;
    int64_t work = 2 * n_blocks;
    int64_t blocks = (work + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    hma::dequant_blocks_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(exps, mants, n_blocks, (uint16_t *)out_bf16);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_bfp8_dequant_bf16(const hma_cache_t *cache, int32_t layer, int32_t which,
                                              const int32_t *page_ids, int64_t token_begin, int64_t n_tokens,
                                              void *out_bf16, void *stream)
{
    if (!cache || layer < 0 || layer >= cache->desc.num_layers || (which != 0 && which != 1) || token_begin < 0 || n_tokens < 0)
        return HMA_ERR_INVALID_ARG;
    if (!hma::on_cache_device(cache)) return HMA_ERR_INVALID_ARG;
    if (n_tokens == 0) return HMA_OK;
    if (!page_ids || !out_bf16) return HMA_ERR_INVALID_ARG;
    if ((uintptr_t)out_bf16 & 15u) return HMA_ERR_ALIGNMENT;
    const int64_t first = token_begin / hma::kPageTokens;
    const int64_t last = (token_begin + n_tokens - 1) / hma::kPageTokens;
    const int64_t n_pages = last - first + 1;
    if (n_pages > 0x7FFFFFFF) return HMA_ERR_INVALID_ARG;
    hma::CacheView cv{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    if (cache->desc.format == HMA_KV_BFP8) {
        hma::RebuildArgs a{nullptr, page_ids, token_begin, n_tokens, which == 0 ? (uint16_t *)out_bf16 : nullptr,
                           which == 1 ? (uint16_t *)out_bf16 : nullptr, 0, 1, (int32_t)n_pages};
        return launch_rebuild(cv, a, stream);
    }
    dim3 grid((unsigned)n_pages, (unsigned)cache->desc.num_kv_heads);
    hma::dequant_paged_kernel<<<grid, 128, 0, (cudaStream_t)stream>>>(cv, which, page_ids, token_begin, n_tokens,
                                                                      (uint16_t *)out_bf16, nullptr);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_bfp8_rebuild_request(const hma_cache_t *cache, const int32_t *page_ids, int64_t token_begin,
                                                 int64_t n_tokens, void *out_bf16, void *stream)
{
    if (!cache || token_begin < 0 || n_tokens < 0) return HMA_ERR_INVALID_ARG;
    if (!hma::on_cache_device(cache)) return HMA_ERR_INVALID_ARG;
    if (n_tokens == 0) return HMA_OK;
    if (!page_ids || !out_bf16) return HMA_ERR_INVALID_ARG;
    if ((uintptr_t)out_bf16 & 15u) return HMA_ERR_ALIGNMENT;
    const int64_t first = token_begin / hma::kPageTokens;
    const int64_t last = (token_begin + n_tokens - 1) / hma::kPageTokens;
    const int64_t n_pages = last - first + 1;
    if (n_pages > 0x7FFFFFFF || cache->desc.num_layers > 32767) return HMA_ERR_INVALID_ARG;
    hma::CacheView cv{(uint8_t *)cache->layers[0], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    if (cache->desc.format == HMA_KV_BFP8) {
        const int64_t tensor = n_tokens * cache->desc.num_kv_heads * hma::kHeadDim;      // elements of one tensor of one layer
        hma::RebuildArgs a{cache->d_layers, page_ids, token_begin, n_tokens, (uint16_t *)out_bf16, (uint16_t *)out_bf16 + tensor,
                           2 * tensor, cache->desc.num_layers, (int32_t)n_pages};
        return launch_rebuild(cv, a, stream);
    }
    dim3 grid((unsigned)n_pages, (unsigned)cache->desc.num_kv_heads, (unsigned)(2 * cache->desc.num_layers));
    hma::dequant_paged_kernel<<<grid, 128, 0, (cudaStream_t)stream>>>(cv, 0, page_ids, token_begin, n_tokens,
                                                                      (uint16_t *)out_bf16, cache->d_layers);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_bfp8_dequant_bf16_naive(const hma_cache_t *cache, int32_t layer, int32_t which,
                                                    const int32_t *page_ids, int64_t token_begin, int64_t n_tokens,
                                                    void *out_bf16, void *stream)
{
    if (!cache || layer < 0 || layer >= cache->desc.num_layers || (which != 0 && which != 1) || token_begin < 0 || n_tokens < 0)
        return HMA_ERR_INVALID_ARG;
    if (!hma::on_cache_device(cache)) return HMA_ERR_INVALID_ARG;
    if (n_tokens == 0) return HMA_OK;
    if (!page_ids || !out_bf16) return HMA_ERR_INVALID_ARG;
    const int64_t total = n_tokens * cache->desc.num_kv_heads * hma::kHeadDim;
    if ((total + 255) / 256 > 0x7FFFFFFF) return HMA_ERR_INVALID_ARG;
    hma::CacheView cv{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    hma::dequant_naive_kernel<<<(unsigned)((total + 255) / 256), 256, 0, (cudaStream_t)stream>>>(cv, which, page_ids, token_begin,
                                                                                                 n_tokens, (uint16_t *)out_bf16);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}
