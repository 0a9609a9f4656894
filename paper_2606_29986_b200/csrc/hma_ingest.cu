// Per-layer ingest: wire bytes (row-major or 32x32 tiles, one producer shard) -> page records
// (sections 3.2 / 3.3: host-to-device copy done by the caller or by mapped reads here, then the
// tiled -> paged re-layout that merges per-chip shards).  Byte values are never changed on a BFP8
// cache; on a BF16 cache each element is decoded while it is scattered.
#include <mutex>

#include "hma_common.cuh"

namespace hma {

constexpr int kMaxShards = 8;
struct IngestArgs {
    const uint8_t *k_wire[kMaxShards], *v_wire[kMaxShards];   // per producer shard
    int32_t head_begin[kMaxShards], head_count[kMaxShards];
    int32_t n_shards;
    const int32_t *page_ids;
    int64_t token_begin, n_tokens;      // range of the request's tokens that this launch writes
    int64_t wire_begin, wire_tokens;    // request token that is wire token 0, and the number of tokens the wire was laid out for
    int32_t layout;
};

// Address of the 16 element bytes of block j of wire token wt of shard head hs, and of its exponent byte.
__device__ __forceinline__ int64_t wire_block_off(int layout, int64_t n_tokens, int hs, int64_t wt, int j, int64_t *exp_off)
{
    if (layout == HMA_WIRE_ROWMAJOR) {
        int64_t row = ((int64_t)hs * n_tokens + wt) * kRowBytes;
        *exp_off = row + j;
        return row + kBlocksPerRow + j * kBlock;
    }
    const int64_t tile_rows = (n_tokens + 31) / 32;
    const int r = (int)(wt & 31);
    const int face = (r >> 4) * 2 + (j & 1);
    const int64_t tile = (((int64_t)hs * tile_rows + (wt >> 5)) * 4 + (j >> 1)) * kTileBytes;
    *exp_off = tile + face * 16 + (r & 15);
    return tile + 64 + face * 256 + (r & 15) * 16;
}

// One CTA per (page of the request, shard head).  Phase 1 stages the page's wire rows in shared
// memory in row-major form (16-byte or 8-byte coalesced reads).  Phase 2 walks the destination
// record word by word, gathers its bytes from the staged rows, and writes whole words; a word that
// mixes tokens inside and outside the range is merged with the bytes already in the cache.
__global__ void __launch_bounds__(128) ingest_kernel(CacheView cv, IngestArgs a)
{
    __shared__ __align__(16) uint8_t rows[2][kPageTokens][kRowBytes + 8];   // +8 keeps element bytes 16-byte aligned
    // blockIdx.y runs over the heads of all shards in turn
    int shard = 0, hs = blockIdx.y;
    while (shard + 1 < a.n_shards && hs >= a.head_count[shard]) hs -= a.head_count[shard++];
    const int h = a.head_begin[shard] + hs;
    const int64_t lp = a.token_begin / kPageTokens + blockIdx.x;            // logical page of the request
    const int32_t pid = a.page_ids[blockIdx.x];
    if (pid < 0 || pid >= cv.num_pages) {
        if (threadIdx.x == 0) atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_INGEST);
        return;
    }
    // tokens of this page that fall in the request range
    int lo = 0, hi = kPageTokens;
    if (lp * kPageTokens < a.token_begin) lo = (int)(a.token_begin - lp * kPageTokens);
    if ((lp + 1) * kPageTokens > a.token_begin + a.n_tokens) hi = (int)(a.token_begin + a.n_tokens - lp * kPageTokens);
    const bool row16 = a.layout == HMA_WIRE_TILE32;   // tile faces are 16-byte aligned; 136-byte rows only 8
    const bool exp_fast = lo == 0 && hi == kPageTokens && (a.wire_begin & 15) == 0;
    for (int item = threadIdx.x; item < 2 * kPageTokens * kBlocksPerRow; item += blockDim.x) {
        const int t = item >> 7 & 1, tok = (item >> 3) & 15, j = item & 7;
        if (tok < lo || tok >= hi) continue;
        const uint8_t *w = t ? a.v_wire[shard] : a.k_wire[shard];
        int64_t eo;
        const int64_t mo = wire_block_off(a.layout, a.wire_tokens, hs, lp * kPageTokens + tok - a.wire_begin, j, &eo);
        uint8_t *dst = &rows[t][tok][8 + 8 + j * kBlock];                    // elements start at byte 16 of the padded row
        if (row16) {
            *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(w + mo);
        } else {
            *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(w + mo);
            *reinterpret_cast<uint2 *>(dst + 8) = *reinterpret_cast<const uint2 *>(w + mo + 8);
        }
        if (!exp_fast) rows[t][tok][j] = w[eo];
    }
    if (exp_fast) {
        // whole page, page-aligned in the wire: the exponents come in 16-byte (tile face) or 8-byte (row) pieces
        const int64_t wt0 = lp * kPageTokens - a.wire_begin;
        if (row16 && threadIdx.x < 16) {
            const int t = threadIdx.x >> 3, j = threadIdx.x & 7;
            const uint8_t *w = t ? a.v_wire[shard] : a.k_wire[shard];
            int64_t eo;
            (void)wire_block_off(a.layout, a.wire_tokens, hs, wt0, j, &eo);
            const uint4 e = *reinterpret_cast<const uint4 *>(w + eo);
            const uint32_t ew[4] = {e.x, e.y, e.z, e.w};
#pragma unroll
            for (int tok = 0; tok < kPageTokens; ++tok) rows[t][tok][j] = (uint8_t)(ew[tok >> 2] >> (8 * (tok & 3)));
        } else if (!row16 && threadIdx.x < 32) {
            const int t = threadIdx.x >> 4, tok = threadIdx.x & 15;
            const uint8_t *w = t ? a.v_wire[shard] : a.k_wire[shard];
            *reinterpret_cast<uint2 *>(&rows[t][tok][0]) =
                *reinterpret_cast<const uint2 *>(w + ((int64_t)hs * a.wire_tokens + wt0 + tok) * kRowBytes);
        }
    }
    __syncthreads();
    uint8_t *rec = cv.layer + ((int64_t)pid * cv.num_kv_heads + h) * (int64_t)record_bytes(cv.format);
    // byte mask of the tokens of a V-side word (tokens 2*tq, 2*tq+1, 2*tq+8, 2*tq+9) that are in range
    auto vmask = [&](int tq) {
        uint32_t m = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int tok = 2 * tq + (k & 1) + 8 * (k >> 1);
            if (tok >= lo && tok < hi) m |= 0xFFu << (8 * k);
        }
        return m;
    };
    auto put = [&](uint32_t *dst, uint32_t val, uint32_t mask) {
        if (mask == 0xFFFFFFFFu) *dst = val;
        else if (mask) *dst = (*dst & ~mask) | (val & mask);
    };
    if (cv.format == HMA_KV_BFP8) {
        uint32_t *rk = reinterpret_cast<uint32_t *>(rec), *rv = reinterpret_cast<uint32_t *>(rec + kBfp8Half);
        // K exponents: word = blocks 4*(w&1)..+3 of token (w>>2) + 8*((w>>1)&1): four consecutive staged bytes
        // V exponents: word = block (w&7) of tokens 2*tq.., tq = w>>3
        if (threadIdx.x < 32) {
            const int w = threadIdx.x, tok = (w >> 2) + 8 * ((w >> 1) & 1);
            put(rk + w, *reinterpret_cast<const uint32_t *>(&rows[0][tok][4 * (w & 1)]), tok >= lo && tok < hi ? 0xFFFFFFFFu : 0u);
        } else if (threadIdx.x < 64) {
            const int w = threadIdx.x - 32, tq = w >> 3, j = w & 7;
            const uint32_t val = rows[1][2 * tq][j] | (rows[1][2 * tq + 1][j] << 8) | (rows[1][2 * tq + 8][j] << 16) |
                                 ((uint32_t)rows[1][2 * tq + 9][j] << 24);
            put(rv + w, val, vmask(tq));
        }
        for (int wi = threadIdx.x; wi < 512; wi += blockDim.x) {
            // K elements: four consecutive channels of one token are one word of the record
            const int c = wi >> 7, lane = (wi >> 2) & 31, w4 = wi & 3, g = lane >> 2, tq = lane & 3;
            const int tok = g + 8 * (c & 1), ch = 16 * (4 * (c >> 1) + w4) + 4 * tq;
            put(rk + 32 + wi, *reinterpret_cast<const uint32_t *>(&rows[0][tok][16 + ch]), tok >= lo && tok < hi ? 0xFFFFFFFFu : 0u);
        }
        for (int it = threadIdx.x; it < 128; it += blockDim.x) {
            // V elements: a 4-token x 4-channel block is read as four words (one per token) and transposed in registers
            // into four words of the record (one per channel)
            const int tq = it >> 5, ch0 = (it & 31) * 4;
            const uint32_t w0 = *reinterpret_cast<const uint32_t *>(&rows[1][2 * tq][16 + ch0]);
            const uint32_t w1 = *reinterpret_cast<const uint32_t *>(&rows[1][2 * tq + 1][16 + ch0]);
            const uint32_t w2 = *reinterpret_cast<const uint32_t *>(&rows[1][2 * tq + 8][16 + ch0]);
            const uint32_t w3 = *reinterpret_cast<const uint32_t *>(&rows[1][2 * tq + 9][16 + ch0]);
            const uint32_t a01 = __byte_perm(w0, w1, 0x5140), b01 = __byte_perm(w0, w1, 0x7362);
            const uint32_t a23 = __byte_perm(w2, w3, 0x5140), b23 = __byte_perm(w2, w3, 0x7362);
            const uint32_t o4[4] = {__byte_perm(a01, a23, 0x5410), __byte_perm(a01, a23, 0x7632), __byte_perm(b01, b23, 0x5410),
                                    __byte_perm(b01, b23, 0x7632)};
            const int j = ch0 >> 4, cb0 = ch0 & 15;
            const int wi0 = (j >> 1) * 128 + ((cb0 & 7) * 4 + tq) * 4 + (j & 1) * 2 + (cb0 >> 3);
            const uint32_t m = vmask(tq);
#pragma unroll
            for (int i = 0; i < 4; ++i) put(rv + 32 + wi0 + 16 * i, o4[i], m);
        }
    } else {
        // BF16 cache: decode while scattering; a word holds two elements
        uint32_t *rk = reinterpret_cast<uint32_t *>(rec), *rv = reinterpret_cast<uint32_t *>(rec + kBf16Half);
        for (int wi = threadIdx.x; wi < kBf16Half / 4; wi += blockDim.x) {
            const int c = wi >> 7, lane = (wi >> 2) & 31, w4 = wi & 3, g = lane >> 2, tq = lane & 3;
            {   // K: channels ch, ch+1 of one token
                const int tok = g + 8 * (c & 1), ch = 16 * (2 * (c >> 1) + (w4 >> 1)) + 4 * tq + 2 * (w4 & 1);
                const uint32_t E = rows[0][tok][ch >> 4];
                const uint32_t val = bfp8_to_bf16_bits(E, rows[0][tok][16 + ch]) | (bfp8_to_bf16_bits(E, rows[0][tok][16 + ch + 1]) << 16);
                put(rk + wi, val, tok >= lo && tok < hi ? 0xFFFFFFFFu : 0u);
            }
            {   // V: one channel of tokens t, t+1
                const int t = 2 * tq + 8 * (w4 >> 1), ch = 16 * c + g + 8 * (w4 & 1);
                const uint32_t val = bfp8_to_bf16_bits(rows[1][t][ch >> 4], rows[1][t][16 + ch]) |
                                     (bfp8_to_bf16_bits(rows[1][t + 1][ch >> 4], rows[1][t + 1][16 + ch]) << 16);
                const uint32_t mask = (t >= lo && t < hi ? 0xFFFFu : 0u) | (t + 1 >= lo && t + 1 < hi ? 0xFFFF0000u : 0u);
                put(rv + wi, val, mask);
            }
        }
    }
}

// ---------------------------------------------------------------- the streaming path: 32x32 tiles -> BFP8 records
// Whole pages of a tiled wire going into a BFP8 cache (the case of sections 3.2 / 3.3: every layer of an arriving
// request) take this kernel.  A work item is one tile row of one head: 32 tokens = two pages.  Its K bytes and its V
// bytes are each one contiguous 4352-byte piece of the wire (four 1088-byte tiles), fetched by one bulk async copy each
// into a four-deep ring; the CTA's 256 threads permute them into the two page records in shared memory (16-byte loads
// and stores for K, 4x4 byte transposes in registers for V), and each finished 4352-byte record leaves by one bulk
// async store.  A few hundred long-lived CTAs walk all items, so that a layer costs the GPU a few microseconds
// instead of thousands of small CTAs each waiting for a free SM beside the persistent attention kernel.
constexpr int kIngestStages = 4;            // tile rows in flight per CTA
constexpr int kIngestOut = 2;               // record pairs being written back
constexpr int kIngestThreads = 256;
constexpr int kTileRowBytes = 4 * kTileBytes;      // 4352: one tensor of one (head, 32 tokens)
constexpr uint32_t kIngestSpin = 1u << 22;

__device__ __forceinline__ uint32_t ing_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool ing_try_wait(uint32_t bar, uint32_t parity)
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

template <bool kMulti>      // kMulti: items run over several layers (the whole-request call)
__global__ void __launch_bounds__(kIngestThreads) ingest_tiles_kernel(CacheView cv, IngestArgs a, int tile_rows, int full_pages,
                                                                      void *const *__restrict__ layers, int n_layers, int64_t layer_stride)
{
    extern __shared__ __align__(128) uint8_t ing_smem[];
    uint8_t *in = ing_smem;                                              // [stages][2 tensors][4352]
    uint8_t *out = in + kIngestStages * 2 * kTileRowBytes;              // [kIngestOut][2 pages][4352]
    uint64_t *bars = reinterpret_cast<uint64_t *>(out + kIngestOut * 2 * kBfp8Record);
    const int tid = threadIdx.x;
    int heads = 0;
    for (int s = 0; s < a.n_shards; ++s) heads += a.head_count[s];
    const int per_layer = heads * tile_rows;
    const int n_items = (kMulti ? n_layers : 1) * per_layer;      // item = (layer, head, tile row); !kMulti: cv.layer is the only layer
    if (tid == 0) {
        for (int s = 0; s < kIngestStages; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(ing_smem_u32(bars + s)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    // launched with programmatic stream serialisation: nothing a predecessor may have written is read before this
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // item -> (layer, shard, head inside the shard, tile row)
    auto layer_of = [&](int item) { return kMulti ? item / per_layer : 0; };      // one layer: no division
    auto locate = [&](int item, int *shard, int *hs, int *tr) {
        if (kMulti) item %= per_layer;
        int hi = item / tile_rows;
        *tr = item - hi * tile_rows;
        int sh = 0;
        while (sh + 1 < a.n_shards && hi >= a.head_count[sh]) hi -= a.head_count[sh++];
        *shard = sh;
        *hs = hi;
    };
    auto load = [&](int item, int stage) {      // thread 0 only
        int shard, hs, tr;
        locate(item, &shard, &hs, &tr);
        const int64_t off = ((int64_t)hs * tile_rows + tr) * kTileRowBytes + (int64_t)layer_of(item) * layer_stride;
        const uint32_t bar = ing_smem_u32(bars + stage), dst = ing_smem_u32(in + stage * 2 * kTileRowBytes);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(2 * kTileRowBytes) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                     "l"(a.k_wire[shard] + off), "r"(kTileRowBytes), "r"(bar)
                     : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst + kTileRowBytes),
                     "l"(a.v_wire[shard] + off), "r"(kTileRowBytes), "r"(bar)
                     : "memory");
    };
    if (tid == 0)
        for (int s = 0; s < kIngestStages; ++s) {
            const int item = blockIdx.x + s * gridDim.x;
            if (item < n_items) load(item, s);
        }
    const int p = tid >> 7, x = tid & 127;      // this thread's page of the item and its slot inside the page
    int n = 0;
    bool gave_up = false;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
        const int stage = n % kIngestStages;
        const uint32_t parity = (n / kIngestStages) & 1;
        // the physical pages of this item are asked for now, so that the table read is over when the records are ready to leave
        int32_t pid2[2] = {-1, -1};
        if (tid == 0) {
            const int tr0 = (kMulti ? item % per_layer : item) % tile_rows;
            if (2 * tr0 < full_pages) pid2[0] = a.page_ids[2 * tr0];
            if (2 * tr0 + 1 < full_pages) pid2[1] = a.page_ids[2 * tr0 + 1];
        }
        {   // bounded wait for the tile row; the CTA decides together whether it arrived
            const uint32_t bar = ing_smem_u32(bars + stage);
            uint32_t it = 0;
            bool here = ing_try_wait(bar, parity);
            while (!here && ++it < kIngestSpin) here = ing_try_wait(bar, parity);
            gave_up = __syncthreads_or(!here);
        }
        if (gave_up) break;
        int shard, hs, tr;
        locate(item, &shard, &hs, &tr);
        const int h = a.head_begin[shard] + hs;
        const int lp = 2 * tr + p;                                       // logical page of the request (from token_begin)
        const bool page_ok = lp < full_pages;
        const uint8_t *src = in + stage * 2 * kTileRowBytes;
        uint8_t *rec = out + ((n % kIngestOut) * 2 + p) * kBfp8Record;
        if (page_ok) {
            const uint8_t *kt = src, *vt = src + kTileRowBytes;
            // K elements: destination 16-byte piece x = blocks 4*(c>>1) .. +3 of token tok, channels 4q .. 4q+3
            {
                const int c = x >> 5, lane = x & 31, tok = (lane >> 2) + 8 * (c & 1), q = lane & 3;
                uint32_t w[4];
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 4 * (c >> 1) + jj;
                    w[jj] = *reinterpret_cast<const uint32_t *>(kt + (j >> 1) * kTileBytes + 64 + (2 * p + (j & 1)) * 256 + tok * 16 + q * 4);
                }
                *reinterpret_cast<uint4 *>(rec + 128 + c * 512 + lane * 16) = make_uint4(w[0], w[1], w[2], w[3]);
            }
            // V elements: four tokens x four channels, transposed in registers.  The lanes of a warp differ in the token
            // quad, the parity of the block and the channel quad, which keeps loads and stores to two-way bank conflicts.
            {
                const int lane = x & 31, tq = lane & 3, j = 2 * (x >> 5) + ((lane >> 2) & 1), cb0 = 4 * (2 * ((lane >> 3) & 1) + (lane >> 4));
                const uint8_t *base = vt + (j >> 1) * kTileBytes + 64 + (2 * p + (j & 1)) * 256 + cb0;
                const uint32_t w0 = *reinterpret_cast<const uint32_t *>(base + (2 * tq) * 16);
                const uint32_t w1 = *reinterpret_cast<const uint32_t *>(base + (2 * tq + 1) * 16);
                const uint32_t w2 = *reinterpret_cast<const uint32_t *>(base + (2 * tq + 8) * 16);
                const uint32_t w3 = *reinterpret_cast<const uint32_t *>(base + (2 * tq + 9) * 16);
                const uint32_t a01 = __byte_perm(w0, w1, 0x5140), b01 = __byte_perm(w0, w1, 0x7362);
                const uint32_t a23 = __byte_perm(w2, w3, 0x5140), b23 = __byte_perm(w2, w3, 0x7362);
                uint32_t *rv = reinterpret_cast<uint32_t *>(rec + kBfp8Half) + 32 + (j >> 1) * 128 + ((cb0 & 7) * 4 + tq) * 4 + (j & 1) * 2 + (cb0 >> 3);
                rv[0] = __byte_perm(a01, a23, 0x5410);
                rv[16] = __byte_perm(a01, a23, 0x7632);
                rv[32] = __byte_perm(b01, b23, 0x5410);
                rv[48] = __byte_perm(b01, b23, 0x7632);
            }
            // exponents: 32 words of K, 32 of V per page
            if (x < 32) {
                const int tok = (x >> 2) + 8 * ((x >> 1) & 1);
                uint32_t val = 0;
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 4 * (x & 1) + jj;
                    val |= (uint32_t)kt[(j >> 1) * kTileBytes + (2 * p + (j & 1)) * 16 + tok] << (8 * jj);
                }
                reinterpret_cast<uint32_t *>(rec)[x] = val;
            } else if (x < 64) {
                const int w = x - 32, tq = w >> 3, j = w & 7;
                const uint8_t *e = vt + (j >> 1) * kTileBytes + (2 * p + (j & 1)) * 16;
                reinterpret_cast<uint32_t *>(rec + kBfp8Half)[w] =
                    e[2 * tq] | (e[2 * tq + 1] << 8) | (e[2 * tq + 8] << 16) | ((uint32_t)e[2 * tq + 9] << 24);
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // this thread's record bytes, before the bulk store reads them
        // the store issued two items ago read the buffer that the next item will fill: it must be through before anybody
        // passes the barrier below (at most the previous item's store is still pending here)
        if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncthreads();
        if (tid == 0) {
            for (int pp = 0; pp < 2; ++pp) {
                const int lpp = 2 * tr + pp;
                if (lpp >= full_pages) continue;
                const int32_t pid = pid2[pp];
                if (pid < 0 || pid >= cv.num_pages) { atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_INGEST); continue; }
                uint8_t *base = kMulti ? (uint8_t *)layers[layer_of(item)] : cv.layer;
                uint8_t *dst = base + ((int64_t)pid * cv.num_kv_heads + h) * (int64_t)kBfp8Record;
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
                             "r"(ing_smem_u32(out + ((n % kIngestOut) * 2 + pp) * kBfp8Record)), "r"(kBfp8Record)
                             : "memory");
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
            const int next = item + kIngestStages * gridDim.x;
            if (next < n_items) load(next, stage);
        }
    }
    if (tid == 0) {
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");         // every record has landed before the CTA leaves
        if (gave_up) {
            // a wait ran out: flag it, and give the copies still in flight a bounded chance to land before the CTA's
            // shared memory is handed to somebody else
            atomicOr(cv.flags, HMA_FLAG_WAIT_TIMEOUT);
            for (int s = 0; s < kIngestStages; ++s)
                for (uint32_t it = 0; it < (1u << 16) && !ing_try_wait(ing_smem_u32(bars + s), 0) && !ing_try_wait(ing_smem_u32(bars + s), 1); ++it) {}
        }
    }
}

// Plain BF16 rows ([head][token][128], KV made on the decode GPU) into a BF16 cache: one CTA per (page, head).
// K: two consecutive channels of a token are one word of the record; V: single elements (tokens pair up in a word).
__global__ void __launch_bounds__(128) ingest_bf16_rows_kernel(CacheView cv, IngestArgs a)
{
    int shard = 0, hs = blockIdx.y;
    while (shard + 1 < a.n_shards && hs >= a.head_count[shard]) hs -= a.head_count[shard++];
    const int h = a.head_begin[shard] + hs;
    const int64_t lp = a.token_begin / kPageTokens + blockIdx.x;
    const int32_t pid = a.page_ids[blockIdx.x];
    if (pid < 0 || pid >= cv.num_pages) {
        if (threadIdx.x == 0) atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_INGEST);
        return;
    }
    int lo = 0, hi = kPageTokens;
    if (lp * kPageTokens < a.token_begin) lo = (int)(a.token_begin - lp * kPageTokens);
    if ((lp + 1) * kPageTokens > a.token_begin + a.n_tokens) hi = (int)(a.token_begin + a.n_tokens - lp * kPageTokens);
    uint8_t *rec = cv.layer + ((int64_t)pid * cv.num_kv_heads + h) * (int64_t)kBf16Record;
    const uint16_t *kw = reinterpret_cast<const uint16_t *>(a.k_wire[shard]), *vw = reinterpret_cast<const uint16_t *>(a.v_wire[shard]);
    for (int i = threadIdx.x; i < kPageTokens * 64; i += blockDim.x) {
        const int tok = i >> 6, ch = (i & 63) * 2;
        if (tok < lo || tok >= hi) continue;
        const int64_t row = ((int64_t)hs * a.wire_tokens + (lp * kPageTokens + tok - a.wire_begin)) * kHeadDim;
        *reinterpret_cast<uint32_t *>(rec + bf16_k_el_off(tok, ch)) = *reinterpret_cast<const uint32_t *>(kw + row + ch);
        const uint32_t v2 = *reinterpret_cast<const uint32_t *>(vw + row + ch);
        *reinterpret_cast<uint16_t *>(rec + bf16_v_el_off(tok, ch)) = (uint16_t)v2;
        *reinterpret_cast<uint16_t *>(rec + bf16_v_el_off(tok, ch + 1)) = (uint16_t)(v2 >> 16);
    }
}

}  // namespace hma

static hma_status_t launch_ingest(hma_cache_t *cache, int32_t layer, int32_t n_shards, const void *const *k_wires,
                                  const void *const *v_wires, int32_t wire_layout, const int32_t *head_begins,
                                  const int32_t *head_counts, const int32_t *page_ids, int64_t token_begin, int64_t n_tokens,
                                  void *stream, int32_t n_layers = 1, size_t layer_stride = 0)
{
    // layers [layer, layer + n_layers); layer l's wire of shard s starts l * layer_stride bytes after k_wires[s] / v_wires[s]
    if (!cache || layer < 0 || n_layers < 1 || layer + n_layers > cache->desc.num_layers) return HMA_ERR_INVALID_ARG;
    if (n_layers > 1 && (layer_stride & 15u)) return HMA_ERR_ALIGNMENT;
    if (!hma::on_cache_device(cache)) return HMA_ERR_INVALID_ARG;
    if (wire_layout != HMA_WIRE_TILE32 && wire_layout != HMA_WIRE_ROWMAJOR && wire_layout != HMA_WIRE_BF16_ROWS) return HMA_ERR_INVALID_ARG;
    if (wire_layout == HMA_WIRE_BF16_ROWS && cache->desc.format != HMA_KV_BF16) return HMA_ERR_INVALID_ARG;
    if (n_shards < 1 || n_shards > hma::kMaxShards || !k_wires || !v_wires || !head_begins || !head_counts) return HMA_ERR_INVALID_ARG;
    if (token_begin < 0 || n_tokens < 0) return HMA_ERR_INVALID_ARG;
    hma::IngestArgs a = {};
    int heads = 0;
    for (int s = 0; s < n_shards; ++s) {
        if (head_begins[s] < 0 || head_counts[s] <= 0 || head_begins[s] + head_counts[s] > cache->desc.num_kv_heads) return HMA_ERR_INVALID_ARG;
        for (int t = 0; t < s; ++t)                                      // two shards may not write the same head
            if (head_begins[s] < head_begins[t] + head_counts[t] && head_begins[t] < head_begins[s] + head_counts[s]) return HMA_ERR_INVALID_ARG;
        a.k_wire[s] = (const uint8_t *)k_wires[s];
        a.v_wire[s] = (const uint8_t *)v_wires[s];
        a.head_begin[s] = head_begins[s];
        a.head_count[s] = head_counts[s];
        heads += head_counts[s];
    }
    if (n_tokens == 0) return HMA_OK;
    if (!page_ids) return HMA_ERR_INVALID_ARG;
    for (int s = 0; s < n_shards; ++s) {
        if (!a.k_wire[s] || !a.v_wire[s]) return HMA_ERR_INVALID_ARG;
        // 136-byte rows are read in 8-byte pieces (what hma_bfp8_encode_rows promises for its output); tiles and BF16 rows in 16-byte pieces
        const uintptr_t need = wire_layout == HMA_WIRE_ROWMAJOR ? 7u : 15u;
        if (((uintptr_t)a.k_wire[s] & need) || ((uintptr_t)a.v_wire[s] & need)) return HMA_ERR_ALIGNMENT;
    }
    const int64_t first = token_begin / hma::kPageTokens;
    const int64_t last = (token_begin + n_tokens - 1) / hma::kPageTokens;
    const int64_t n_pages = last - first + 1;
    if (n_pages > 0x7FFFFFFF) return HMA_ERR_INVALID_ARG;
    hma::CacheView cv{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    a.n_shards = n_shards;
    a.page_ids = page_ids;
    a.token_begin = token_begin;
    a.n_tokens = n_tokens;
    a.wire_begin = token_begin;
    a.wire_tokens = n_tokens;
    a.layout = wire_layout;
    cudaStream_t st = (cudaStream_t)stream;
    const bool streaming = wire_layout == HMA_WIRE_TILE32 && cache->desc.format == HMA_KV_BFP8 && (token_begin & 15) == 0 &&
                           n_tokens >= hma::kPageTokens && n_tokens / hma::kPageTokens <= 0x3FFFFFFF &&
                           (int64_t)n_layers * heads * ((n_tokens + 31) / 32) <= 0x7FFFFFFF;
    if (n_layers > 1 && !streaming) {
        // no streaming path for this case: layer by layer
        for (int l = 0; l < n_layers; ++l) {
            const void *kw[hma::kMaxShards], *vw[hma::kMaxShards];
            for (int s = 0; s < n_shards; ++s) {
                kw[s] = (const uint8_t *)k_wires[s] + (size_t)l * layer_stride;
                vw[s] = (const uint8_t *)v_wires[s] + (size_t)l * layer_stride;
            }
            const hma_status_t r = launch_ingest(cache, layer + l, n_shards, kw, vw, wire_layout, head_begins, head_counts, page_ids,
                                                 token_begin, n_tokens, stream);
            if (r != HMA_OK) return r;
        }
        return HMA_OK;
    }
    if (streaming) {
        // whole pages of a tiled wire: the streaming kernel; a ragged last page (if any) follows through the general kernel
        static std::mutex setup_lock;
        static int sm_count[64] = {};
        int dev = 0;
        HMA_CUDA_OK(cudaGetDevice(&dev));
        if (dev < 0 || dev >= 64) return HMA_ERR_UNSUPPORTED_SHAPE;
        const size_t smem = (size_t)(hma::kIngestStages * 2 * hma::kTileRowBytes + hma::kIngestOut * 2 * hma::kBfp8Record + hma::kIngestStages * 8);
        {
            std::lock_guard<std::mutex> guard(setup_lock);
            if (!sm_count[dev]) {
                int n = 0;
                HMA_CUDA_OK(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
                HMA_CUDA_OK(cudaFuncSetAttribute(hma::ingest_tiles_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
                HMA_CUDA_OK(cudaFuncSetAttribute(hma::ingest_tiles_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
                sm_count[dev] = n;
            }
        }
        const int full_pages = (int)(n_tokens / hma::kPageTokens);
        const int tile_rows = (int)((n_tokens + 31) / 32);
        const int64_t items = (int64_t)heads * ((full_pages + 1) / 2);
        // items are numbered over all tile rows of the wire; a last tile row without a whole page holds no item to do,
        // but keeping the wire's own row count in the numbering keeps the addressing plain
        (void)items;
        const int64_t n_items = (int64_t)n_layers * heads * tile_rows;
        const int64_t max_ctas = (int64_t)sm_count[dev] * 4;
        const unsigned grid_x = (unsigned)(n_items < max_ctas ? n_items : max_ctas);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid_x);
        cfg.blockDim = dim3(hma::kIngestThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        void *const *layers = n_layers > 1 ? (void *const *)(cache->d_layers + layer) : nullptr;
        if (n_layers > 1)
            HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::ingest_tiles_kernel<true>, cv, a, tile_rows, full_pages, layers, (int)n_layers, (int64_t)layer_stride));
        else
            HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::ingest_tiles_kernel<false>, cv, a, tile_rows, full_pages, layers, 1, (int64_t)0));
        hma::count_launch();
        const int64_t rest = n_tokens - (int64_t)full_pages * hma::kPageTokens;
        if (rest == 0) return HMA_OK;
        a.token_begin = token_begin + (int64_t)full_pages * hma::kPageTokens;
        a.n_tokens = rest;
        a.page_ids = page_ids + full_pages;
        dim3 tail_grid(1u, (unsigned)heads);
        for (int l = 0; l < n_layers; ++l) {      // the ragged last page, layer by layer, through the general kernel
            cv.layer = (uint8_t *)cache->layers[layer + l];
            for (int s = 0; s < n_shards; ++s) {
                a.k_wire[s] = (const uint8_t *)k_wires[s] + (size_t)l * layer_stride;
                a.v_wire[s] = (const uint8_t *)v_wires[s] + (size_t)l * layer_stride;
            }
            hma::ingest_kernel<<<tail_grid, 128, 0, st>>>(cv, a);
            hma::count_launch();
        }
        HMA_CUDA_OK(cudaGetLastError());
        return HMA_OK;
    }
    dim3 grid((unsigned)n_pages, (unsigned)heads);
    if (wire_layout == HMA_WIRE_BF16_ROWS) hma::ingest_bf16_rows_kernel<<<grid, 128, 0, st>>>(cv, a);
    else hma::ingest_kernel<<<grid, 128, 0, st>>>(cv, a);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_kv_ingest_layer(hma_cache_t *cache, int32_t layer, const void *k_wire, const void *v_wire,
                                            int32_t wire_layout, int32_t head_begin, int32_t head_count,
                                            const int32_t *page_ids, int64_t token_begin, int64_t n_tokens, void *stream)
{
    return launch_ingest(cache, layer, 1, &k_wire, &v_wire, wire_layout, &head_begin, &head_count, page_ids, token_begin,
                         n_tokens, stream);
}

extern "C" hma_status_t hma_kv_ingest_layer_shards(hma_cache_t *cache, int32_t layer, int32_t n_shards,
                                                   const void *const *k_wires, const void *const *v_wires,
                                                   int32_t wire_layout, const int32_t *head_begins, const int32_t *head_counts,
                                                   const int32_t *page_ids, int64_t token_begin, int64_t n_tokens, void *stream)
{
    return launch_ingest(cache, layer, n_shards, k_wires, v_wires, wire_layout, head_begins, head_counts, page_ids,
                         token_begin, n_tokens, stream);
}

extern "C" hma_status_t hma_kv_ingest_request_shards(hma_cache_t *cache, int32_t n_shards, const void *const *k_wires,
                                                     const void *const *v_wires, size_t layer_stride_bytes, int32_t wire_layout,
                                                     const int32_t *head_begins, const int32_t *head_counts, const int32_t *page_ids,
                                                     int64_t token_begin, int64_t n_tokens, void *stream)
{
    if (!cache) return HMA_ERR_INVALID_ARG;
    return launch_ingest(cache, 0, n_shards, k_wires, v_wires, wire_layout, head_begins, head_counts, page_ids, token_begin, n_tokens,
                         stream, cache->desc.num_layers, layer_stride_bytes);
}

