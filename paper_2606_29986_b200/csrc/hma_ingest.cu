// Per-layer ingest: wire bytes (row-major or 32x32 tiles, one producer shard) -> page records
// (sections 3.2 / 3.3: host-to-device copy done by the caller or by mapped reads here, then the
// tiled -> paged re-layout that merges per-chip shards).  Byte values are never changed on a BFP8
// cache; on a BF16 cache each element is decoded while it is scattered.
#include "hma_common.cuh"

namespace hma {

struct IngestArgs {
    const uint8_t *k_wire, *v_wire;
    const int32_t *page_ids;
    int64_t token_begin, n_tokens;
    int32_t layout, head_begin, head_count;
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
__global__ void __launch_bounds__(256) ingest_kernel(CacheView cv, IngestArgs a)
{
    __shared__ __align__(16) uint8_t rows[2][kPageTokens][kRowBytes + 8];   // +8 keeps element bytes 16-byte aligned
    const int hs = blockIdx.y;
    const int h = a.head_begin + hs;
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
    for (int item = threadIdx.x; item < 2 * kPageTokens * kBlocksPerRow; item += blockDim.x) {
        const int t = item >> 7 & 1, tok = (item >> 3) & 15, j = item & 7;
        if (tok < lo || tok >= hi) continue;
        const uint8_t *w = t ? a.v_wire : a.k_wire;
        int64_t eo;
        const int64_t mo = wire_block_off(a.layout, a.n_tokens, hs, lp * kPageTokens + tok - a.token_begin, j, &eo);
        uint8_t *dst = &rows[t][tok][8 + 8 + j * kBlock];                    // elements start at byte 16 of the padded row
        if (row16) {
            *reinterpret_cast<uint4 *>(dst) = *reinterpret_cast<const uint4 *>(w + mo);
        } else {
            *reinterpret_cast<uint2 *>(dst) = *reinterpret_cast<const uint2 *>(w + mo);
            *reinterpret_cast<uint2 *>(dst + 8) = *reinterpret_cast<const uint2 *>(w + mo + 8);
        }
        rows[t][tok][j] = w[eo];
    }
    __syncthreads();
    uint8_t *rec = cv.layer + ((int64_t)pid * cv.num_kv_heads + h) * (int64_t)record_bytes(cv.format);
    const bool full = lo == 0 && hi == kPageTokens;
    if (cv.format == HMA_KV_BFP8) {
        for (int wi = threadIdx.x; wi < kBfp8Record / 4; wi += blockDim.x) {
            const int t = wi >= kBfp8Half / 4;
            const int o = wi * 4 - t * kBfp8Half;        // offset inside the K or V part
            uint32_t val = 0, mask = 0;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                int tok, src;
                const int ob = o + k;
                if (ob < 128) {                          // exponent bytes
                    int j;
                    if (t == 0) { tok = (ob >> 4) + 8 * ((ob >> 3) & 1); j = ob & 7; }
                    else { const int kk = ob & 3; tok = 2 * (ob >> 5) + (kk & 1) + 8 * (kk >> 1); j = (ob >> 2) & 7; }
                    src = j;
                } else {                                  // element bytes
                    const int e = ob - 128, c = e >> 9, r = e & 511, lane = r >> 4, w4 = (r >> 2) & 3, kk = r & 3;
                    const int g = lane >> 2, tq = lane & 3;
                    int ch;
                    if (t == 0) { tok = g + 8 * (c & 1); ch = 16 * (4 * (c >> 1) + w4) + 4 * tq + kk; }
                    else { tok = 2 * tq + (kk & 1) + 8 * (kk >> 1); ch = 16 * (2 * c + (w4 >> 1)) + g + 8 * (w4 & 1); }
                    src = 16 + ch;
                }
                if (tok >= lo && tok < hi) {
                    val |= (uint32_t)rows[t][tok][src] << (8 * k);
                    mask |= 0xFFu << (8 * k);
                }
            }
            uint32_t *dst = reinterpret_cast<uint32_t *>(rec) + wi;
            if (mask == 0xFFFFFFFFu) *dst = val;
            else if (mask) *dst = (*dst & ~mask) | val;
        }
    } else {
        (void)full;
        for (int wi = threadIdx.x; wi < kBf16Record / 4; wi += blockDim.x) {
            const int t = wi >= kBf16Half / 4;
            const int o = wi * 4 - t * kBf16Half;
            uint32_t val = 0, mask = 0;
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int ob = o + 2 * k, c = ob >> 9, r = ob & 511, lane = r >> 4, w4 = (r >> 2) & 3, kk = (r >> 1) & 1;
                const int g = lane >> 2, tq = lane & 3;
                int tok, ch;
                if (t == 0) { tok = g + 8 * (c & 1); ch = 16 * (2 * (c >> 1) + (w4 >> 1)) + 4 * tq + 2 * (w4 & 1) + kk; }
                else { tok = 2 * tq + kk + 8 * (w4 >> 1); ch = 16 * c + g + 8 * (w4 & 1); }
                if (tok >= lo && tok < hi) {
                    val |= bfp8_to_bf16_bits(rows[t][tok][ch >> 4], rows[t][tok][16 + ch]) << (16 * k);
                    mask |= 0xFFFFu << (16 * k);
                }
            }
            uint32_t *dst = reinterpret_cast<uint32_t *>(rec) + wi;
            if (mask == 0xFFFFFFFFu) *dst = val;
            else if (mask) *dst = (*dst & ~mask) | val;
        }
    }
}

}  // namespace hma

extern "C" hma_status_t hma_kv_ingest_layer(hma_cache_t *cache, int32_t layer, const void *k_wire, const void *v_wire,
                                            int32_t wire_layout, int32_t head_begin, int32_t head_count,
                                            const int32_t *page_ids, int64_t token_begin, int64_t n_tokens, void *stream)
{
    if (!cache || layer < 0 || layer >= cache->desc.num_layers) return HMA_ERR_INVALID_ARG;
    if (wire_layout != HMA_WIRE_TILE32 && wire_layout != HMA_WIRE_ROWMAJOR) return HMA_ERR_INVALID_ARG;
    if (head_begin < 0 || head_count <= 0 || head_begin + head_count > cache->desc.num_kv_heads) return HMA_ERR_INVALID_ARG;
    if (token_begin < 0 || n_tokens < 0) return HMA_ERR_INVALID_ARG;
    if (n_tokens == 0) return HMA_OK;
    if (!k_wire || !v_wire || !page_ids) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)k_wire & 15u) || ((uintptr_t)v_wire & 15u)) return HMA_ERR_ALIGNMENT;
    const int64_t first = token_begin / hma::kPageTokens;
    const int64_t last = (token_begin + n_tokens - 1) / hma::kPageTokens;
    const int64_t n_pages = last - first + 1;
    if (n_pages > 0x7FFFFFFF) return HMA_ERR_INVALID_ARG;
    hma::CacheView cv{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags};
    hma::IngestArgs a{(const uint8_t *)k_wire, (const uint8_t *)v_wire, page_ids, token_begin, n_tokens,
                      wire_layout, head_begin, head_count};
    dim3 grid((unsigned)n_pages, (unsigned)head_count);
    hma::ingest_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(cv, a);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}
