// Stand-alone BFP8 -> BF16 reconstruction (section 3.3: block-float decode to BF16, bit-exact).
#include "hma_common.cuh"

namespace hma {

// Flat blocks: two threads per block, 8 elements each; 8-byte loads, 16-byte stores, both coalesced.
__global__ void __launch_bounds__(256) dequant_blocks_kernel(const uint8_t *__restrict__ exps,
                                                             const uint8_t *__restrict__ mants, int64_t n_blocks,
                                                             uint16_t *__restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // index of an 8-element half block
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < 2 * n_blocks; i += stride) {
        uint32_t E = exps[i >> 1];
        uint2 m = *reinterpret_cast<const uint2 *>(mants + i * 8);
        uint32_t w[2] = {m.x, m.y};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t lo = bfp8_to_bf16_bits(E, (w[k >> 1] >> ((k & 1) * 16)) & 0xFFu);
            uint32_t hi = bfp8_to_bf16_bits(E, (w[k >> 1] >> ((k & 1) * 16 + 8)) & 0xFFu);
            o[k] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4 *>(out + i * 8) = make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// One CTA per (logical page of the request, kv head): stage the K or V part of the record in shared
// memory, then each thread rebuilds 8 consecutive channels of one token and stores 16 bytes.
__global__ void __launch_bounds__(128) dequant_paged_kernel(CacheView cv, int which, const int32_t *__restrict__ page_ids,
                                                            int64_t token_begin, int64_t n_tokens,
                                                            uint16_t *__restrict__ out)
{
    __shared__ __align__(16) uint8_t rec[kBf16Half];
    const int h = blockIdx.y;
    const int64_t first_page = token_begin / kPageTokens;
    const int64_t lp = first_page + blockIdx.x;
    const int32_t pid = page_ids[blockIdx.x];
    const bool bad = pid < 0 || pid >= cv.num_pages;
    const int half = cv.format == HMA_KV_BFP8 ? kBfp8Half : kBf16Half;
    if (!bad) {
        const uint8_t *src = cv.layer + ((int64_t)pid * cv.num_kv_heads + h) * (int64_t)(2 * half) + (int64_t)which * half;
        for (int o = threadIdx.x * 16; o < half; o += blockDim.x * 16)
            *reinterpret_cast<uint4 *>(rec + o) = *reinterpret_cast<const uint4 *>(src + o);
    } else if (threadIdx.x == 0) {
        atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_DEQUANT);
    }
    __syncthreads();
    for (int item = threadIdx.x; item < kPageTokens * 16; item += blockDim.x) {
        const int tok = item >> 4, c0 = (item & 15) * 8;
        const int64_t gt = lp * kPageTokens + tok;
        if (gt < token_begin || gt >= token_begin + n_tokens) continue;
        uint32_t o[4] = {0, 0, 0, 0};
        if (!bad) {
            if (cv.format == HMA_KV_BFP8) {
                // `rec` holds one half record: offsets are relative to the start of that half
                const uint32_t E = which == 0 ? rec[bfp8_k_exp_off(tok, c0 >> 4)] : rec[bfp8_v_exp_off(tok, c0 >> 4) - kBfp8Half];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int ch = c0 + k;
                    const uint32_t b = which == 0 ? rec[bfp8_k_el_off(tok, ch)] : rec[bfp8_v_el_off(tok, ch) - kBfp8Half];
                    o[k >> 1] |= bfp8_to_bf16_bits(E, b) << ((k & 1) * 16);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const int ch = c0 + k;
                    const int off = which == 0 ? bf16_k_el_off(tok, ch) : bf16_v_el_off(tok, ch) - kBf16Half;
                    o[k >> 1] |= (uint32_t)(*reinterpret_cast<const uint16_t *>(rec + off)) << ((k & 1) * 16);
                }
            }
        }
        uint16_t *row = out + ((gt - token_begin) * cv.num_kv_heads + h) * kHeadDim;
        if (which == 0 && cv.key_layout == HMA_KEYS_INTERLEAVED) {
            // keys cached with rotary pairs interleaved leave in half-split order (section 3.3, key re-layout):
            // cached channels c0, c0+2, .. go to c0/2 .., cached channels c0+1, c0+3, .. to 64 + c0/2 ..
            const uint32_t e0 = (o[0] & 0xFFFFu) | (o[1] << 16), e1 = (o[2] & 0xFFFFu) | (o[3] << 16);
            const uint32_t d0 = (o[0] >> 16) | (o[1] & 0xFFFF0000u), d1 = (o[2] >> 16) | (o[3] & 0xFFFF0000u);
            *reinterpret_cast<uint2 *>(row + (c0 >> 1)) = make_uint2(e0, e1);
            *reinterpret_cast<uint2 *>(row + 64 + (c0 >> 1)) = make_uint2(d0, d1);
        } else {
            *reinterpret_cast<uint4 *>(row + c0) = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

}  // namespace hma

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
    if (n_tokens == 0) return HMA_OK;
    if (!page_ids || !out_bf16) return HMA_ERR_INVALID_ARG;
    if ((uintptr_t)out_bf16 & 15u) return HMA_ERR_ALIGNMENT;
    const int64_t first = token_begin / hma::kPageTokens;
    const int64_t last = (token_begin + n_tokens - 1) / hma::kPageTokens;
    const int64_t n_pages = last - first + 1;
    if (n_pages > 0x7FFFFFFF) return HMA_ERR_INVALID_ARG;
    hma::CacheView cv{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    dim3 grid((unsigned)n_pages, (unsigned)cache->desc.num_kv_heads);
    hma::dequant_paged_kernel<<<grid, 128, 0, (cudaStream_t)stream>>>(cv, which, page_ids, token_begin, n_tokens,
                                                                      (uint16_t *)out_bf16);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}
