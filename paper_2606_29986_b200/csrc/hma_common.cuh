// Shared definitions of the CUDA library: cache geometry, record layouts, bit-exact element decode.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hma.h"

namespace hma {

constexpr int kHeadDim = 128;
constexpr int kPageTokens = 16;
constexpr int kBlock = 16;
constexpr int kBlocksPerRow = kHeadDim / kBlock;           // 8
constexpr int kRowBytes = kBlocksPerRow + kHeadDim;        // 136: wire bytes of one (token, head, tensor)
constexpr int kTileBytes = 1088;                           // one 32x32 wire tile
constexpr int kBfp8Half = 2176;                            // K (or V) part of a BFP8 record
constexpr int kBfp8Record = 2 * kBfp8Half;                 // 4352
constexpr int kBf16Half = 4096;
constexpr int kBf16Record = 2 * kBf16Half;                 // 8192
constexpr int kMaxGroup = 8;                               // q heads per kv head
constexpr int kMaxKvHeads = 64;                            // kv heads per layer

struct CacheView {
    uint8_t *layer;        // base of one layer
    int64_t num_pages;
    int32_t num_kv_heads;
    int32_t num_q_heads;
    int32_t format;        // hma_kv_format_t
    uint32_t *flags;       // device flag word
    int32_t key_layout;    // hma_key_layout_t
};

__host__ __device__ inline int record_bytes(int format) { return format == HMA_KV_BFP8 ? kBfp8Record : kBf16Record; }

// ---- positions inside a BFP8 record (K part at 0, V part at kBfp8Half) ----
__host__ __device__ inline int bfp8_k_exp_off(int tok, int j) { return (tok & 7) * 16 + (tok >> 3) * 8 + j; }
__host__ __device__ inline int bfp8_k_el_off(int tok, int ch)
{
    int j = ch >> 4, cb = ch & 15;
    return 128 + ((tok >> 3) + 2 * (j >> 2)) * 512 + ((tok & 7) * 4 + (cb >> 2)) * 16 + (j & 3) * 4 + (cb & 3);
}
__host__ __device__ inline int bfp8_v_tok_k(int tok) { return (tok & 1) + 2 * (tok >> 3); }
__host__ __device__ inline int bfp8_v_exp_off(int tok, int j)
{
    return kBfp8Half + ((tok & 7) >> 1) * 32 + j * 4 + bfp8_v_tok_k(tok);
}
__host__ __device__ inline int bfp8_v_el_off(int tok, int ch)
{
    int j = ch >> 4, cb = ch & 15;
    return kBfp8Half + 128 + (j >> 1) * 512 + ((cb & 7) * 4 + ((tok & 7) >> 1)) * 16 + ((j & 1) * 2 + (cb >> 3)) * 4 +
           bfp8_v_tok_k(tok);
}
// ---- positions (in bytes) inside a BF16 record ----
__host__ __device__ inline int bf16_k_el_off(int tok, int ch)
{
    int j = ch >> 4, cb = ch & 15;
    return ((tok >> 3) + 2 * (j >> 1)) * 512 + ((tok & 7) * 4 + (cb >> 2)) * 16 + (j & 1) * 8 + (cb & 3) * 2;
}
__host__ __device__ inline int bf16_v_el_off(int tok, int ch)
{
    int j = ch >> 4, cb = ch & 15;
    return kBf16Half + j * 512 + ((cb & 7) * 4 + ((tok & 7) >> 1)) * 16 + ((tok >> 3) * 2 + (cb >> 3)) * 4 + (tok & 1) * 2;
}

// Block-float decode of one element to its BF16 bit pattern by integer bit assembly
// (shifts, masks, ORs: section 3.3).  value = (-1)^s * m * 2^(E-133); exact for every E <= 254.
__device__ __forceinline__ uint32_t bfp8_to_bf16_bits(uint32_t E, uint32_t b)
{
    uint32_t m = b & 0x7Fu;
    uint32_t s = (b & 0x80u) << 8;
    if (m == 0) return s;
    int p = 31 - __clz(m);                 // position of the leading one, 0..6
    int ef = (int)E + p - 6;               // BF16 exponent field of the normalised value
    uint32_t r;
    if (ef >= 255) r = 0x7F80u;            // only E = 255, m >= 64: overflow to Inf
    else if (ef >= 1) r = ((uint32_t)ef << 7) | ((m << (7 - p)) & 0x7Fu);
    else r = m << E;                       // BF16 subnormal: m * 2^E units of 2^-133
    return s | r;
}

// half-split position of cached key channel c when keys are cached with rotary pairs interleaved
__host__ __device__ inline int key_channel_of_query(int c, int key_layout) { return key_layout == HMA_KEYS_INTERLEAVED ? (c >> 1) + 64 * (c & 1) : c; }

__device__ __forceinline__ float bf16_bits_to_float(uint32_t h) { return __uint_as_float(h << 16); }

void count_launch();

}  // namespace hma

struct hma_cache {
    hma_cache_desc_t desc;
    void **layers;       // host copy of the device pointers
    uint32_t *flags;     // device flag word (first word of the handle's one device allocation)
    void **d_layers;     // device copy of the layer pointers (same allocation, after the flag word)
    int device;
};

namespace hma {
void note_cuda_error(cudaError_t e);
// A handle holds pointers of the device it was created on: every launch path refuses to run with another device current.
inline bool on_cache_device(const hma_cache *c)
{
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == c->device;
}
}  // namespace hma

#define HMA_CUDA_OK(expr)                          \
    do {                                           \
        cudaError_t hma_e_ = (expr);               \
        if (hma_e_ != cudaSuccess) {               \
            hma::note_cuda_error(hma_e_);          \
            (void)cudaGetLastError();              \
            return HMA_ERR_CUDA;                   \
        }                                          \
    } while (0)
