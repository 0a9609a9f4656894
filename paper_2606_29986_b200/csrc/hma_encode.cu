// FP32 / BF16 rows -> BFP8 wire rows on the GPU (the producer-side format of section 3.1, written here so that
// KV made on the decode GPU, e.g. of freshly generated tokens, can enter the same cache through the ingest call).
// Bit-identical to the reference encoder: shared exponent = largest FP32 exponent field of the 16-element block,
// significands shifted to it and rounded to nearest-even onto 7 bits, a carry saturates at 127, FP32 subnormals
// encode as zero, the sign bit is always copied.  NaN/Inf inputs raise HMA_FLAG_BAD_VALUE_ENCODE and encode as zero.
#include "hma_common.cuh"

namespace hma {

// One warp per row of 128 channels: lane l holds channels 4l .. 4l+3, four lanes share a block.
template <bool kBf16In>
__global__ void __launch_bounds__(256) encode_rows_kernel(const void *__restrict__ x, int64_t n_rows, uint8_t *__restrict__ wire,
                                                          uint32_t *__restrict__ flags)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    bool bad = false;
    for (int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); row < n_rows; row += warps) {
        uint32_t bits[4];
        if (kBf16In) {
            const uint2 v = reinterpret_cast<const uint2 *>(x)[row * 32 + lane];
            bits[0] = v.x << 16; bits[1] = v.x & 0xFFFF0000u; bits[2] = v.y << 16; bits[3] = v.y & 0xFFFF0000u;
        } else {
            const uint4 v = reinterpret_cast<const uint4 *>(x)[row * 32 + lane];
            bits[0] = v.x; bits[1] = v.y; bits[2] = v.z; bits[3] = v.w;
        }
        uint32_t E = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t e = (bits[k] >> 23) & 0xFFu;
            if (e == 0xFFu) { bad = true; bits[k] &= 0x80000000u; e = 0; }
            E = max(E, e);
        }
        E = max(E, __shfl_xor_sync(0xFFFFFFFFu, E, 1));
        E = max(E, __shfl_xor_sync(0xFFFFFFFFu, E, 2));
        uint32_t packed = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t e = (bits[k] >> 23) & 0xFFu;
            uint32_t q = 0;
            if (e != 0) {
                const uint32_t sig = 0x800000u | (bits[k] & 0x7FFFFFu);
                const uint32_t sh = 17u + (E - e);
                if (sh < 32u) {
                    q = sig >> sh;
                    const uint32_t rem = sig & ((1u << sh) - 1u), half = 1u << (sh - 1u);
                    if (rem > half || (rem == half && (q & 1u))) ++q;
                }
                q = min(q, 127u);
            }
            packed |= (((bits[k] >> 31) << 7) | q) << (8 * k);
        }
        uint8_t *out = wire + row * kRowBytes;
        *reinterpret_cast<uint32_t *>(out + kBlocksPerRow + 4 * lane) = packed;
        if ((lane & 3) == 0) out[lane >> 2] = (uint8_t)E;
    }
    if (bad) atomicOr(flags, HMA_FLAG_BAD_VALUE_ENCODE);
}

}  // namespace hma

extern "C" hma_status_t hma_bfp8_encode_rows(const hma_cache_t *cache, const void *x, int32_t x_is_bf16, int64_t n_rows,
                                             void *wire_rowmajor, void *stream)
{
    if (!cache || n_rows < 0 || (x_is_bf16 != 0 && x_is_bf16 != 1)) return HMA_ERR_INVALID_ARG;
    if (!hma::on_cache_device(cache)) return HMA_ERR_INVALID_ARG;
    if (n_rows == 0) return HMA_OK;
    if (!x || !wire_rowmajor) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)x & 15u) || ((uintptr_t)wire_rowmajor & 7u)) return HMA_ERR_ALIGNMENT;
    int64_t blocks = (n_rows + 7) / 8;
    if (blocks > 148 * 16) blocks = 148 * 16;
    if (x_is_bf16)
        hma::encode_rows_kernel<true><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(x, n_rows, (uint8_t *)wire_rowmajor, cache->flags);
    else
        hma::encode_rows_kernel<false><<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(x, n_rows, (uint8_t *)wire_rowmajor, cache->flags);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}
