// Instrumentation only: a plain contiguous read of device memory, the simplest upper bound on what any
// read-only kernel can pull from HBM on this GPU (section 2.2: decode attention is memory-bound, so its ceiling
// is a read stream).  Not part of the decode path.
#include "hma_common.cuh"

namespace hma {

// Grid-stride 16-byte streaming loads, eight in flight per thread; the XOR of everything read is kept live by a
// store that practically never happens.
__global__ void __launch_bounds__(512) hbm_read_kernel(const uint4 *__restrict__ src, int64_t n16, uint32_t *sink)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint4 acc = make_uint4(0u, 0u, 0u, 0u);
    for (; i + 7 * stride < n16; i += 8 * stride) {
        uint4 v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = __ldcs(src + i + k * stride);
#pragma unroll
        for (int k = 0; k < 8; ++k) { acc.x ^= v[k].x; acc.y ^= v[k].y; acc.z ^= v[k].z; acc.w ^= v[k].w; }
    }
    for (; i < n16; i += stride) {
        const uint4 v = __ldcs(src + i);
        acc.x ^= v.x; acc.y ^= v.y; acc.z ^= v.z; acc.w ^= v.w;
    }
    if ((acc.x ^ acc.y) == 0x9E3779B9u && (acc.z ^ acc.w) == 0x7F4A7C15u) atomicAdd(sink, 1u);
}

// A streaming read of `r16` 16-byte pieces mixed with a streaming write of `w16` pieces (r16 <= w16 < 2^31): written
// piece i carries source piece (i * ratio) >> 32 with ratio = floor(2^32 r16 / w16), so neighbouring threads share
// source sectors and every source byte is read once from HBM.  The simplest kernel with the byte counts of a conversion that expands its input.
__global__ void __launch_bounds__(512) hbm_copy_kernel(const uint4 *__restrict__ src, uint64_t ratio, uint4 *__restrict__ dst, int64_t w16)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < w16; i += stride) {
        uint4 v = __ldcs(src + (((uint64_t)i * ratio) >> 32));
        v.x += (uint32_t)i;
        __stcs(dst + i, v);
    }
}

}  // namespace hma

extern "C" hma_status_t hma_hbm_read_probe(const void *src, size_t bytes, void *sink4, void *stream)
{
    if (!src || !sink4) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)src & 15u) || ((uintptr_t)sink4 & 3u)) return HMA_ERR_ALIGNMENT;
    if (bytes < 16) return HMA_OK;
    int dev = 0, n_sm = 0;
    HMA_CUDA_OK(cudaGetDevice(&dev));
    HMA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    hma::hbm_read_kernel<<<(unsigned)(n_sm * 4), 512, 0, (cudaStream_t)stream>>>((const uint4 *)src, (int64_t)(bytes / 16), (uint32_t *)sink4);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_hbm_copy_probe(const void *src, size_t read_bytes, void *dst, size_t write_bytes, void *stream)
{
    if (!src || !dst || read_bytes > write_bytes || write_bytes / 16 > 0x7FFFFFFFull) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)src & 15u) || ((uintptr_t)dst & 15u)) return HMA_ERR_ALIGNMENT;
    if (read_bytes < 16) return HMA_OK;
    int dev = 0, n_sm = 0;
    HMA_CUDA_OK(cudaGetDevice(&dev));
    HMA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    hma::hbm_copy_kernel<<<(unsigned)(n_sm * 16), 512, 0, (cudaStream_t)stream>>>((const uint4 *)src, ((uint64_t)(read_bytes / 16) << 32) / (write_bytes / 16),
                                                                                  (uint4 *)dst, (int64_t)(write_bytes / 16));
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}
