// Cache handle, status strings, flag word, launch accounting (host side of the C ABI).
#include <atomic>
#include <cstdlib>
#include <cstring>

#include "hma_common.cuh"

namespace hma {
static std::atomic<long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
static thread_local cudaError_t g_last_error = cudaSuccess;
void note_cuda_error(cudaError_t e) { g_last_error = e; }
}  // namespace hma

static bool desc_ok(const hma_cache_desc_t *d)
{
    if (!d) return false;
    if (d->head_dim != hma::kHeadDim || d->page_tokens != hma::kPageTokens || d->bfp_block != hma::kBlock) return false;
    if (d->num_layers <= 0 || d->num_kv_heads <= 0 || d->num_q_heads <= 0 || d->num_pages <= 0) return false;
    if (d->num_kv_heads > hma::kMaxKvHeads) return false;
    if (d->num_q_heads % d->num_kv_heads) return false;
    int g = d->num_q_heads / d->num_kv_heads;
    if (g < 1 || g > hma::kMaxGroup) return false;
    if (d->format != HMA_KV_BFP8 && d->format != HMA_KV_BF16) return false;
    if (d->key_layout != HMA_KEYS_AS_QUERIES && d->key_layout != HMA_KEYS_INTERLEAVED) return false;
    return true;
}

extern "C" size_t hma_cache_layer_bytes(const hma_cache_desc_t *desc)
{
    if (!desc_ok(desc)) return 0;
    return (size_t)desc->num_pages * (size_t)desc->num_kv_heads * (size_t)hma::record_bytes(desc->format);
}

extern "C" hma_status_t hma_cache_create(const hma_cache_desc_t *desc, void *const *layer_ptrs, hma_cache_t **out)
{
    if (!out) return HMA_ERR_INVALID_ARG;
    *out = nullptr;
    if (!desc || !layer_ptrs) return HMA_ERR_INVALID_ARG;
    if (!desc_ok(desc)) return HMA_ERR_UNSUPPORTED_SHAPE;
    for (int l = 0; l < desc->num_layers; ++l) {
        if (!layer_ptrs[l]) return HMA_ERR_INVALID_ARG;
        if ((uintptr_t)layer_ptrs[l] & 255u) return HMA_ERR_ALIGNMENT;
    }
    hma_cache *c = (hma_cache *)std::calloc(1, sizeof(hma_cache));
    if (!c) return HMA_ERR_INVALID_ARG;
    c->desc = *desc;
    c->layers = (void **)std::malloc(sizeof(void *) * (size_t)desc->num_layers);
    std::memcpy(c->layers, layer_ptrs, sizeof(void *) * (size_t)desc->num_layers);
    // one small device allocation: the flag word (16 bytes reserved), then the table of layer pointers
    const size_t table = sizeof(void *) * (size_t)desc->num_layers;
    if (cudaGetDevice(&c->device) != cudaSuccess || cudaMalloc((void **)&c->flags, 16 + table) != cudaSuccess ||
        cudaMemset(c->flags, 0, 16) != cudaSuccess ||
        cudaMemcpy((uint8_t *)c->flags + 16, layer_ptrs, table, cudaMemcpyHostToDevice) != cudaSuccess) {
        if (c->flags) (void)cudaFree(c->flags);
        (void)cudaGetLastError();
        std::free(c->layers);
        std::free(c);
        return HMA_ERR_CUDA;
    }
    c->d_layers = (void **)((uint8_t *)c->flags + 16);
    *out = c;
    return HMA_OK;
}

extern "C" void hma_cache_destroy(hma_cache_t *cache)
{
    if (!cache) return;
    if (cache->flags) (void)cudaFree(cache->flags);
    std::free(cache->layers);
    std::free(cache);
}

extern "C" hma_status_t hma_error_flags(const hma_cache_t *cache, uint32_t *host_out, void *stream)
{
    if (!cache || !host_out) return HMA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    HMA_CUDA_OK(cudaMemcpyAsync(host_out, cache->flags, sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
    HMA_CUDA_OK(cudaMemsetAsync(cache->flags, 0, sizeof(uint32_t), s));
    HMA_CUDA_OK(cudaStreamSynchronize(s));
    return HMA_OK;
}

extern "C" const char *hma_status_string(int32_t status)
{
    switch (status) {
        case HMA_OK: return "ok";
        case HMA_ERR_INVALID_ARG: return "invalid argument";
        case HMA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case HMA_ERR_ALIGNMENT: return "misaligned pointer";
        case HMA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case HMA_ERR_CUDA: return "CUDA runtime error";
        case HMA_ERR_STATIC_LIMIT: return "request exceeds the built-in scratch array of hma_decode_attention_static";
        default: return "unknown status";
    }
}

extern "C" const char *hma_last_cuda_error(void) { return cudaGetErrorString(hma::g_last_error); }

extern "C" int64_t hma_launch_count(void) { return (int64_t)hma::g_launches.load(std::memory_order_relaxed); }
