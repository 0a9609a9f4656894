// Plain decode attention: one CTA per (sequence, kv head), CUDA cores only, every element decoded to
// BF16 first and widened to fp32 (the elementwise reconstruction of section 3.3).  Slow by design;
// it is the on-device cross-check of the fast kernel and shares no device code with it beyond the
// record layout and the element decode.
#include "hma_common.cuh"

namespace hma {

constexpr int kSimpleWarps = 8;

template <int G>
__global__ void __launch_bounds__(kSimpleWarps * 32) attn_simple_kernel(CacheView cv, const uint16_t *__restrict__ q,
                                                                        void *__restrict__ out, int out_dtype,
                                                                        const int32_t *__restrict__ block_table,
                                                                        int max_pages, const int32_t *__restrict__ ctx,
                                                                        float sm_scale)
{
    __shared__ float sq[G][kHeadDim];
    __shared__ float sm[kSimpleWarps][G], sl[kSimpleWarps][G];
    __shared__ float so[kSimpleWarps][G][kHeadDim];
    const int b = blockIdx.x, g = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = ctx[b];
    for (int i = threadIdx.x; i < G * kHeadDim; i += blockDim.x)
        sq[i / kHeadDim][i % kHeadDim] = bf16_bits_to_float(q[((int64_t)b * cv.num_q_heads + g * G) * kHeadDim + i]);
    __syncthreads();
    float m[G], l[G], o[G][4];
#pragma unroll
    for (int h = 0; h < G; ++h) { m[h] = -INFINITY; l[h] = 0.f; o[h][0] = o[h][1] = o[h][2] = o[h][3] = 0.f; }
    const int rb = record_bytes(cv.format);
    for (int t = warp; t < T; t += kSimpleWarps) {
        const int32_t pid = block_table[(int64_t)b * max_pages + t / kPageTokens];
        if (pid < 0 || pid >= cv.num_pages) {
            if (lane == 0) atomicOr(cv.flags, HMA_FLAG_BAD_PAGE_ATTENTION);
            continue;
        }
        const uint8_t *rec = cv.layer + ((int64_t)pid * cv.num_kv_heads + g) * (int64_t)rb;
        const int tok = t % kPageTokens;
        float kf[4], vf[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int ch = lane * 4 + k;
            if (cv.format == HMA_KV_BFP8) {
                kf[k] = bf16_bits_to_float(bfp8_to_bf16_bits(rec[bfp8_k_exp_off(tok, ch >> 4)], rec[bfp8_k_el_off(tok, ch)]));
                vf[k] = bf16_bits_to_float(bfp8_to_bf16_bits(rec[bfp8_v_exp_off(tok, ch >> 4)], rec[bfp8_v_el_off(tok, ch)]));
            } else {
                kf[k] = bf16_bits_to_float(*reinterpret_cast<const uint16_t *>(rec + bf16_k_el_off(tok, ch)));
                vf[k] = bf16_bits_to_float(*reinterpret_cast<const uint16_t *>(rec + bf16_v_el_off(tok, ch)));
            }
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < 4; ++k) s = fmaf(sq[h][key_channel_of_query(lane * 4 + k, cv.key_layout)], kf[k], s);
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
            s *= sm_scale;
            const float mn = fmaxf(m[h], s);
            const float a = __expf(m[h] - mn), p = __expf(s - mn);
            l[h] = l[h] * a + p;
#pragma unroll
            for (int k = 0; k < 4; ++k) o[h][k] = o[h][k] * a + p * vf[k];
            m[h] = mn;
        }
    }
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (lane == 0) { sm[warp][h] = m[h]; sl[warp][h] = l[h]; }
#pragma unroll
        for (int k = 0; k < 4; ++k) so[warp][h][lane * 4 + k] = o[h][k];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < G * kHeadDim; i += blockDim.x) {
        const int h = i / kHeadDim, d = i % kHeadDim;
        float M = -INFINITY;
        for (int w = 0; w < kSimpleWarps; ++w) M = fmaxf(M, sm[w][h]);
        float num = 0.f, den = 0.f;
        for (int w = 0; w < kSimpleWarps; ++w) {
            if (sm[w][h] == -INFINITY) continue;
            const float a = __expf(sm[w][h] - M);
            num += a * so[w][h][d];
            den += a * sl[w][h];
        }
        const float r = den > 0.f ? num / den : 0.f;
        const int64_t idx = ((int64_t)b * cv.num_q_heads + g * G + h) * kHeadDim + d;
        if (out_dtype == HMA_OUT_F32) reinterpret_cast<float *>(out)[idx] = r;
        else {
            // fp32 -> BF16, round to nearest even
            uint32_t u = __float_as_uint(r);
            u += 0x7FFFu + ((u >> 16) & 1u);
            reinterpret_cast<uint16_t *>(out)[idx] = (uint16_t)(u >> 16);
        }
    }
}

}  // namespace hma

extern "C" hma_status_t hma_decode_attention_simple(const hma_cache_t *cache, int32_t layer, const void *q, void *out,
                                                    int32_t out_dtype, const int32_t *block_table, int32_t max_pages_per_seq,
                                                    const int32_t *context_lens, int32_t batch, float sm_scale, void *stream)
{
    if (!cache || layer < 0 || layer >= cache->desc.num_layers || batch < 0 || max_pages_per_seq < 0) return HMA_ERR_INVALID_ARG;
    if (!hma::on_cache_device(cache)) return HMA_ERR_INVALID_ARG;
    if (out_dtype != HMA_OUT_BF16 && out_dtype != HMA_OUT_F32) return HMA_ERR_INVALID_ARG;
    if (batch == 0) return HMA_OK;
    if (!q || !out || !block_table || !context_lens) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15u) || ((uintptr_t)out & 15u)) return HMA_ERR_ALIGNMENT;
    hma::CacheView cv{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                      cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    dim3 grid((unsigned)batch, (unsigned)cache->desc.num_kv_heads);
    cudaStream_t s = (cudaStream_t)stream;
    const int G = cache->desc.num_q_heads / cache->desc.num_kv_heads;
#define HMA_SIMPLE_CASE(GG)                                                                                            \
    case GG:                                                                                                           \
        hma::attn_simple_kernel<GG><<<grid, hma::kSimpleWarps * 32, 0, s>>>(cv, (const uint16_t *)q, out, out_dtype,   \
                                                                            block_table, max_pages_per_seq,            \
                                                                            context_lens, sm_scale);                   \
        break;
    switch (G) {
        HMA_SIMPLE_CASE(1) HMA_SIMPLE_CASE(2) HMA_SIMPLE_CASE(3) HMA_SIMPLE_CASE(4)
        HMA_SIMPLE_CASE(5) HMA_SIMPLE_CASE(6) HMA_SIMPLE_CASE(7) HMA_SIMPLE_CASE(8)
        default: return HMA_ERR_UNSUPPORTED_SHAPE;
    }
#undef HMA_SIMPLE_CASE
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}
