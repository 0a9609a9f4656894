// Fused BFP8 paged decode attention for sm_100a (section 3.3: BFP8 pages stay raw in HBM and are
// rebuilt inside the attention kernel).
//
// Shape of the kernel
//   * persistent grid, one CTA per SM.  All (sequence, kv head, page) records of the batch form one
//     linear work list that is cut into equal contiguous ranges, one per CTA (no tail effect, any
//     mix of context lengths).  A CTA that holds only part of a (sequence, kv head) segment emits a
//     partial (max, sum, 128-vector) per q head; a second small kernel merges partials in fixed order.
//   * one producer warp streams 4352-byte page records HBM -> shared memory with 1-D bulk async
//     copies (cp.async.bulk + mbarrier transaction counts) through a deep ring; eight consumer warps
//     each own whole records.
//   * unpack is two integer instructions per pair of elements (byte permute + mask): the element
//     byte s<<7|m becomes the FP16 bit pattern s<<15|m, which *is* the number +-m * 2^-24 (an FP16
//     subnormal), so mantissas enter mma.sync.m16n8k16 exactly.  The shared block exponent never
//     touches the elements: for Q.K^T one MMA k-step is one 16-channel block of each token, so
//     2^E scales the fp32 partial product; for P.V it is folded into the softmax weights, relative
//     to a running per-block reference exponent that is handled like the running softmax maximum.
//   * the softmax weights go to the second MMA as FP16 (11 significant bits), not BF16.
#include <cuda_fp16.h>

#include "hma_common.cuh"

namespace hma {

// 15 consumer warps + 1 producer warp = 16 warps, four per SM sub-partition: each sub-partition has 16384
// registers, so a 17th warp would cap every thread at 96 registers instead of 128.
constexpr int kConsumerWarps = 15;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kStages = 45;                       // ring depth
// A ring slot must be used by the same consumer warp every time round (within a segment): a warp that ran two
// laps ahead of the slot's previous owner would see the slot's older completed phase and read stale bytes.
static_assert(kStages % kConsumerWarps == 0, "ring depth must be a multiple of one round of the consumer warps");
constexpr int kTileFloats = 8 * kHeadDim + 16;    // partial tile: o[8][128], m[8], l[8]
constexpr int kSlots = 4;                         // states held in shared memory during the merge
constexpr int kSlotFloats = 1024 + 16;            // one warp's state: 32 accumulators per lane, then m, l per head pair
static_assert(kSlots * kSlotFloats * 4 >= kConsumerWarps * 768, "per-warp scratch tables live inside the merge slots");
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr int kMaxBatch = 768;
constexpr int kMaxCtas = 1024;

struct AttnArgs {
    CacheView cv;
    const uint16_t *q;
    void *out;
    int out_dtype;
    const int32_t *block_table;
    int max_pages;
    const int32_t *ctx;
    int batch;
    float sm_scale;
    int32_t *cum;        // workspace: pages before each sequence, batch+1 entries
    float *tiles;        // workspace: partial tiles
};

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (or when another thread of the CTA already gave up),
// raises the CTA's abort word and the device flag, and returns false.  Nothing spins forever.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_word, uint32_t *flags)
{
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u && *abort_word) return false;
    }
    *abort_word = 1;
    atomicOr(flags, HMA_FLAG_WAIT_TIMEOUT);
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void sts64(uint32_t addr, uint32_t x, uint32_t y)
{
    asm volatile("st.shared.v2.u32 [%0], {%1,%2};" ::"r"(addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w)
{
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, const float (&c)[4])
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
        : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c[0]), "f"(c[1]), "f"(c[2]), "f"(c[3]));
}
__device__ __forceinline__ void mma_f16_acc(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a)
{
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); }
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi)
{
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&h);
}
__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b)
{
    __half2 r = __hmul2(*reinterpret_cast<__half2 *>(&a), *reinterpret_cast<__half2 *>(&b));
    return *reinterpret_cast<uint32_t *>(&r);
}
// 2^e as fp32 from an exponent field value in [0, 254] (0 gives 0.0)
__device__ __forceinline__ float pow2_field(int field) { return __uint_as_float((uint32_t)field << 23); }
__device__ __forceinline__ uint16_t f32_to_bf16_rne(float r)
{
    uint32_t u = __float_as_uint(r);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0;
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

// pages of sequence b (context clamped to what the block table can address)
__device__ __forceinline__ int pages_of(const AttnArgs &a, int b)
{
    int T = a.ctx[b];
    T = max(0, min(T, a.max_pages * kPageTokens));
    return (T + kPageTokens - 1) / kPageTokens;
}

// ---------------------------------------------------------------- main kernel
extern __shared__ __align__(128) uint8_t smem_raw[];

// kMode 0: attention.  1: stream the records through the ring, no arithmetic (bandwidth probe).
// 2: the arithmetic of every record on whatever the ring holds, nothing loaded or written (issue-rate probe).
template <int kMode>
__global__ void __launch_bounds__(kThreads, 1) attn_bfp8_kernel(const AttnArgs a)
{
    // shared memory carve-up
    uint8_t *ring = smem_raw;                                                   // kStages x 4352
    float *comb = reinterpret_cast<float *>(ring + kStages * kBfp8Record);       // merge slots / per-warp scratch
    uint64_t *bars = reinterpret_cast<uint64_t *>(comb + kSlots * kSlotFloats);   // full[kStages], empty[kStages]
    int *stage_ok = reinterpret_cast<int *>(bars + 2 * kStages);                 // [kStages]
    int *misc = stage_ok + kStages;                                              // [0] abort word, [1..] scan scratch
    int *cum = misc + 16 + kThreads;                                             // [batch + 1]
    volatile int *abort_word = misc;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hkv = a.cv.num_kv_heads, G = a.cv.num_q_heads / Hkv, B = a.batch;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + kStages);

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, 1);
        }
        misc[0] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // exclusive prefix of pages per sequence
    {
        const int per = (B + kThreads - 1) / kThreads;
        const int b0 = min(B, tid * per), b1 = min(B, b0 + per);
        int sum = 0;
        for (int b = b0; b < b1; ++b) sum += pages_of(a, b);
        misc[16 + tid] = sum;
        __syncthreads();
        if (tid == 0) {
            int run = 0;
            for (int i = 0; i < kThreads; ++i) { int v = misc[16 + i]; misc[16 + i] = run; run += v; }
            cum[B] = run;
        }
        __syncthreads();
        int run = misc[16 + tid];
        for (int b = b0; b < b1; ++b) { cum[b] = run; run += pages_of(a, b); }
        __syncthreads();
    }
    if (blockIdx.x == 0)
        for (int b = tid; b <= B; b += kThreads) a.cum[b] = cum[b];

    const int64_t W = (int64_t)Hkv * cum[B];
    const int64_t N = gridDim.x;
    const int64_t w0 = (int64_t)blockIdx.x * W / N, w1 = (int64_t)(blockIdx.x + 1) * W / N;
    if (w0 >= w1) return;

    // locate the segment (b, g) that holds w0
    int b_cur, g_cur;
    {
        int lo = 0, hi = B - 1;
        while (lo < hi) {   // largest b with Hkv*cum[b] <= w0
            int mid = (lo + hi + 1) >> 1;
            if ((int64_t)Hkv * cum[mid] <= w0) lo = mid; else hi = mid - 1;
        }
        while (cum[lo + 1] == cum[lo]) ++lo;   // cannot run off: w0 < W
        b_cur = lo;
        const int np = cum[lo + 1] - cum[lo];
        g_cur = (int)((w0 - (int64_t)Hkv * cum[lo]) / np);
    }

    if (warp == kConsumerWarps) {
        // ------------------------------------------------------------ producer warp
        // Every lane owns one record of a chunk of up to 32 consecutive pages of a segment: it waits for
        // its ring slot, then issues its own bulk copy, so 32 copies are set up in parallel.  The block
        // table entries of the next chunk are fetched before the current chunk waits.
        uint64_t policy;
        asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
        constexpr int rb = kBfp8Record;
        int b = b_cur, g = g_cur;
        int np = cum[b + 1] - cum[b];
        int p = (int)(w0 - ((int64_t)Hkv * cum[b] + (int64_t)g * np));
        const int R = (int)(w1 - w0);
        int r = 0;
        int chunk = min(min(32, np - p), R - r);
        int32_t pid = lane < chunk ? a.block_table[(int64_t)b * a.max_pages + p + lane] : 0;
        bool alive = true;
        if (kMode == 2) return;              // arithmetic-only diagnostic: nothing is loaded
        while (r < R) {
            const int c_chunk = chunk, c_g = g, c_r = r;
            const int32_t c_pid = pid;
            // advance to the next chunk and prefetch its page ids
            r += chunk;
            p += chunk;
            if (p == np) {
                p = 0;
                if (++g == Hkv) {
                    g = 0;
                    do { ++b; } while (b < B && cum[b + 1] == cum[b]);
                    if (b < B) np = cum[b + 1] - cum[b];
                }
            }
            if (r < R) {
                chunk = min(min(32, np - p), R - r);
                pid = lane < chunk ? a.block_table[(int64_t)b * a.max_pages + p + lane] : 0;
            }
            if (lane < c_chunk) {
                const int rr = c_r + lane;
                const int s = rr % kStages;
                if (rr >= kStages) alive = mbar_wait(empty0 + 8 * s, (uint32_t)((rr / kStages) - 1) & 1u, abort_word, a.cv.flags);
                if (alive) {
                    if (c_pid >= 0 && c_pid < a.cv.num_pages) {
                        stage_ok[s] = 1;
                        mbar_arrive_expect_tx(full0 + 8 * s, rb);
                        bulk_load(smem_u32(ring + s * rb), a.cv.layer + ((int64_t)c_pid * Hkv + c_g) * rb, rb, full0 + 8 * s, policy);
                    } else {
                        stage_ok[s] = 0;
                        atomicOr(a.cv.flags, HMA_FLAG_BAD_PAGE_ATTENTION);
                        mbar_arrive(full0 + 8 * s);
                    }
                }
            }
            if (!__all_sync(0xFFFFFFFFu, alive)) {
                // a wait ran out: give the copies already issued a bounded chance to land, then leave
                const int issued = c_r;   // records below c_r were all issued
                for (int s = lane; s < kStages; s += 32) {
                    int last = -1;
                    for (int q = s; q < issued; q += kStages) last = q;
                    if (last < 0) continue;
                    for (uint32_t it = 0; it < kSpinLimit && !mbar_try_wait(full0 + 8 * s, (uint32_t)(last / kStages) & 1u); ++it) {}
                }
                return;
            }
        }
        return;
    }

    // ---------------------------------------------------------------- consumer warps
    // One record (16 tokens of one kv head) per warp iteration; a ring slot belongs to the same warp on every lap.
    const int gq = lane >> 2, t4 = lane & 3;
    const float kLog2e = 1.4426950408889634f;
    // per-warp scratch inside the merge area (idle until the segment ends):
    // fp32 Q.K^T scales 2^(E-127) of every (token, block) and FP16 P.V scales of every (token pair, block)
    const uint32_t scrK = smem_u32(comb) + warp * 768;     // 512 B
    const uint32_t scrV = scrK + 512;                      // 256 B
    int64_t w = w0;
    int b = b_cur, g = g_cur;
    bool alive = true;
    while (w < w1 && alive) {
        const int np = cum[b + 1] - cum[b];
        const int64_t seg0 = (int64_t)Hkv * cum[b] + (int64_t)g * np, seg1 = seg0 + np;
        const int64_t lo = max(seg0, w0), hi = min(seg1, w1);
        const int T = min(a.ctx[b], a.max_pages * kPageTokens);
        const int rbase = (int)(lo - w0);            // CTA-local index of the segment's first record here
        const int rend = (int)(hi - w0);
        const int page0 = (int)(lo - seg0);          // page of the sequence that record rbase holds
        const int tail = T - (np - 1) * kPageTokens; // valid tokens of the sequence's last page, 1..16

        // ---- Q fragments of this (sequence, kv head): FP16, one power-of-two scale per head ----
        uint32_t qf[8][2];
        float cs0, cs1;   // score multipliers of heads 2*t4, 2*t4+1
        {
            float f[8][4];
            float amax = 0.f;
            const bool hv = gq < G && kMode == 0;      // the probes have no Q: nothing is read through a.q
            const uint16_t *qp = a.q + ((int64_t)b * a.cv.num_q_heads + (int64_t)g * G + (hv ? gq : 0)) * kHeadDim + 4 * t4;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                uint2 v = hv ? *reinterpret_cast<const uint2 *>(qp + 16 * j) : make_uint2(0u, 0u);
                f[j][0] = __uint_as_float(v.x << 16);
                f[j][1] = __uint_as_float(v.x & 0xFFFF0000u);
                f[j][2] = __uint_as_float(v.y << 16);
                f[j][3] = __uint_as_float(v.y & 0xFFFF0000u);
#pragma unroll
                for (int k = 0; k < 4; ++k) amax = fmaxf(amax, fabsf(f[j][k]));
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
            int shift = 0;
            if (amax > 0.f && amax < INFINITY) shift = 14 - ((int)((__float_as_uint(amax) >> 23) & 0xFF) - 127);
            shift = max(-120, min(120, shift));
            const float up = pow2_field(127 + shift), down = pow2_field(127 - shift);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                qf[j][0] = pack_half2(f[j][0] * up, f[j][1] * up);
                qf[j][1] = pack_half2(f[j][2] * up, f[j][3] * up);
            }
            // mantissas enter as m * 2^-24 and exponents as 2^(E-127) while values are m * 2^(E-133): 2^18 is owed
            const float cs = a.sm_scale * kLog2e * down * 262144.f;
            cs0 = __shfl_sync(0xFFFFFFFFu, cs, (2 * t4) * 4);
            cs1 = __shfl_sync(0xFFFFFFFFu, cs, (2 * t4 + 1) * 4);
        }

        float m0 = -INFINITY, m1 = -INFINITY;          // running maxima (log2 domain) of heads 2*t4, 2*t4+1
        float lacc[4] = {0.f, 0.f, 0.f, 0.f};          // running sums, via an all-ones MMA
        float o[8][4];
#pragma unroll
        for (int j = 0; j < 8; ++j) o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f;
        int Rmine = 0;                                  // reference exponent of V channel block (lane & 7)

        int r = rbase + warp;
        int stage = r % kStages;
        uint32_t par = (uint32_t)(r / kStages) & 1u;
        int page = page0 + warp;
        for (; r < rend; r += kConsumerWarps, page += kConsumerWarps) {
            if (kMode < 2) {
                alive = mbar_wait(full0 + 8 * stage, par, abort_word, a.cv.flags);
                if (!alive) break;
            }
            const uint32_t sp = smem_u32(ring) + stage * kBfp8Record;
            const uint32_t my_empty = empty0 + 8 * stage;
            const bool ok = kMode == 2 || stage_ok[stage] != 0;
            stage += kConsumerWarps;
            if (stage >= kStages) { stage -= kStages; par ^= 1u; }
            if (kMode == 1 || !ok) {
                __syncwarp();
                if (lane == 0) mbar_arrive(my_empty);
                continue;
            }
            const int nvalid = page == np - 1 ? tail : kPageTokens;

            // ---- exponents: fp32 scales for Q.K^T, reference-exponent check and FP16 scales for P.V ----
            {
                const uint32_t kw = lds32(sp + lane * 4);
                uint32_t vw = lds32(sp + kBfp8Half + lane * 4);
                if (nvalid < kPageTokens) {
                    // exponent bytes of masked tokens count as 0: they neither raise the reference exponent
                    // nor produce non-finite weights
                    uint32_t keep = 0;
                    const int tt = lane >> 3;
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        if (2 * tt + (k & 1) + 8 * (k >> 1) < nvalid) keep |= 0xFFu << (8 * k);
                    vw &= keep;
                }
                sts128(scrK + lane * 16, (kw << 23) & 0x7F800000u, (kw << 15) & 0x7F800000u, (kw << 7) & 0x7F800000u,
                       (kw >> 1) & 0x7F800000u);
                const uint32_t mx2 = __vmaxu2((vw >> 8) & 0x00FF00FFu, vw & 0x00FF00FFu);
                int emax = (int)max(mx2 & 0xFFFFu, mx2 >> 16);
                if (__any_sync(0xFFFFFFFFu, emax > Rmine)) {
                    // a V block exponent above the reference: raise it and rescale that block's accumulators
                    emax = max(emax, __shfl_xor_sync(0xFFFFFFFFu, emax, 8));
                    emax = max(emax, __shfl_xor_sync(0xFFFFFFFFu, emax, 16));
                    const int Rnew = max(Rmine, emax);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int dlt = __shfl_sync(0xFFFFFFFFu, Rmine, j) - __shfl_sync(0xFFFFFFFFu, Rnew, j);   // <= 0
                        const float fr = dlt < -126 ? 0.f : pow2_field(127 + dlt);
                        o[j][0] *= fr; o[j][1] *= fr; o[j][2] *= fr; o[j][3] *= fr;
                    }
                    Rmine = Rnew;
                }
                // FP16 scale 2^(E - R + 15) of every (token pair, block): exponent field max(E - R + 30, 0)
                const uint32_t kmine = ((uint32_t)(30 - Rmine) & 0xFFFFu) * 0x00010001u;
                sts64(scrV + lane * 8, __viaddmax_s16x2_relu(prmt(vw, 0u, 0x4140u), kmine, 0u) << 10,
                      __viaddmax_s16x2_relu(prmt(vw, 0u, 0x4342u), kmine, 0u) << 10);
            }
            uint4 km[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) km[c] = lds128(sp + 128 + c * 512 + lane * 16);
            __syncwarp();

            // ================= Q.K^T =================
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
            {
                float ks[16];      // 2^(E-127): token gq blocks 0..7, token gq+8 blocks 0..7
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint4 v = lds128(scrK + gq * 64 + c * 16);
                    ks[4 * c] = __uint_as_float(v.x); ks[4 * c + 1] = __uint_as_float(v.y);
                    ks[4 * c + 2] = __uint_as_float(v.z); ks[4 * c + 3] = __uint_as_float(v.w);
                }
                const float zero4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 &klo = km[(j >> 2) * 2], &khi = km[(j >> 2) * 2 + 1];
                    const uint32_t wl = (j & 3) == 0 ? klo.x : (j & 3) == 1 ? klo.y : (j & 3) == 2 ? klo.z : klo.w;
                    const uint32_t wh = (j & 3) == 0 ? khi.x : (j & 3) == 1 ? khi.y : (j & 3) == 2 ? khi.z : khi.w;
                    uint32_t af[4];
                    af[0] = prmt(wl, 0u, 0x1100u) & 0x807F807Fu;
                    af[1] = prmt(wh, 0u, 0x1100u) & 0x807F807Fu;
                    af[2] = prmt(wl, 0u, 0x3322u) & 0x807F807Fu;
                    af[3] = prmt(wh, 0u, 0x3322u) & 0x807F807Fu;
                    float d[4];
                    mma_f16(d, af, qf[j][0], qf[j][1], zero4);
                    sc[0] = fmaf(d[0], ks[j], sc[0]);
                    sc[1] = fmaf(d[1], ks[j], sc[1]);
                    sc[2] = fmaf(d[2], ks[8 + j], sc[2]);
                    sc[3] = fmaf(d[3], ks[8 + j], sc[3]);
                }
            }
            // the V element words go to registers now, so that the ring slot can be refilled during softmax and P.V
            uint4 vm[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) vm[c] = lds128(sp + kBfp8Half + 128 + c * 512 + lane * 16);
            __syncwarp();
            if (lane == 0 && kMode < 2) mbar_arrive(my_empty);
            float s0 = sc[0] * cs0, s1 = sc[1] * cs1, s2 = sc[2] * cs0, s3 = sc[3] * cs1;
            if (nvalid < kPageTokens) {
                if (gq >= nvalid) { s0 = -INFINITY; s1 = -INFINITY; }
                if (gq + 8 >= nvalid) { s2 = -INFINITY; s3 = -INFINITY; }
            }
            // ================= online softmax (log2 domain) =================
            // The warp-wide maximum is only formed when some score exceeds the running maximum.
            if (__any_sync(0xFFFFFFFFu, fmaxf(s0, s2) > m0 || fmaxf(s1, s3) > m1)) {
                float mx0 = fmaxf(s0, s2), mx1 = fmaxf(s1, s3);
#pragma unroll
                for (int d = 4; d <= 16; d <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, d));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, d));
                }
                const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                const float a0 = mn0 == -INFINITY ? 1.f : ex2f(m0 - mn0), a1 = mn1 == -INFINITY ? 1.f : ex2f(m1 - mn1);
                m0 = mn0;
                m1 = mn1;
                lacc[0] *= a0; lacc[1] *= a1; lacc[2] *= a0; lacc[3] *= a1;
#pragma unroll
                for (int j = 0; j < 8; ++j) { o[j][0] *= a0; o[j][1] *= a1; o[j][2] *= a0; o[j][3] *= a1; }
            }
            // weights as FP16, transposed from (token, head) accumulator layout to the B-operand layout
            const uint32_t pb0 = movmatrix_trans(pack_half2(ex2f(s0 - m0), ex2f(s1 - m1)));   // tokens 2*t4, 2*t4+1 of head gq
            const uint32_t pb1 = movmatrix_trans(pack_half2(ex2f(s2 - m0), ex2f(s3 - m1)));   // tokens 2*t4+8, 2*t4+9
            {
                const uint32_t ones[4] = {0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u};
                mma_f16_acc(lacc, ones, pb0, pb1);
            }
            // ================= P.V =================
            {
                uint4 vs[4];           // (f01, f89) of blocks 2c, 2c+1
#pragma unroll
                for (int c = 0; c < 4; ++c) vs[c] = lds128(scrV + t4 * 64 + c * 16);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint4 &vv = vm[j >> 1];
                    const uint32_t wl = (j & 1) ? vv.z : vv.x, wh = (j & 1) ? vv.w : vv.y;   // channels gq, gq+8 of block j
                    uint32_t af[4];
                    af[0] = prmt(wl, 0u, 0x1100u) & 0x807F807Fu;
                    af[1] = prmt(wh, 0u, 0x1100u) & 0x807F807Fu;
                    af[2] = prmt(wl, 0u, 0x3322u) & 0x807F807Fu;
                    af[3] = prmt(wh, 0u, 0x3322u) & 0x807F807Fu;
                    const uint32_t f01 = (j & 1) ? vs[j >> 1].z : vs[j >> 1].x, f89 = (j & 1) ? vs[j >> 1].w : vs[j >> 1].y;
                    mma_f16_acc(o[j], af, hmul2_u32(pb0, f01), hmul2_u32(pb1, f89));
                }
            }
            __syncwarp();      // every lane is done with the scratch tables
        }

        // ---- merge the warps' states of this segment: pairwise tree, at most kSlots states in shared memory ----
        consumer_bar_sync();                           // the scratch tables (same memory as the slots) are idle now
        if (kMode != 1 && alive) {
            // to true units: accumulators hold sum p * m * 2^(E - R - 9); values are m * 2^(E-133)
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float vsc = pow2_field(min(__shfl_sync(0xFFFFFFFFu, Rmine, j) + 3, 254));
                o[j][0] *= vsc; o[j][1] *= vsc; o[j][2] *= vsc; o[j][3] *= vsc;
            }
        }
        float l0 = lacc[0], l1 = lacc[1];
#pragma unroll 1
        for (int n = kConsumerWarps; n > 1; n = (n + 1) / 2) {
            const int half = (n + 1) / 2;              // warps [half, n) hand their state to warps [0, n - half)
#pragma unroll 1
            for (int base = 0; base < n - half; base += kSlots) {
                const int wr = warp - half - base;     // slot this warp writes in this round, if in [0, kSlots)
                if (kMode != 1 && warp >= half && warp < n && wr >= 0 && wr < kSlots) {
                    float *slot = comb + wr * kSlotFloats;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
#pragma unroll
                        for (int k = 0; k < 4; ++k) slot[(j * 4 + k) * 32 + lane] = o[j][k];
                    if (gq == 0) {
                        slot[1024 + t4 * 4 + 0] = m0; slot[1024 + t4 * 4 + 1] = m1;
                        slot[1024 + t4 * 4 + 2] = l0; slot[1024 + t4 * 4 + 3] = l1;
                    }
                }
                consumer_bar_sync();
                const int rd = warp - base;            // slot this warp reads in this round, if in [0, kSlots)
                if (kMode != 1 && warp < n - half && rd >= 0 && rd < kSlots) {
                    const float *slot = comb + rd * kSlotFloats;
                    const float pm0 = slot[1024 + t4 * 4 + 0], pm1 = slot[1024 + t4 * 4 + 1];
                    const float pl0 = slot[1024 + t4 * 4 + 2], pl1 = slot[1024 + t4 * 4 + 3];
                    const float M0 = fmaxf(m0, pm0), M1 = fmaxf(m1, pm1);
                    const float a0 = m0 == -INFINITY ? 0.f : ex2f(m0 - M0), a1 = m1 == -INFINITY ? 0.f : ex2f(m1 - M1);
                    const float c0 = pm0 == -INFINITY ? 0.f : ex2f(pm0 - M0), c1 = pm1 == -INFINITY ? 0.f : ex2f(pm1 - M1);
                    l0 = l0 * a0 + pl0 * c0;
                    l1 = l1 * a1 + pl1 * c1;
                    m0 = M0;
                    m1 = M1;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        o[j][0] = o[j][0] * a0 + slot[(j * 4 + 0) * 32 + lane] * c0;
                        o[j][1] = o[j][1] * a1 + slot[(j * 4 + 1) * 32 + lane] * c1;
                        o[j][2] = o[j][2] * a0 + slot[(j * 4 + 2) * 32 + lane] * c0;
                        o[j][3] = o[j][3] * a1 + slot[(j * 4 + 3) * 32 + lane] * c1;
                    }
                }
                consumer_bar_sync();
            }
        }
        if (warp == 0 && (kMode == 0 || (kMode == 2 && a.batch < 0)) && alive) {   // the issue-rate probe never stores, but keeps its arithmetic live
            const bool whole = lo == seg0 && hi == seg1;
            const int h0 = 2 * t4, h1 = 2 * t4 + 1;
            if (whole) {
                const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
                const int64_t ob = ((int64_t)b * a.cv.num_q_heads + (int64_t)g * G) * kHeadDim;
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int h = (k & 1) ? h1 : h0, c = 16 * j + gq + 8 * (k >> 1);
                        if (h < G) {
                            const float res = o[j][k] * ((k & 1) ? i1 : i0);
                            if (a.out_dtype == HMA_OUT_F32) reinterpret_cast<float *>(a.out)[ob + h * kHeadDim + c] = res;
                            else reinterpret_cast<uint16_t *>(a.out)[ob + h * kHeadDim + c] = f32_to_bf16_rne(res);
                        }
                    }
            } else {
                float *tp = a.tiles + ((int64_t)blockIdx.x + ((int64_t)b * Hkv + g)) * kTileFloats;
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int k = 0; k < 4; ++k) tp[((k & 1) ? h1 : h0) * kHeadDim + 16 * j + gq + 8 * (k >> 1)] = o[j][k];
                if (gq == 0) {
                    tp[8 * kHeadDim + h0] = m0; tp[8 * kHeadDim + h1] = m1;
                    tp[8 * kHeadDim + 8 + h0] = l0; tp[8 * kHeadDim + 8 + h1] = l1;
                }
            }
        }

        w = hi;
        if (++g == Hkv) {
            g = 0;
            do { ++b; } while (b < B && cum[b + 1] == cum[b]);
        }
    }
}

// ---------------------------------------------------------------- cross-split reduction
// One CTA per (sequence, kv head).  Segments that one CTA of the main kernel covered entirely were
// already written there; the rest are merged here from their partial tiles, in CTA order.
__global__ void __launch_bounds__(128) attn_reduce_kernel(const AttnArgs a, int n_ctas)
{
    const int Hkv = a.cv.num_kv_heads, G = a.cv.num_q_heads / Hkv;
    const int b = blockIdx.x / Hkv, g = blockIdx.x % Hkv, c = threadIdx.x;
    const int np = a.cum[b + 1] - a.cum[b];
    const int64_t W = (int64_t)Hkv * a.cum[a.batch], N = n_ctas;
    const int64_t obase = ((int64_t)b * a.cv.num_q_heads + (int64_t)g * G) * kHeadDim + c;
    if (np == 0) {
        for (int h = 0; h < G; ++h) {
            if (a.out_dtype == HMA_OUT_F32) reinterpret_cast<float *>(a.out)[obase + h * kHeadDim] = 0.f;
            else reinterpret_cast<uint16_t *>(a.out)[obase + h * kHeadDim] = 0;
        }
        return;
    }
    const int64_t ws = (int64_t)Hkv * a.cum[b] + (int64_t)g * np, we = ws + np;
    const int64_t i0 = ((ws + 1) * N - 1) / W, i1 = (we * N - 1) / W;     // first and last CTA touching the segment
    if (i0 == i1) return;
    for (int h = 0; h < G; ++h) {
        float M = -INFINITY;
        for (int64_t i = i0; i <= i1; ++i) {
            if (i * W / N >= (i + 1) * W / N) continue;   // CTA with an empty range wrote nothing
            M = fmaxf(M, a.tiles[(i + blockIdx.x) * kTileFloats + 8 * kHeadDim + h]);
        }
        float num = 0.f, den = 0.f;
        for (int64_t i = i0; i <= i1; ++i) {
            if (i * W / N >= (i + 1) * W / N) continue;
            const float *tp = a.tiles + (i + blockIdx.x) * kTileFloats;
            const float mw = tp[8 * kHeadDim + h];
            const float wgt = mw == -INFINITY ? 0.f : ex2f(mw - M);
            num = fmaf(wgt, tp[h * kHeadDim + c], num);
            den = fmaf(wgt, tp[8 * kHeadDim + 8 + h], den);
        }
        const float res = den > 0.f ? num / den : 0.f;
        if (a.out_dtype == HMA_OUT_F32) reinterpret_cast<float *>(a.out)[obase + h * kHeadDim] = res;
        else reinterpret_cast<uint16_t *>(a.out)[obase + h * kHeadDim] = f32_to_bf16_rne(res);
    }
}

static size_t attn_smem_bytes(int batch)
{
    return (size_t)kStages * kBfp8Record + (size_t)kSlots * kSlotFloats * 4 + 2 * kStages * 8 + kStages * 4 +
           (16 + kThreads) * 4 + ((size_t)batch + 1) * 4;
}

static size_t cum_bytes(int batch) { return (((size_t)batch + 1) * 4 + 255) & ~(size_t)255; }

}  // namespace hma

extern "C" size_t hma_decode_attention_workspace_bytes(const hma_cache_desc_t *desc, int32_t batch)
{
    if (!desc || batch < 0 || desc->num_kv_heads <= 0) return 0;
    return hma::cum_bytes(batch) + ((size_t)hma::kMaxCtas + (size_t)batch * desc->num_kv_heads) * hma::kTileFloats * 4;
}

static hma_status_t launch_attention(const hma_cache_t *cache, int32_t layer, const void *q, void *out, int32_t out_dtype,
                                     const int32_t *block_table, int32_t max_pages_per_seq, const int32_t *context_lens,
                                     int32_t batch, float sm_scale, void *workspace, size_t workspace_bytes, void *stream,
                                     int probe)
{
    if (!cache || layer < 0 || layer >= cache->desc.num_layers || batch < 0 || max_pages_per_seq < 0) return HMA_ERR_INVALID_ARG;
    if (out_dtype != HMA_OUT_BF16 && out_dtype != HMA_OUT_F32) return HMA_ERR_INVALID_ARG;
    if (batch == 0) return HMA_OK;
    if (!block_table || !context_lens || !workspace || (!probe && (!q || !out))) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15u) || ((uintptr_t)out & 15u) || ((uintptr_t)workspace & 255u)) return HMA_ERR_ALIGNMENT;
    if (batch > hma::kMaxBatch || max_pages_per_seq > (1 << 26)) return HMA_ERR_UNSUPPORTED_SHAPE;
    if (workspace_bytes < hma_decode_attention_workspace_bytes(&cache->desc, batch)) return HMA_ERR_WORKSPACE_TOO_SMALL;
    if (cache->desc.format != HMA_KV_BFP8 && probe) return HMA_ERR_UNSUPPORTED_SHAPE;
    if (cache->desc.format != HMA_KV_BFP8) {
        // BF16 caches are served by the plain kernel until the tensor-core BF16 variant lands
        return hma_decode_attention_simple(cache, layer, q, out, out_dtype, block_table, max_pages_per_seq, context_lens,
                                           batch, sm_scale, stream);
    }
    static int n_sm = 0;
    static bool attr_set = false;
    if (!n_sm) {
        int dev = 0;
        HMA_CUDA_OK(cudaGetDevice(&dev));
        HMA_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    }
    const size_t smem = hma::attn_smem_bytes(batch);
    if (!attr_set) {
        HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_bfp8_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_bfp8_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_bfp8_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr_set = true;
    }
    if (smem > 227 * 1024) return HMA_ERR_UNSUPPORTED_SHAPE;
    hma::AttnArgs a;
    a.cv = hma::CacheView{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                          cache->desc.num_q_heads, cache->desc.format, cache->flags};
    a.q = (const uint16_t *)q;
    a.out = out;
    a.out_dtype = out_dtype;
    a.block_table = block_table;
    a.max_pages = max_pages_per_seq;
    a.ctx = context_lens;
    a.batch = batch;
    a.sm_scale = sm_scale;
    a.cum = (int32_t *)workspace;
    a.tiles = (float *)((uint8_t *)workspace + hma::cum_bytes(batch));
    const int n_ctas = n_sm < hma::kMaxCtas ? n_sm : hma::kMaxCtas;
    cudaStream_t s = (cudaStream_t)stream;
    if (probe == 0) hma::attn_bfp8_kernel<0><<<n_ctas, hma::kThreads, smem, s>>>(a);
    else if (probe == 1) hma::attn_bfp8_kernel<1><<<n_ctas, hma::kThreads, smem, s>>>(a);
    else hma::attn_bfp8_kernel<2><<<n_ctas, hma::kThreads, smem, s>>>(a);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    if (probe) return HMA_OK;
    hma::attn_reduce_kernel<<<batch * cache->desc.num_kv_heads, 128, 0, s>>>(a, n_ctas);
    hma::count_launch();
    HMA_CUDA_OK(cudaGetLastError());
    return HMA_OK;
}

extern "C" hma_status_t hma_decode_attention(const hma_cache_t *cache, int32_t layer, const void *q, void *out,
                                             int32_t out_dtype, const int32_t *block_table, int32_t max_pages_per_seq,
                                             const int32_t *context_lens, int32_t batch, float sm_scale, void *workspace,
                                             size_t workspace_bytes, void *stream)
{
    return launch_attention(cache, layer, q, out, out_dtype, block_table, max_pages_per_seq, context_lens, batch, sm_scale,
                            workspace, workspace_bytes, stream, 0);
}

extern "C" hma_status_t hma_kv_read_probe(const hma_cache_t *cache, int32_t layer, const int32_t *block_table,
                                          int32_t max_pages_per_seq, const int32_t *context_lens, int32_t batch,
                                          void *workspace, size_t workspace_bytes, void *stream)
{
    return launch_attention(cache, layer, nullptr, nullptr, HMA_OUT_BF16, block_table, max_pages_per_seq, context_lens, batch,
                            1.0f, workspace, workspace_bytes, stream, 1);
}

// Diagnostic twin of the probe: the consumer warps run the full arithmetic of every record on whatever
// the ring holds; nothing is loaded and nothing is written.  Its time is the kernel's instruction-issue floor.
extern "C" hma_status_t hma_attention_alu_probe(const hma_cache_t *cache, int32_t layer, const int32_t *block_table,
                                                int32_t max_pages_per_seq, const int32_t *context_lens, int32_t batch,
                                                void *workspace, size_t workspace_bytes, void *stream)
{
    return launch_attention(cache, layer, nullptr, nullptr, HMA_OUT_BF16, block_table, max_pages_per_seq, context_lens, batch,
                            1.0f, workspace, workspace_bytes, stream, 2);
}
