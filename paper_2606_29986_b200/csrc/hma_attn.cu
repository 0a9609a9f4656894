// Fused BFP8 paged decode attention for sm_100a (section 3.3: BFP8 pages stay raw in HBM and are
// rebuilt inside the attention kernel).
//
// Shape of the kernel
//   * persistent grid, one CTA of 16 warps per SM (four warps per SM sub-partition, 128 registers each).
//     All (sequence, kv head, page) records of the batch form one linear work list that is cut into
//     contiguous ranges of equal cost, one per *warp* (any mix of context lengths, no barrier between
//     warps; starting a segment is charged like two records).  A warp that holds only part of a
//     (sequence, kv head) segment leaves a partial (max, sum, 128-vector) per q head in its own ring slots; when
//     every warp of the CTA is done the CTA combines, in warp order, the partials that belong to one segment.  A
//     segment that lies inside one CTA is finished there; one that several CTAs share goes to global memory as one
//     partial per CTA, and the CTA that arrives last (an arrival counter per segment in the workspace) merges them
//     in CTA order.  Every order is fixed, so results are bitwise repeatable; there is no second kernel.
//   * every warp feeds itself: it keeps three 4352-byte page records in flight with 1-D bulk async
//     copies (cp.async.bulk + mbarrier transaction counts) and re-arms a ring slot as soon as its
//     Q.K^T phase has pulled the record's words into registers.
//   * unpack is two integer instructions per pair of elements (byte permute + mask): the element
//     byte s<<7|m becomes the FP16 bit pattern s<<15|m, which *is* the number +-m * 2^-24 (an FP16
//     subnormal), so mantissas enter mma.sync.m16n8k16 exactly.  The shared block exponent never
//     touches the elements: for Q.K^T one MMA k-step is one 16-channel block of each token, so
//     2^E scales the fp32 partial product; for P.V it is folded into the softmax weights, relative
//     to a running per-block reference exponent that is handled like the running softmax maximum.
//   * the softmax weights go to the second MMA as FP16 (11 significant bits), not BF16.
#include <cuda_fp16.h>
#include <mutex>

#include "hma_common.cuh"

namespace hma {

constexpr int kWarps = 16;                        // warps per CTA on a BFP8 cache (and the bound used to size the workspace)
constexpr int kDepth = 3;                         // ring slots per warp
constexpr int kScratch = 768;                     // per warp: 512 B of fp32 K scales + 256 B of FP16 V scales
// Per cache format: a BF16 record is 8192 B, so only 8 warps x 3 slots fit in shared memory; its arithmetic is
// light enough (no unpack) for 8 warps.
// kQ: query tokens a warp works on at once (one MMA n-tile of up to 8 heads each).  Two tiles need about 56 more
// registers per thread, so that variant runs 8 warps of 256 registers, each with a ring twice as deep.
template <int kFmt, int kQ = 1>
struct Geo {
    static constexpr int warps = kFmt == HMA_KV_BFP8 ? kWarps / kQ : 8;
    static constexpr int depth = kFmt == HMA_KV_BFP8 ? kDepth * kQ : kDepth;      // ring slots per warp
    static constexpr int threads = warps * 32;
    static constexpr int stages = warps * depth;
    static constexpr int record = kFmt == HMA_KV_BFP8 ? kBfp8Record : kBf16Record;
    static constexpr int scratch = kFmt == HMA_KV_BFP8 ? kScratch : 0;
};
constexpr int kTileFloats = 8 * kHeadDim + 16;    // partial tile in global memory: o[8][128], m[8], l[8]
constexpr int kPieceStride = kHeadDim + 4;        // floats per head of a partial parked in a ring slot (bank-conflict-free)
constexpr int kPieceFloats = 8 * kPieceStride + 16;   // 1072 floats = 4288 B: fits the smallest ring slot (4352 B)
static_assert(kPieceFloats * 4 <= kBfp8Record && kTileFloats * 4 <= kBfp8Record, "a parked partial must fit a ring slot");
constexpr uint32_t kSpinLimit = 1u << 20;           // polls of a bounded wait
constexpr uint32_t kSuspendNs = 2000;              // a failed poll may keep the thread parked this long
constexpr int kMaxBatch = 1024;
constexpr int kSegCost = 2;                        // what starting a segment costs a warp, in records (Q load, partial tile)
constexpr int kMaxCtas = 192;                       // CTAs launched = min(SM count, kMaxCtas); sizes the workspace
constexpr int kMinRecords = 4;                    // fewest records a worker takes
constexpr int kAlignedMaxPages = 8;               // a plan gives every segment to one warp when none is longer than this
constexpr int kMaxDevices = 64;
constexpr int kMaxGroups = 32;       // more than a CTA can have: a group holds a boundary between two of its (at most 16) warps, or one of its own ends
constexpr int kGroupInts = 6;        // sequence, kv head, member mask, flags (1 whole segment, 2 has tail, tail warp << 8), parts, first CTA

// A plan holds what the kernel's set-up works out from the context lengths and the block table alone, so that the calls
// of one decode step (same lengths and table for every layer) do it once: the two page prefixes, every warp's record
// range with its first segment and its first 32 record addresses, and every CTA's reduction plan.  Written by kMode 5,
// read by kMode 6.  Layout: header (256 B) | one PlanWorker per warp slot | 32 record offsets per warp slot |
// kPlanGroupInts ints per CTA | cum, ecum.  Everything but the prefixes sits at offsets that do not depend on the batch, so
// a planned kernel may load its own entries before it has checked the header: any plan buffer is large enough for that.
constexpr uint32_t kPlanMagic = 0x504C414Eu;
constexpr int kPlanGroupInts = kMaxGroups * kGroupInts + 4;
struct PlanHeader {
    uint32_t magic;
    int32_t rows, hkv, warps, grid, kq, fmt, q_len, max_pages, num_pages;
};
struct __align__(16) PlanWorker {
    long long wlo, whi;          // record range of the warp
    int32_t u;                   // worker index, -1: the warp is no worker
    int32_t b, g, page;          // segment and page of record wlo
};
__host__ __device__ inline size_t plan_cum_bytes(int rows) { return ((size_t)2 * (rows + 1) * 4 + 255) & ~(size_t)255; }
__host__ __device__ inline size_t plan_workers_off(int) { return 256; }
__host__ __device__ inline size_t plan_roff_off(int rows) { return plan_workers_off(rows) + (size_t)kMaxCtas * kWarps * sizeof(PlanWorker); }
__host__ __device__ inline size_t plan_groups_off(int rows) { return plan_roff_off(rows) + (size_t)kMaxCtas * kWarps * 32 * 4; }
__host__ __device__ inline size_t plan_cum_off(int rows) { return plan_groups_off(rows) + (size_t)kMaxCtas * kPlanGroupInts * 4; }
__host__ __device__ inline size_t plan_total_bytes(int rows) { return plan_cum_off(rows) + plan_cum_bytes(rows); }

struct AttnArgs {
    CacheView cv;
    const uint16_t *q;
    void *out;
    int out_dtype;
    const int32_t *block_table;
    int max_pages;
    const int32_t *ctx;
    int batch;                      // rows of q and out: sequences x query tokens per sequence
    int q_len;                      // query tokens per sequence
    int rows_per_seq;               // rows of the work list per sequence: q_len / (query tokens per warp); row r belongs
                                    // to sequence r / rows_per_seq and holds its queries (r % rows_per_seq) * kQ ..
    float sm_scale;
    int32_t *counters;              // workspace: one arrival counter per (sequence, kv head); zero between calls
    int32_t *cum;                   // workspace: a reserved region between the counters and the tiles (unused)
    float *tiles;                   // workspace: per-CTA partial tiles; CTA c's partial of segment s is tile c + s
    float *tails;                   // workspace: one tile per segment, for the warp that holds the segment's end and goes on
    uint8_t *plan;                  // kMode 5 writes it, kMode 6 reads it (see PlanHeader)
    const float *extra;             // kMode 3: the tiles such a launch left (its `tails`), folded into every segment before it is written
#ifdef HMA_TRACE
    unsigned long long *trace;      // workspace, after the tiles: kTraceWords words per worker (see trace_stamp)
    long long drill_record;         // timeout drill: this record of the work list is announced 16 bytes too long (-1: none)
    uint32_t spin_limit;            // polls of a bounded wait (the drill shortens it)
#endif
};

// Per-warp timing instrumentation, compiled in only with -DHMA_TRACE (a separate library image; the default build
// carries none of it).  Each worker writes kTraceWords 64-bit words after the partial tiles of the workspace:
//   0 SM id   1 after the grid-dependency wait   2 end of the prologue   3 first record landed
//   4 end of the record loop   5 after the last partial/output store   6 records taken   7 kernel entry (before the wait)
//   8 CTA-level reduction begins (all warps of the CTA are done)   9 its segments are reduced
//   10 arrivals on the shared segments' counters are done   11 the CTA leaves   12 the CTA leaves (wall clock)
//   13 record range known   14 first record requested   15 after the reduction was planned
// Words 1-5, 7 and 12-15 are %globaltimer nanoseconds; words 8-11 are the SM's cycle counter (only differences inside a CTA mean anything).
[[maybe_unused]] constexpr int kTraceWords = 16;
#ifdef HMA_TRACE
__device__ __forceinline__ unsigned long long trace_now()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ unsigned trace_smid()
{
    unsigned v;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(v));
    return v;
}
#define HMA_TRACE_STAMP(a, u, i, v)  do { if ((threadIdx.x & 31) == 0 && (a).trace) (a).trace[(u) * kTraceWords + (i)] = (v); } while (0)   /* a plan launch has no workspace, hence no trace area */
#else
#define HMA_TRACE_STAMP(a, u, i, v)  do { } while (0)
#endif

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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendNs)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls (or when another thread of the CTA already gave up),
// raises the CTA's abort word and the device flag, and returns false.  Nothing spins forever.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_word, uint32_t *flags, uint32_t limit = kSpinLimit)
{
    for (uint32_t it = 0; it < limit; ++it) {
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
__device__ __forceinline__ void mma_bf16_acc(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// fp32 pair -> packed BF16 (round to nearest even), first argument in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
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

// Tokens that row b of the work list attends to.  With one query token per sequence that is the sequence's context
// (clamped to what the block table can address).  With q_len query tokens the cache already holds all of them: query i
// sees the context less the q_len - 1 - i newer tokens (causal inside the new tokens), and the rows of a sequence share
// its block table row.
// A row of kQ queries walks the pages its newest query sees; its older queries see one token fewer each.
template <int kQ>
__device__ __forceinline__ int context_of(const AttnArgs &a, int b)
{
    const int s = b / a.rows_per_seq, i = (b - s * a.rows_per_seq) * kQ + kQ - 1;      // the row's newest query
    const int T = max(0, min(a.ctx[s], a.max_pages * kPageTokens));
    return max(0, T - (a.q_len - 1 - i));
}
template <int kQ>
__device__ __forceinline__ int pages_of(const AttnArgs &a, int b) { return (context_of<kQ>(a, b) + kPageTokens - 1) / kPageTokens; }
// row of q and out that holds query t of work-list row b
__device__ __forceinline__ int64_t query_row(int q_len, int rows_per_seq, int kq, int b, int t)
{
    const int s = b / rows_per_seq;
    return (int64_t)s * q_len + (int64_t)(b - s * rows_per_seq) * kq + t;
}

__device__ __forceinline__ void store_out(const AttnArgs &a, int64_t idx, float v)
{
    if (a.out_dtype == HMA_OUT_F32) reinterpret_cast<float *>(a.out)[idx] = v;
    else reinterpret_cast<uint16_t *>(a.out)[idx] = f32_to_bf16_rne(v);
}

// How the work list (WX cost units) is dealt out: `nwk` workers (warps) over the first `ctas` CTAs of the grid.
struct Split {
    int64_t nwk;
    int64_t ctas;
};
__host__ __device__ inline Split make_split(int64_t WX, int grid_ctas, int warps_per_cta)
{
    Split s;
    s.nwk = WX / kMinRecords;
    if (s.nwk > (int64_t)grid_ctas * warps_per_cta) s.nwk = (int64_t)grid_ctas * warps_per_cta;
    if (s.nwk < 1) s.nwk = 1;
    s.ctas = s.nwk < grid_ctas ? s.nwk : grid_ctas;
    return s;
}
// CTA that holds worker u, and the CTAs [c0, c0 + count) whose records meet segment (b, g) of np records; `first` is the
// cost position of the segment's first record.
__host__ __device__ inline int64_t cta_of_worker(const Split &s, int64_t u) { return ((u + 1) * s.ctas - 1) / s.nwk; }
__host__ __device__ inline void segment_ctas(const Split &s, int64_t WX, int64_t first, int np, int64_t *c0, int *count)
{
    const int64_t u0 = ((first + 1) * s.nwk - 1) / WX, u1 = ((first + np) * s.nwk - 1) / WX;   // first and last worker
    *c0 = cta_of_worker(s, u0);
    *count = (int)(cta_of_worker(s, u1) - *c0 + 1);
}

// Two-cache attention: folds the tile that the other cache's launch left for a segment into the running (acc, M, den) of
// q head h; this lane holds channels 4 * lane .. 4 * lane + 3.  `tile` is that segment's tile.
__device__ __forceinline__ void fold_extra(const float *tile, int h, int lane, float4 &acc, float &M, float &den)
{
    const float mi = __ldcg(tile + 8 * kHeadDim + h), li = __ldcg(tile + 8 * kHeadDim + 8 + h);
    const float4 v = __ldcg(reinterpret_cast<const float4 *>(tile + h * kHeadDim) + lane);
    if (mi == -INFINITY) return;                   // nothing of this segment in the other cache (its vector is not meaningful)
    const float Mn = fmaxf(M, mi);
    const float keep = M == -INFINITY ? 0.f : ex2f(M - Mn), wgt = ex2f(mi - Mn);
    acc.x = fmaf(wgt, v.x, acc.x * keep); acc.y = fmaf(wgt, v.y, acc.y * keep);
    acc.z = fmaf(wgt, v.z, acc.z * keep); acc.w = fmaf(wgt, v.w, acc.w * keep);
    den = fmaf(wgt, li, den * keep);
    M = Mn;
}

// ---------------------------------------------------------------- CTA-level reduction and cross-CTA merge
// Runs once per CTA after all of its warps have parked their last partial (a function of its own so that its
// registers do not weigh on the record loop).
struct EpilogueArgs {       // what the reduction needs of AttnArgs, by value (registers, not a stack copy of the parameters)
    void *out;
    float *tiles, *tails;
    int32_t *counters;
    int out_dtype, batch, q_len, rows_per_seq;
    struct { int num_kv_heads, num_q_heads; } cv;
    const float *extra;
    const int32_t *ctx;             // planned calls: what the plan's page counts are checked against at the very end
    const int *cum;
    uint32_t *flags;
    int max_pages;
#ifdef HMA_TRACE
    unsigned long long *trace;      // this warp's trace words
#endif
};
#ifdef HMA_TRACE
#define HMA_TRACE_EPI(a, i)  do { if ((threadIdx.x & 31) == 0) (a).trace[i] = (unsigned long long)clock64(); } while (0)   /* SM cycles: cheap to read */
#else
#define HMA_TRACE_EPI(a, i)  do { } while (0)
#endif
// ---- group descriptors: what the CTA-level reduction has to do, worked out once per CTA right after the warps know
// their ranges (everybody is waiting for first data then), so that nothing of it is on the critical path at the end
// One full warp plans the groups of the CTA.  A group is a segment of the CTA's record range that no single warp held
// entirely: `members` are the warps whose last partial (ring slot 0) belongs to it; a warp that held the segment's end
// and went on contributes its tail tile (ring slot 1) after them.  If the CTA holds only part of the segment,
// parts = number of CTAs that share it, first CTA = the lowest.  gstate[0] = number of groups.
template <int kFmt, int kQ>
__device__ __noinline__ void plan_groups(int Hkv, int B, const long long *wr, const int *wseg, const int *cum,
                                         const int *ecum, int *gdesc, int *gstate)
{
    constexpr int kWarps = Geo<kFmt, kQ>::warps;
    const int lane = threadIdx.x & 31;
    const long long my_lo = lane < kWarps ? wr[2 * lane] : 0, my_hi = lane < kWarps ? wr[2 * lane + 1] : 0;   // lane i: range of warp i
    const unsigned have = __ballot_sync(0xFFFFFFFFu, my_lo < my_hi);
    if (have == 0) {
        if (lane == 0) gstate[0] = 0;
        return;
    }
    const long long clo = __shfl_sync(0xFFFFFFFFu, my_lo, __ffs(have) - 1), chi = __shfl_sync(0xFFFFFFFFu, my_hi, 31 - __clz(have));
    int sb = wseg[2 * (__ffs(have) - 1)], sg = wseg[2 * (__ffs(have) - 1) + 1];     // segment of the CTA's first record
    int npb = cum[sb + 1] - cum[sb], n = 0;
    for (;;) {
        const long long s_lo = (long long)Hkv * cum[sb] + (long long)sg * npb, s_hi = s_lo + npb;
        if (s_lo >= chi || n == kMaxGroups) break;
        const long long lo = max(s_lo, clo), hi = min(s_hi, chi);
        unsigned mem = __ballot_sync(0xFFFFFFFFu, my_lo < my_hi && my_lo < hi && my_hi > lo);     // warps with records of this segment
        const int i1 = 31 - __clz(mem);
        const bool one_warp_whole = (mem & (mem - 1)) == 0 && __shfl_sync(0xFFFFFFFFu, my_lo <= s_lo && my_hi >= s_hi, i1);
        if (!one_warp_whole) {
            const bool has_tail = __shfl_sync(0xFFFFFFFFu, my_hi > s_hi, i1);     // the last warp went on into the next segment
            if (has_tail) mem &= ~(1u << i1);
            const bool whole_seg = lo == s_lo && hi == s_hi;
            if (lane == 0) {
                int parts = 0;
                int64_t c0 = 0;
                if (!whole_seg) {
                    const int64_t WX = (int64_t)Hkv * ecum[B];
                    const Split sp = make_split(WX, (int)gridDim.x, kWarps);
                    const int64_t first = (int64_t)Hkv * ecum[sb] + (int64_t)sg * (npb + kSegCost) + kSegCost;   // cost position of the first record
                    segment_ctas(sp, WX, first, npb, &c0, &parts);
                }
                int *d = gdesc + n * kGroupInts;
                d[0] = sb; d[1] = sg; d[2] = (int)mem; d[3] = (whole_seg ? 1 : 0) | (has_tail ? 2 : 0) | (i1 << 8);
                d[4] = parts; d[5] = (int)c0;
            }
            ++n;
        }
        if (++sg == Hkv) {
            sg = 0;
            do { ++sb; } while (sb < B && cum[sb + 1] == cum[sb]);
            if (sb >= B) break;
            npb = cum[sb + 1] - cum[sb];
        }
    }
    if (lane == 0) gstate[0] = n;
}

__device__ __forceinline__ void store_quad(void *out, int out_dtype, int64_t oi, float x, float y, float z, float w)
{
    if (out_dtype == HMA_OUT_F32) *reinterpret_cast<float4 *>(reinterpret_cast<float *>(out) + oi) = make_float4(x, y, z, w);
    else
        *reinterpret_cast<uint2 *>(reinterpret_cast<uint16_t *>(out) + oi) =
            make_uint2(f32_to_bf16_rne(x) | ((uint32_t)f32_to_bf16_rne(y) << 16), f32_to_bf16_rne(z) | ((uint32_t)f32_to_bf16_rne(w) << 16));
}
__device__ __forceinline__ float4 lds_f4(uint32_t addr)
{
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}

// ---------------------------------------------------------------- CTA-level reduction and cross-CTA merge
// Runs once per CTA after all of its warps have parked their last partial (a function of its own so that its
// registers do not weigh on the record loop).  Work items are (group, q head): one warp each, four channels per
// lane; lane i weighs the partial of warp i (lane kWarps: the tail tile), so the weights of a group cost one round of
// loads and two shuffle reductions, and the 128-vectors are then summed in warp order, all loads in flight.  With two
// query tiles per warp every (segment, q head) item exists once per tile.
template <int kFmt, int kQ, bool kExtra, bool kEmit, bool kPlanned>
__device__ __noinline__ void cta_epilogue(const EpilogueArgs a, const uint8_t *ring,
                                          int *misc, const int *gdesc, const int *gstate)
{
    constexpr int kWarps = Geo<kFmt, kQ>::warps, kRecord = Geo<kFmt, kQ>::record, kDepth = Geo<kFmt, kQ>::depth;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int Hkv = a.cv.num_kv_heads, Hq = a.cv.num_q_heads, G = Hq / Hkv;
    const bool aborted = misc[0] != 0;            // outputs of this CTA are void (and flagged); arrivals still happen
    HMA_TRACE_EPI(a, 8);
    const uint32_t ring_s = smem_u32(ring);
    int n_open = 0;                               // segments this CTA shares with other CTAs (at most its first and last)
    {
        const int n = gstate[0];
        if (!aborted)
            for (int item = warp; item < n * kQ * 8; item += kWarps) {
                const int h = item & 7, t = (item >> 3) % kQ;
                if (h >= G) continue;
                const int *d = gdesc + (item >> 3) / kQ * kGroupInts;
                const int sb = d[0], sg = d[1];
                const unsigned mem = (unsigned)d[2];
                const bool whole_seg = d[3] & 1, has_tail = d[3] & 2;
                const uint32_t gtail = ring_s + ((d[3] >> 8) * kDepth + kQ + t) * kRecord;      // dense tile layout
                float mine_m = -INFINITY, mine_l = 0.f;
                if (lane < kWarps && (mem >> lane & 1u)) {
                    const uint32_t pc = ring_s + (lane * kDepth + t) * kRecord + (8 * kPieceStride + h) * 4;
                    mine_m = __uint_as_float(lds32(pc)); mine_l = __uint_as_float(lds32(pc + 32));
                } else if (lane == kWarps && has_tail) {
                    mine_m = __uint_as_float(lds32(gtail + (8 * kHeadDim + h) * 4)); mine_l = __uint_as_float(lds32(gtail + (8 * kHeadDim + 8 + h) * 4));
                }
                // every 128-vector load is issued before the weights are needed; summed in warp order, the tail tile last
                float4 v[kWarps + 1];
#pragma unroll
                for (int i = 0; i < kWarps; ++i) {
                    v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (mem >> i & 1u) v[i] = lds_f4(ring_s + (i * kDepth + t) * kRecord + (h * kPieceStride + 4 * lane) * 4);
                }
                v[kWarps] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (has_tail) v[kWarps] = lds_f4(gtail + (h * kHeadDim + 4 * lane) * 4);
                float M = mine_m;
#pragma unroll
                for (int dd = 16; dd > 0; dd >>= 1) M = fmaxf(M, __shfl_xor_sync(0xFFFFFFFFu, M, dd));
                const float mine_w = mine_m == -INFINITY ? 0.f : ex2f(mine_m - M);
                float den = mine_w * mine_l;
#pragma unroll
                for (int dd = 16; dd > 0; dd >>= 1) den += __shfl_xor_sync(0xFFFFFFFFu, den, dd);      // fixed butterfly order
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int i = 0; i <= kWarps; ++i) {
                    const float wgt = __shfl_sync(0xFFFFFFFFu, mine_w, i);      // 0 for a warp that is no member
                    acc.x = fmaf(wgt, v[i].x, acc.x); acc.y = fmaf(wgt, v[i].y, acc.y);
                    acc.z = fmaf(wgt, v[i].z, acc.z); acc.w = fmaf(wgt, v[i].w, acc.w);
                }
                if (whole_seg && kEmit) {                 // the finished segment, as a tile for the other cache's launch
                    float *tp = a.tails + (((int64_t)sb * Hkv + sg) * kQ + t) * kTileFloats;
                    *reinterpret_cast<float4 *>(tp + h * kHeadDim + 4 * lane) = acc;
                    if (lane == 0) { tp[8 * kHeadDim + h] = M; tp[8 * kHeadDim + 8 + h] = den; }
                } else if (whole_seg) {
                    if (kExtra) fold_extra(a.extra + ((int64_t)sb * Hkv + sg) * kTileFloats, h, lane, acc, M, den);
                    const float inv = den > 0.f ? 1.f / den : 0.f;
                    store_quad(a.out, a.out_dtype, (query_row(a.q_len, a.rows_per_seq, kQ, sb, t) * Hq + (int64_t)sg * G + h) * kHeadDim + 4 * lane,
                               acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
                } else {
                    float *tp = a.tiles + (((int64_t)blockIdx.x + (int64_t)sb * Hkv + sg) * kQ + t) * kTileFloats;
                    *reinterpret_cast<float4 *>(tp + h * kHeadDim + 4 * lane) = acc;
                    if (lane == 0) { tp[8 * kHeadDim + h] = M; tp[8 * kHeadDim + 8 + h] = den; }
                }
            }
        for (int g = 0; g < n; ++g) {                 // note the shared segments (the same in every thread)
            const int *d = gdesc + g * kGroupInts;
            if (d[4] > 0 && n_open < 2) {
                if (tid == 0) { misc[4 + 4 * n_open] = d[4]; misc[5 + 4 * n_open] = d[5]; misc[6 + 4 * n_open] = d[0]; misc[7 + 4 * n_open] = d[1]; }
                ++n_open;
            }
        }
    }
    // A planned call checks, once and after its own work, that the plan's page counts are those of the context lengths it
    // was called with (lengths may have grown inside their last pages since the plan was made).  Nothing unsafe happens
    // otherwise (pages are looked up in the live table and range-checked), but the results are void and the call says so.
    if constexpr (kPlanned)
        for (int bb = blockIdx.x * kWarps * 32 + tid; bb < a.batch; bb += gridDim.x * kWarps * 32) {
            const int s = bb / a.rows_per_seq, i = (bb - s * a.rows_per_seq) * kQ + kQ - 1;
            const int T = max(0, max(0, min(a.ctx[s], a.max_pages * kPageTokens)) - (a.q_len - 1 - i));
            if ((T + kPageTokens - 1) / kPageTokens != a.cum[bb + 1] - a.cum[bb]) atomicOr(a.flags, HMA_FLAG_BAD_PLAN);
        }
    HMA_TRACE_EPI(a, 9);
    if (n_open == 0) return;                      // the same for every thread of the CTA
    // Arrival: the CTA's tile stores happen before the barrier, the release of the arriving thread's atomic carries
    // them (cumulativity) to whoever acquires the counter after the last arrival.
    __syncthreads();
    if (lane == 0 && warp < n_open) {
        int32_t *ctr = a.counters + (int64_t)misc[6 + 4 * warp] * Hkv + misc[7 + 4 * warp];
        int prev;
        asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(prev) : "l"(ctr) : "memory");
        const bool last = prev == misc[4 + 4 * warp] - 1;
        if (last) *ctr = 0;                       // everybody has arrived: leave the counter ready for the next call
        else misc[4 + 4 * warp] = 0;
    }
    __syncthreads();
    HMA_TRACE_EPI(a, 10);
    for (int item = warp; item < n_open * kQ * 8; item += kWarps) {
        const int k = (item >> 3) / kQ, t = (item >> 3) % kQ, h = item & 7;
        const int parts = misc[4 + 4 * k];
        if (parts == 0 || h >= G) continue;       // another CTA will arrive later and finish this segment
        const int ob = misc[6 + 4 * k], og = misc[7 + 4 * k];
        const float *t0 = a.tiles + (((int64_t)misc[5 + 4 * k] + (int64_t)ob * Hkv + og) * kQ + t) * kTileFloats;      // part i is at t0 + i * kQ * kTileFloats
        // parts in CTA order, four at a time (one trip to L2 for the usual two to four parts), running maximum
        float M = -INFINITY, den = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int p0 = 0; p0 < parts; p0 += 4) {
            float mi[4], li[4];
            float4 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float *tp = t0 + (int64_t)(p0 + j) * kQ * kTileFloats;
                const bool ok = p0 + j < parts;
                mi[j] = ok ? __ldcg(tp + 8 * kHeadDim + h) : -INFINITY;
                li[j] = ok ? __ldcg(tp + 8 * kHeadDim + 8 + h) : 0.f;
                v[j] = ok ? __ldcg(reinterpret_cast<const float4 *>(tp + h * kHeadDim) + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            const float Mn = fmaxf(fmaxf(fmaxf(mi[0], mi[1]), fmaxf(mi[2], mi[3])), M);
            const float keep = M == -INFINITY ? 0.f : ex2f(M - Mn);
            acc.x *= keep; acc.y *= keep; acc.z *= keep; acc.w *= keep; den *= keep;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float wgt = mi[j] == -INFINITY ? 0.f : ex2f(mi[j] - Mn);
                acc.x = fmaf(wgt, v[j].x, acc.x); acc.y = fmaf(wgt, v[j].y, acc.y);
                acc.z = fmaf(wgt, v[j].z, acc.z); acc.w = fmaf(wgt, v[j].w, acc.w);
                den = fmaf(wgt, li[j], den);
            }
            M = Mn;
        }
        if (kEmit) {
            float *tp = a.tails + (((int64_t)ob * Hkv + og) * kQ + t) * kTileFloats;
            *reinterpret_cast<float4 *>(tp + h * kHeadDim + 4 * lane) = acc;
            if (lane == 0) { tp[8 * kHeadDim + h] = M; tp[8 * kHeadDim + 8 + h] = den; }
            continue;
        }
        if (kExtra) fold_extra(a.extra + ((int64_t)ob * Hkv + og) * kTileFloats, h, lane, acc, M, den);
        const float inv = den > 0.f ? 1.f / den : 0.f;
        store_quad(a.out, a.out_dtype, (query_row(a.q_len, a.rows_per_seq, kQ, ob, t) * Hq + (int64_t)og * G + h) * kHeadDim + 4 * lane,
                   acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    }
    HMA_TRACE_EPI(a, 11);
#ifdef HMA_TRACE
    if ((threadIdx.x & 31) == 0) a.trace[12] = trace_now();     // wall clock at the CTA's exit
#endif
}

// kMode 0: attention.  1: stream the records through the ring, no arithmetic (bandwidth probe).
// 2: the arithmetic of every record on whatever the ring holds, nothing loaded or written (issue-rate probe).
// 4: attention over two caches, first launch: `out` is never written; every finished segment leaves its unnormalised tile
//    (vectors, maxima, sums) in tails[segment] instead.
// 5: only the set-up, written out as a plan (no record is touched).  6: attention that takes its set-up from a plan.
// 7, 8: modes 3 and 4 with the set-up taken from a plan.
// 3: attention over two caches, second launch: the launch before this one (the other cache, mode 4) left
//    tiles that are folded into every segment before it is written.  Nothing that launch writes is read before
//    the grid-dependency wait, which here comes late: right before the first fold.  Everything else this kernel reads
//    was complete before that launch passed its own wait (it releases its dependents only after it), so the record loop
//    of this launch runs beside it.
extern __shared__ __align__(128) uint8_t smem_raw[];

template <int kMode, int kFmt, int kQ>
__global__ void __launch_bounds__(Geo<kFmt, kQ>::threads, 1) attn_kernel(const AttnArgs a)
{
    constexpr int kWarps = Geo<kFmt, kQ>::warps, kThreads = Geo<kFmt, kQ>::threads, kStages = Geo<kFmt, kQ>::stages;
    constexpr int kRecord = Geo<kFmt, kQ>::record, kDepth = Geo<kFmt, kQ>::depth;
    static_assert(kQ == 1 || kFmt == HMA_KV_BFP8, "two query tiles per warp exist for BFP8 caches only");
    static_assert((kMode != 3 && kMode != 7) || kQ == 1, "two-cache attention takes one query token per sequence");
    constexpr bool kAttn = kMode == 0 || kMode == 3 || kMode == 4 || kMode >= 6, kExtra = kMode == 3 || kMode == 7, kEmit = kMode == 4 || kMode == 8;
    constexpr bool kPlanOnly = kMode == 5, kPlanned = kMode >= 6;
    constexpr bool kBfp8 = kFmt == HMA_KV_BFP8;
    uint8_t *ring = smem_raw;                                                     // kStages records
    uint8_t *scratch = ring + kStages * kRecord;                                  // kWarps x kScratch (BFP8 only)
    uint64_t *bars = reinterpret_cast<uint64_t *>(scratch + kWarps * Geo<kFmt, kQ>::scratch);   // full[kStages]
    int *stage_ok = reinterpret_cast<int *>(bars + kStages);                      // [kStages]
    int *misc = stage_ok + kStages;                                               // [0] abort word, [4..12) epilogue, [16..80) scan scratch
    long long *wr = reinterpret_cast<long long *>(misc + 16 + 64);                // [kWarps][2] record range of each warp
    int *wseg = reinterpret_cast<int *>(wr + 2 * kWarps);                         // [kWarps][2] sequence and kv head of its first record
    int *gdesc = wseg + 2 * kWarps;                                               // [kMaxGroups][kGroupInts] plan of the CTA-level reduction
    int *gstate = gdesc + kMaxGroups * kGroupInts;                                // [4]
    int *cum = gstate + 4;                                                        // [batch + 1] pages before each sequence
    int *ecum = cum + a.batch + 1;                                                // [batch + 1] same, plus kSegCost per non-empty sequence
    volatile int *abort_word = misc;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int Hkv = a.cv.num_kv_heads, Hq = a.cv.num_q_heads, G = Hq / Hkv, B = a.batch;

    constexpr bool kPlannedMode = kMode >= 7;       // the planned two-cache modes, whose short first launch is all head
    if (kPlannedMode && lane == 0) {
        // a planned warp requests its first record before the CTA's first barrier: it prepares its own slots
        for (int s = 0; s < kDepth; ++s) mbar_init(smem_u32(bars + warp * kDepth + s), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (tid == 0) {
        if (!kPlannedMode)
            for (int s = 0; s < kStages; ++s) mbar_init(smem_u32(bars + s), 1);
        misc[0] = 0;
        misc[1] = 0;                     // warps that have published their record range
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    // The kernel is launched with programmatic stream serialisation: its CTAs may be placed while the previous
    // kernel of the stream drains.  Nothing that a predecessor could have written is read before this wait.
#ifdef HMA_TRACE
    const unsigned long long tr_entry = trace_now();
#endif
    if (!kExtra) asm volatile("griddepcontrol.wait;" ::: "memory");
#ifdef HMA_TRACE
    const unsigned long long tr_wait = trace_now();
#endif
    PlanWorker pw = {0, 0, -1, 0, 0, 0};
    constexpr uint32_t kNoRecord = 0xFFFFFFFFu;
    uint32_t plan_roff = kNoRecord;               // planned: this lane's record of the warp's first window
    bool first_requested = false;                 // planned: the warp's first record is already on its way
    if constexpr (kMode == 6) {
        // the plan must have been made for this very launch shape; a call with any other is refused as a whole
        const PlanHeader *ph = reinterpret_cast<const PlanHeader *>(a.plan);
        if (ph->magic != kPlanMagic || ph->rows != B || ph->hkv != Hkv || ph->warps != kWarps || ph->grid != (int)gridDim.x ||
            ph->kq != kQ || ph->fmt != kFmt || ph->q_len != a.q_len || ph->max_pages != a.max_pages || ph->num_pages != (int32_t)a.cv.num_pages) {
            if (tid == 0) atomicOr(a.cv.flags, HMA_FLAG_BAD_PLAN);
            return;
        }
        const int *pc = reinterpret_cast<const int *>(a.plan + plan_cum_off(B));
        for (int i = tid; i < 2 * (B + 1); i += kThreads) cum[i] = pc[i];            // cum and ecum are neighbours
        const int *pg = reinterpret_cast<const int *>(a.plan + plan_groups_off(B)) + (size_t)blockIdx.x * kPlanGroupInts;
        for (int i = tid; i < kPlanGroupInts; i += kThreads) gdesc[i] = pg[i];       // gdesc and gstate are neighbours
        pw = reinterpret_cast<const PlanWorker *>(a.plan + plan_workers_off(B))[blockIdx.x * kWarps + warp];
        __syncthreads();
    } else if constexpr (kPlanned) {
        // The planned two-cache modes: their first launch is short and nearly all head, so the head is cut further (the same
        // order of loads in the one-cache kernel made its record loop 0.8 us slower through different code generation).
        // One trip to L2 for the header, the warp's entry, its first record addresses and the CTA's reduction plan (all at
        // offsets that hold for any plan buffer); then the header is checked: the plan must have been made for this very
        // launch shape, a call with any other is refused as a whole.
        const PlanHeader hd = *reinterpret_cast<const PlanHeader *>(a.plan);
        pw = reinterpret_cast<const PlanWorker *>(a.plan + plan_workers_off(B))[blockIdx.x * kWarps + warp];
        plan_roff = reinterpret_cast<const uint32_t *>(a.plan + plan_roff_off(B))[(blockIdx.x * kWarps + warp) * 32 + lane];
        const int *pg = reinterpret_cast<const int *>(a.plan + plan_groups_off(B)) + (size_t)blockIdx.x * kPlanGroupInts;
        static_assert(kPlanGroupInts <= kThreads, "one thread per word of the CTA's reduction plan");
        const int gword = tid < kPlanGroupInts ? pg[tid] : 0;
        if (hd.magic != kPlanMagic || hd.rows != B || hd.hkv != Hkv || hd.warps != kWarps || hd.grid != (int)gridDim.x ||
            hd.kq != kQ || hd.fmt != kFmt || hd.q_len != a.q_len || hd.max_pages != a.max_pages || hd.num_pages != (int32_t)a.cv.num_pages) {
            if (tid == 0) atomicOr(a.cv.flags, HMA_FLAG_BAD_PLAN);
            return;
        }
        // the warp's first record is requested right away (its slots were prepared by its own lane 0 above)
        const uint32_t r0 = __shfl_sync(0xFFFFFFFFu, plan_roff, 0);
        if (kPlannedMode && pw.u >= 0 && pw.wlo < pw.whi && r0 != kNoRecord) {
            if (lane == 0) {
                uint64_t pol;
                asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
                const uint32_t bar0 = smem_u32(bars + warp * kDepth);
                stage_ok[warp * kDepth] = 1;
#ifdef HMA_TRACE
                mbar_arrive_expect_tx(bar0, kRecord + (pw.wlo == a.drill_record ? 16 : 0));
#else
                mbar_arrive_expect_tx(bar0, kRecord);
#endif
                bulk_load(smem_u32(ring + warp * kDepth * kRecord), a.cv.layer + (uint64_t)r0 * 128u, kRecord, bar0, pol);
            }
            first_requested = true;
        }
        if (tid < kPlanGroupInts) gdesc[tid] = gword;                                // gdesc and gstate are neighbours
        const int *pc = reinterpret_cast<const int *>(a.plan + plan_cum_off(B));
        for (int i = tid; i < 2 * (B + 1); i += kThreads) cum[i] = pc[i];            // cum and ecum are neighbours
        __syncthreads();
    } else {
        // Exclusive prefixes per sequence of (pages) and of (pages + kSegCost if the sequence is not empty): each thread
        // owns `per` consecutive sequences, warps scan with shuffles, one warp scans the warp totals.
        const int per = (B + kThreads - 1) / kThreads;
        const int b0 = min(B, tid * per), b1 = min(B, b0 + per);
        int mine = 0, emine = 0;
        for (int b = b0; b < b1; ++b) { const int n = pages_of<kQ>(a, b); mine += n; emine += n ? n + kSegCost : 0; }
        int incl = mine, eincl = emine;                    // inclusive scans inside the warp
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xFFFFFFFFu, incl, d), ev = __shfl_up_sync(0xFFFFFFFFu, eincl, d);
            if (lane >= d) { incl += v; eincl += ev; }
        }
        if (lane == 31) { misc[16 + warp] = incl; misc[16 + 32 + warp] = eincl; }
        __syncthreads();
        if (warp == 0) {
            int tot = lane < kWarps ? misc[16 + lane] : 0, run = tot;
            int etot = lane < kWarps ? misc[16 + 32 + lane] : 0, erun = etot;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int v = __shfl_up_sync(0xFFFFFFFFu, run, d), ev = __shfl_up_sync(0xFFFFFFFFu, erun, d);
                if (lane >= d) { run += v; erun += ev; }
            }
            if (lane < kWarps) { misc[16 + lane] = run - tot; misc[16 + 32 + lane] = erun - etot; }
            if (lane == kWarps - 1) { cum[B] = run; ecum[B] = erun; }
        }
        __syncthreads();
        int run = misc[16 + warp] + incl - mine, erun = misc[16 + 32 + warp] + eincl - emine;
        for (int b = b0; b < b1; ++b) {
            const int n = pages_of<kQ>(a, b);
            cum[b] = run; ecum[b] = erun;
            run += n; erun += n ? n + kSegCost : 0;
        }
        __syncthreads();
    }
#ifdef HMA_TRACE
    const unsigned long long tr_pro = trace_now();
#endif
    // the next kernel of the stream may be placed as SMs free up; it waits on this grid by itself
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // from here to the CTA-level reduction at the end the warps never synchronise with one another
    const int64_t W = (int64_t)Hkv * cum[B];
    // The work list is cut by cost, not by record count: every (sequence, kv head) segment is charged kSegCost
    // extra units at its start, so a warp whose range crosses a segment boundary (a second Q load, a second partial)
    // gets that many records fewer.  WX is the list's length in cost units.
    const int64_t WX = (int64_t)Hkv * ecum[B];
    // Small batches use fewer workers, at least kMinRecords units each, so that a segment is never cut into more
    // partials than it is worth.  Workers are dealt to the CTAs in contiguous runs (CTA c holds workers
    // [c * NWK / C, (c + 1) * NWK / C) of the C CTAs in use), so a CTA owns one contiguous range of records.
    Split sp = make_split(WX, (int)gridDim.x, kWarps);
    // A plan for short segments (the decode-side tail of two-cache attention: a few pages per sequence) gives every
    // (sequence, kv head) segment to one warp, worker u = sequence * Hkv + head: no segment is shared, so the kernel that
    // follows the plan has no CTA-level reduction and no cross-CTA merge to do at its end.  (Its loop over empty sequences
    // steps by the cost-based worker count; with this numbering worker u = b covers sequence b, and a second visit writes
    // the same bytes.)
    bool aligned = false;
    if constexpr (kPlanOnly) {
        int maxnp = 0;
        for (int bb = 0; bb < B; ++bb) maxnp = max(maxnp, cum[bb + 1] - cum[bb]);
        aligned = maxnp > 0 && maxnp <= kAlignedMaxPages && (int64_t)B * Hkv <= (int64_t)gridDim.x * kWarps;
        if (aligned) {
            sp.nwk = (int64_t)B * Hkv;
            sp.ctas = sp.nwk < (int64_t)gridDim.x ? sp.nwk : (int64_t)gridDim.x;
        }
    }
    const int64_t NWK = sp.nwk;
    int64_t u;                                                      // this warp's worker index (if it is a worker)
    bool worker;
    if constexpr (kPlanned) {
        u = pw.u;
        worker = pw.u >= 0;
    } else {
        const int64_t ubase = (int64_t)blockIdx.x < sp.ctas ? (int64_t)blockIdx.x * NWK / sp.ctas : NWK;
        const int nmine = (int64_t)blockIdx.x < sp.ctas ? (int)(((int64_t)blockIdx.x + 1) * NWK / sp.ctas - ubase) : 0;
        u = ubase + warp;
        worker = warp < nmine;
        if (lane == 0) { wr[2 * warp] = 0; wr[2 * warp + 1] = 0; }  // no records until shown otherwise
    }
    PlanWorker *pw_out = nullptr;
    if constexpr (kPlanOnly) {
        pw_out = reinterpret_cast<PlanWorker *>(a.plan + plan_workers_off(B)) + blockIdx.x * kWarps + warp;
        if (lane == 0) *pw_out = PlanWorker{0, 0, worker ? (int32_t)u : -1, 0, 0, 0};
    }

    // Every warp publishes its record range exactly once; the warp that publishes last plans the CTA-level reduction
    // (who has to combine what at the end) while everybody is still waiting for first data.
    auto publish = [&]() {
        if (kPlanned) return;                      // the plan holds the CTA's reduction plan already
        __syncwarp();
        int cnt = 0;
        if (lane == 0) { __threadfence_block(); cnt = atomicAdd(&misc[1], 1); }
        cnt = __shfl_sync(0xFFFFFFFFu, cnt, 0);
        if (cnt == kWarps - 1 && (kAttn || kPlanOnly)) {
            __threadfence_block();
            plan_groups<kFmt, kQ>(Hkv, B, wr, wseg, cum, ecum, gdesc, gstate);
        }
    };

    do {    // ---- this warp's share of the work list; `break` leaves for the CTA-level reduction ----
    if (!worker) { publish(); break; }
    if (kAttn)                                                    // empty sequences get rows of zeros
        for (int64_t b = u; b < B; b += NWK)
            if (cum[b + 1] == cum[b]) {
                if (kEmit) {
                    // as tiles: maximum -inf, sum 0 (the vectors are not read then)
                    for (int i = lane; i < Hkv * kQ * 16; i += 32)
                        a.tails[(b * Hkv * kQ + i / 16) * kTileFloats + 8 * kHeadDim + (i & 15)] = (i & 8) ? 0.f : -INFINITY;
                } else if (kExtra) {
                    // nothing in this cache: the row is whatever the other cache's launch left for it
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    for (int gh = 0; gh < Hkv * G; ++gh) {
                        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        float M = -INFINITY, den = 0.f;
                        fold_extra(a.extra + (b * Hkv + gh / G) * kTileFloats, gh % G, lane, acc, M, den);
                        const float inv = den > 0.f ? 1.f / den : 0.f;
                        store_quad(a.out, a.out_dtype, (b * Hq + gh) * kHeadDim + 4 * lane, acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
                    }
                } else {
                    for (int i = lane; i < kQ * Hq * kHeadDim; i += 32)
                        store_out(a, query_row(a.q_len, a.rows_per_seq, kQ, (int)b, i / (Hq * kHeadDim)) * Hq * kHeadDim + i % (Hq * kHeadDim), 0.f);
                }
            }

    // number of records that lie before cost position p
    auto records_before = [&](int64_t p) -> int64_t {
        if (p >= WX) return W;
        int lo = 0, hi = B - 1;
        while (lo < hi) {   // largest b with Hkv*ecum[b] <= p: the (non-empty) sequence that holds p
            const int mid = (lo + hi + 1) >> 1;
            if ((int64_t)Hkv * ecum[mid] <= p) lo = mid; else hi = mid - 1;
        }
        const int n = cum[lo + 1] - cum[lo];
        const int64_t off = p - (int64_t)Hkv * ecum[lo];
        const int gg = (int)(off / (n + kSegCost)), r = (int)(off - (int64_t)gg * (n + kSegCost));
        return (int64_t)Hkv * cum[lo] + (int64_t)gg * n + max(0, r - kSegCost);
    };
    int64_t wlo, whi;
    if constexpr (kPlanned) {
        wlo = pw.wlo;
        whi = pw.whi;
    } else {
        if (kPlanOnly && aligned) {
            const int bb = (int)(u / Hkv), gg = (int)(u - (int64_t)bb * Hkv), npb = cum[bb + 1] - cum[bb];
            wlo = (int64_t)Hkv * cum[bb] + (int64_t)gg * npb;
            whi = wlo + npb;
        } else {
            wlo = records_before(u * WX / NWK);
            whi = records_before((u + 1) * WX / NWK);
        }
    }
    if (wlo >= whi) { publish(); break; }
    const int Rw = (int)(whi - wlo);
    HMA_TRACE_STAMP(a, u, 0, (unsigned long long)trace_smid());
    HMA_TRACE_STAMP(a, u, 1, tr_wait);
    HMA_TRACE_STAMP(a, u, 2, tr_pro);
    HMA_TRACE_STAMP(a, u, 7, tr_entry);
    HMA_TRACE_STAMP(a, u, 6, (unsigned long long)Rw);
    HMA_TRACE_STAMP(a, u, 13, trace_now());      // the warp knows its record range

    // the segment (b, g) and page that hold record wlo
    int b, g, page, np;
    if constexpr (kPlanned) {
        b = pw.b; g = pw.g; page = pw.page;
        np = cum[b + 1] - cum[b];
    } else {
        int lo = 0, hi = B - 1;
        while (lo < hi) {   // largest b with Hkv*cum[b] <= wlo
            int mid = (lo + hi + 1) >> 1;
            if ((int64_t)Hkv * cum[mid] <= wlo) lo = mid; else hi = mid - 1;
        }
        while (cum[lo + 1] == cum[lo]) ++lo;   // cannot run off: wlo < W
        b = lo;
        np = cum[lo + 1] - cum[lo];
        const int64_t off = wlo - (int64_t)Hkv * cum[lo];
        g = (int)(off / np);
        page = (int)(off - (int64_t)g * np);
    }
    if (!kPlanned && lane == 0) { wr[2 * warp] = wlo; wr[2 * warp + 1] = whi; wseg[2 * warp] = b; wseg[2 * warp + 1] = g; }

    // ---- the warp's own feed: three ring slots; record addresses are worked out 32 at a time, one per lane ----
    const uint32_t full0 = smem_u32(bars + warp * kDepth);
    const uint32_t ring0 = smem_u32(ring + warp * kDepth * kRecord);
    uint32_t roff = kNoRecord;                    // this lane's record of the current window, in units of 128 bytes
    int kwin = 0;                                 // the window covers records [kwin, kwin + 32) of this warp
    int kissue = 0;                               // next record to request
    int islot = 0;
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    auto refill = [&]() {
        // lane i resolves record kwin + i: sequence by binary search over the page prefix, then head and page
        roff = kNoRecord;
        const int kk = kwin + lane;
        if (kk < Rw) {
            const int64_t wr = wlo + kk;
            int lo = 0, hi = B - 1;
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if ((int64_t)Hkv * cum[mid] <= wr) lo = mid; else hi = mid - 1;
            }
            const int npb = cum[lo + 1] - cum[lo];
            const int off = (int)(wr - (int64_t)Hkv * cum[lo]);
            const int gg = off / npb, pp = off - gg * npb;
            const int32_t pid = a.block_table[(int64_t)(lo / a.rows_per_seq) * a.max_pages + pp];
            if (pid >= 0 && pid < a.cv.num_pages) roff = (uint32_t)(((int64_t)pid * Hkv + gg) * (kRecord / 128));
        }
    };
    auto issue = [&]() {
        if (kMode == 2) return;
        const uint32_t off = __shfl_sync(0xFFFFFFFFu, roff, kissue - kwin);
        if (lane == 0) {
            if (off != kNoRecord) {
                stage_ok[warp * kDepth + islot] = 1;
#ifdef HMA_TRACE
                // the drill: the copy delivers kRecord bytes, the barrier waits for 16 more, the bounded wait runs out
                mbar_arrive_expect_tx(full0 + 8 * islot, kRecord + (wlo + kissue == a.drill_record ? 16 : 0));
#else
                mbar_arrive_expect_tx(full0 + 8 * islot, kRecord);
#endif
                bulk_load(ring0 + islot * kRecord, a.cv.layer + (uint64_t)off * 128u, kRecord, full0 + 8 * islot, policy);
            } else {
                stage_ok[warp * kDepth + islot] = 0;
                atomicOr(a.cv.flags, HMA_FLAG_BAD_PAGE_ATTENTION);
                mbar_arrive(full0 + 8 * islot);
            }
        }
        if (++islot == kDepth) islot = 0;
        if (++kissue == kwin + 32 && kissue < Rw) { kwin = kissue; refill(); }
    };
    if constexpr (kMode == 6) roff = reinterpret_cast<const uint32_t *>(a.plan + plan_roff_off(B))[(blockIdx.x * kWarps + warp) * 32 + lane];
    else if constexpr (kPlanned) roff = plan_roff;
    else if (kMode != 2) refill();
    if constexpr (kPlanOnly) {
        if (lane == 0) *pw_out = PlanWorker{wlo, whi, (int32_t)u, b, g, page};
        reinterpret_cast<uint32_t *>(a.plan + plan_roff_off(B))[(blockIdx.x * kWarps + warp) * 32 + lane] = roff;
        publish();
        break;
    }
    // Only the first record is requested now; the other slots are armed after the first segment's Q loads have been
    // issued, so that across the GPU every warp's first record is ahead of anybody's second in the memory queues.
    if (kPlanned && first_requested) {            // record 0 went out before the CTA's first barrier
        kissue = 1;
        islot = kDepth > 1 ? 1 : 0;
        if (kissue == kwin + 32 && kissue < Rw) { kwin = kissue; refill(); }      // (never: a window holds 32 records)
    } else {
        issue();
    }
    HMA_TRACE_STAMP(a, u, 14, trace_now());      // block table read, first record requested
    publish();
    HMA_TRACE_STAMP(a, u, 15, trace_now());      // (the last warp of the CTA planned the reduction)

    // ---- consumer state ----
    const int gq = lane >> 2, t4 = lane & 3;
    const float kLog2e = 1.4426950408889634f;
    const uint32_t scrK = smem_u32(scratch + warp * Geo<kFmt, kQ>::scratch);   // fp32 2^(E-127) of every (token, block) of K
    const uint32_t scrV = scrK + 512;                            // FP16 scales of every (token pair, block) of V
    // per query tile t (one query token of the row, its up to 8 heads on the MMA's N side):
    uint32_t qf[kQ][8][2];
    float cs0[kQ], cs1[kQ];                        // score multipliers of heads 2*t4, 2*t4+1
    float m0[kQ], m1[kQ];                          // running maxima (log2 domain) of heads 2*t4, 2*t4+1
    float lacc[kQ][4];                             // running sums, via an all-ones MMA
    float o[kQ][8][4];
    int Rmine = 0;                                 // reference exponent of V channel block (lane & 7)
    int T = 0, tail = kPageTokens;
    bool whole = false;                            // this warp holds every record of the current segment
    int64_t tail_seg = -1;                         // segment whose end this warp held before going on (its tail tile is in global memory)

    auto begin_segment = [&](int k) {
        np = cum[b + 1] - cum[b];
        T = context_of<kQ>(a, b);
        tail = T - (np - 1) * kPageTokens;
        whole = page == 0 && Rw - k >= np;
        // Q fragments of this (sequence, kv head), per query token: FP16, one power-of-two scale per head
        const bool hv = gq < G && kAttn;           // the probes have no Q: nothing is read through a.q
        const bool inter = a.cv.key_layout == HMA_KEYS_INTERLEAVED;
#pragma unroll
        for (int t = 0; t < kQ; ++t) {
            float f[8][4];
            float amax = 0.f;
            const uint16_t *qrow = a.q + ((query_row(a.q_len, a.rows_per_seq, kQ, b, t) * Hq + (int64_t)g * G + (hv ? gq : 0))) * kHeadDim;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                // this lane's cached key channels 16j + 4*t4 .. +3 meet the query channels of the same rotary pairs
                uint2 v = make_uint2(0u, 0u);
                if (hv && !inter) v = *reinterpret_cast<const uint2 *>(qrow + 16 * j + 4 * t4);
                if (hv && inter) {
                    const uint32_t lo = *reinterpret_cast<const uint32_t *>(qrow + 8 * j + 2 * t4);        // q[a], q[a+1]
                    const uint32_t hi = *reinterpret_cast<const uint32_t *>(qrow + 8 * j + 2 * t4 + 64);   // q[a+64], q[a+65]
                    v.x = (lo & 0xFFFFu) | (hi << 16);            // key channels 4*t4, 4*t4+1  <- q[a], q[a+64]
                    v.y = (lo >> 16) | (hi & 0xFFFF0000u);        // key channels 4*t4+2, +3    <- q[a+1], q[a+65]
                }
                f[j][0] = __uint_as_float(v.x << 16);
                f[j][1] = __uint_as_float(v.x & 0xFFFF0000u);
                f[j][2] = __uint_as_float(v.y << 16);
                f[j][3] = __uint_as_float(v.y & 0xFFFF0000u);
#pragma unroll
                for (int c = 0; c < 4; ++c) amax = fmaxf(amax, fabsf(f[j][c]));
            }
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
            amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 2));
            float cs;
            if (kBfp8) {
                int shift = 0;
                if (amax > 0.f && amax < INFINITY) shift = 14 - ((int)((__float_as_uint(amax) >> 23) & 0xFF) - 127);
                shift = max(-120, min(120, shift));
                const float up = pow2_field(127 + shift), down = pow2_field(127 - shift);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    qf[t][j][0] = pack_half2(f[j][0] * up, f[j][1] * up);
                    qf[t][j][1] = pack_half2(f[j][2] * up, f[j][3] * up);
                }
                // mantissas enter as m * 2^-24 and exponents as 2^(E-127) while values are m * 2^(E-133): 2^18 is owed
                cs = a.sm_scale * kLog2e * down * 262144.f;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) {       // Q stays BF16: exact repacking of the loaded bits
                    qf[t][j][0] = (__float_as_uint(f[j][0]) >> 16) | (__float_as_uint(f[j][1]) & 0xFFFF0000u);
                    qf[t][j][1] = (__float_as_uint(f[j][2]) >> 16) | (__float_as_uint(f[j][3]) & 0xFFFF0000u);
                }
                cs = a.sm_scale * kLog2e;
            }
            cs0[t] = __shfl_sync(0xFFFFFFFFu, cs, (2 * t4) * 4);
            cs1[t] = __shfl_sync(0xFFFFFFFFu, cs, (2 * t4 + 1) * 4);
            m0[t] = -INFINITY;
            m1[t] = -INFINITY;
            lacc[t][0] = lacc[t][1] = lacc[t][2] = lacc[t][3] = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) o[t][j][0] = o[t][j][1] = o[t][j][2] = o[t][j][3] = 0.f;
        }
        Rmine = 0;
    };

    // The warp is done with its records of the current segment.  A segment it held entirely is finished here (written
    // to `out`, or as a partial tile for the two-cache merge).  Otherwise the partial (o, m, l) waits for the CTA-level
    // reduction: in the warp's ring slot 0 if these were the warp's last records (the ring is idle by then), else (the
    // warp goes on into the next segment, so it held the end of this one, and only one warp does) in the segment's
    // tail tile in global memory, which the warp copies back into its ring slot kQ + t once its ring is idle (per query
    // tile t: slots 0 .. kQ-1 hold the last partial, slots kQ .. 2kQ-1 the tail tile).
    auto finish_segment = [&](bool at_end) {
        if (kMode == 1) return;
        const int h0 = 2 * t4, h1 = 2 * t4 + 1;
        const int64_t seg = (int64_t)b * Hkv + g;
        if (!whole && !at_end) tail_seg = seg;
#pragma unroll
        for (int t = 0; t < kQ; ++t) {
            if (kBfp8) {
                // to true units: accumulators hold sum p * m * 2^(E - R - 9); values are m * 2^(E-133)
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float vsc = pow2_field(min(__shfl_sync(0xFFFFFFFFu, Rmine, j) + 3, 254));
                    o[t][j][0] *= vsc; o[t][j][1] *= vsc; o[t][j][2] *= vsc; o[t][j][3] *= vsc;
                }
            }
            const float l0 = lacc[t][0], l1 = lacc[t][1];
            // a softmax sum that is not finite: scores overflowed fp32 (K exponents beyond the supported range)
            if (kAttn && (!(l0 < INFINITY) || !(l1 < INFINITY))) atomicOr(a.cv.flags, HMA_FLAG_EXPONENT_RANGE);
            if (kMode == 2 && a.batch >= 0) continue;    // the issue-rate probe never stores, but keeps its arithmetic live
            if (whole && !kEmit) {
                const int64_t ob = (query_row(a.q_len, a.rows_per_seq, kQ, b, t) * Hq + (int64_t)g * G) * kHeadDim;
                float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
                if (kExtra) {
                    // the other cache's parts of this segment, folded in the accumulator layout (heads h0, h1 of this lane)
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    const float *tp = a.extra + seg * kTileFloats;
                    float ll0 = l0, ll1 = l1;
                    const float e0 = __ldcg(tp + 8 * kHeadDim + h0), e1 = __ldcg(tp + 8 * kHeadDim + h1);
                    const float n0 = fmaxf(m0[t], e0), n1 = fmaxf(m1[t], e1);
                    const float k0 = m0[t] == -INFINITY ? 0.f : ex2f(m0[t] - n0), k1 = m1[t] == -INFINITY ? 0.f : ex2f(m1[t] - n1);
                    const float w0 = e0 == -INFINITY ? 0.f : ex2f(e0 - n0), w1 = e1 == -INFINITY ? 0.f : ex2f(e1 - n1);
                    ll0 = fmaf(w0, __ldcg(tp + 8 * kHeadDim + 8 + h0), ll0 * k0);
                    ll1 = fmaf(w1, __ldcg(tp + 8 * kHeadDim + 8 + h1), ll1 * k1);
#pragma unroll
                    for (int j = 0; j < 8; ++j)
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            // a head the other cache holds nothing of contributes nothing, whatever its vector's bytes are
                            const float wv = (c & 1) ? w1 : w0;
                            const float x = __ldcg(tp + ((c & 1) ? h1 : h0) * kHeadDim + 16 * j + gq + 8 * (c >> 1));
                            o[t][j][c] = fmaf(wv, wv > 0.f ? x : 0.f, o[t][j][c] * ((c & 1) ? k1 : k0));
                        }
                    i0 = ll0 > 0.f ? 1.f / ll0 : 0.f;
                    i1 = ll1 > 0.f ? 1.f / ll1 : 0.f;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j)
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        const int h = (c & 1) ? h1 : h0;
                        if (h < G) store_out(a, ob + h * kHeadDim + 16 * j + gq + 8 * (c >> 1), o[t][j][c] * ((c & 1) ? i1 : i0));
                    }
                continue;
            }
            float *tp;
            int hs;           // floats between heads
            if (whole) {      // two-cache attention, first launch: the finished segment's tile, for the other cache's launch
                tp = a.tails + (seg * kQ + t) * kTileFloats;
                hs = kHeadDim;
            } else if (at_end) {
                tp = reinterpret_cast<float *>(ring + (warp * kDepth + t) * kRecord);
                hs = kPieceStride;
            } else {
                tp = a.tails + (seg * kQ + t) * kTileFloats;
                hs = kHeadDim;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j)
#pragma unroll
                for (int c = 0; c < 4; ++c) tp[((c & 1) ? h1 : h0) * hs + 16 * j + gq + 8 * (c >> 1)] = o[t][j][c];
            if (gq == 0) {
                tp[8 * hs + h0] = m0[t]; tp[8 * hs + h1] = m1[t];
                tp[8 * hs + 8 + h0] = l0; tp[8 * hs + 8 + h1] = l1;
            }
        }
    };

    // ---- the records of this warp ----
    int slot = 0;
    uint32_t par = 0;
    int left = 0;                                  // records of the current segment still to do
    bool alive = true;
    for (int k = 0; k < Rw; ++k) {
        if (left == 0) {
            if (k > 0) {
                finish_segment(false);
                page = 0;
                if (++g == Hkv) {
                    g = 0;
                    do { ++b; } while (b < B && cum[b + 1] == cum[b]);
                }
            }
            begin_segment(k);
            if (k == 0)
                for (int kk = 1; kk < kDepth && kk < Rw; ++kk) issue();
            left = min(np - page, Rw - k);
        }
        --left;
        const uint32_t sp = ring0 + slot * kRecord;
        const int s_idx = warp * kDepth + slot;
        if (kMode != 2) {
#ifdef HMA_TRACE
            alive = mbar_wait(full0 + 8 * slot, par, abort_word, a.cv.flags, a.spin_limit);
#else
            alive = mbar_wait(full0 + 8 * slot, par, abort_word, a.cv.flags);
#endif
            if (!alive) break;
#ifdef HMA_TRACE
            if (k == 0) HMA_TRACE_STAMP(a, u, 3, trace_now());
#endif
        }
        if (++slot == kDepth) { slot = 0; par ^= 1u; }
        const bool ok = kMode == 2 || stage_ok[s_idx] != 0;
        const bool last_page = page == np - 1;
        const int nvalid = last_page ? tail : kPageTokens;
        ++page;
        if (kMode == 1 || !ok) {
            __syncwarp();
            if (k + kDepth < Rw) issue();
            continue;
        }

        if constexpr (kBfp8) {
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
                    for (int c = 0; c < 4; ++c)
                        if (2 * tt + (c & 1) + 8 * (c >> 1) < nvalid) keep |= 0xFFu << (8 * c);
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
                    if (kAttn && Rnew > 250) atomicOr(a.cv.flags, HMA_FLAG_EXPONENT_RANGE);   // beyond the supported range
    #pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int dlt = __shfl_sync(0xFFFFFFFFu, Rmine, j) - __shfl_sync(0xFFFFFFFFu, Rnew, j);   // <= 0
                        const float fr = dlt < -126 ? 0.f : pow2_field(127 + dlt);
    #pragma unroll
                        for (int t = 0; t < kQ; ++t) { o[t][j][0] *= fr; o[t][j][1] *= fr; o[t][j][2] *= fr; o[t][j][3] *= fr; }
                    }
                    Rmine = Rnew;
                }
                // FP16 scale 2^(E - R + 15) of every (token pair, block): exponent field max(E - R + 30, 0)
                const uint32_t kmine = ((uint32_t)(30 - Rmine) & 0xFFFFu) * 0x00010001u;
                sts64(scrV + ((lane & 6) << 5) + ((lane >> 3) << 4) + ((lane & 1) << 3), __viaddmax_s16x2_relu(prmt(vw, 0u, 0x4140u), kmine, 0u) << 10,
                      __viaddmax_s16x2_relu(prmt(vw, 0u, 0x4342u), kmine, 0u) << 10);
            }
            uint4 km[4];
    #pragma unroll
            for (int c = 0; c < 4; ++c) km[c] = lds128(sp + 128 + c * 512 + lane * 16);
            __syncwarp();

            // ================= Q.K^T =================
            float sc[kQ][4];
    #pragma unroll
            for (int t = 0; t < kQ; ++t) sc[t][0] = sc[t][1] = sc[t][2] = sc[t][3] = 0.f;
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
    #pragma unroll
                    for (int t = 0; t < kQ; ++t) {       // the unpacked keys serve every query tile
                        float d[4];
                        mma_f16(d, af, qf[t][j][0], qf[t][j][1], zero4);
                        sc[t][0] = fmaf(d[0], ks[j], sc[t][0]);
                        sc[t][1] = fmaf(d[1], ks[j], sc[t][1]);
                        sc[t][2] = fmaf(d[2], ks[8 + j], sc[t][2]);
                        sc[t][3] = fmaf(d[3], ks[8 + j], sc[t][3]);
                    }
                }
            }
            // the V element words go to registers now, so that the ring slot can be re-armed for the record
            // three ahead while softmax and P.V run
            uint4 vm[4];
    #pragma unroll
            for (int c = 0; c < 4; ++c) vm[c] = lds128(sp + kBfp8Half + 128 + c * 512 + lane * 16);
            __syncwarp();
            if (k + kDepth < Rw) {
                if (lane == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // reads above, bulk write below
                issue();
            }
            uint32_t pb0[kQ], pb1[kQ];
    #pragma unroll
            for (int t = 0; t < kQ; ++t) {
                float s0 = sc[t][0] * cs0[t], s1 = sc[t][1] * cs1[t], s2 = sc[t][2] * cs0[t], s3 = sc[t][3] * cs1[t];
                // query t of the row sees kQ - 1 - t tokens fewer than the row's newest query: they are the last tokens
                // of the last page
                const int nv = kQ == 1 ? nvalid : nvalid - (last_page ? kQ - 1 - t : 0);
                if (nv < kPageTokens) {
                    if (gq >= nv) { s0 = -INFINITY; s1 = -INFINITY; }
                    if (gq + 8 >= nv) { s2 = -INFINITY; s3 = -INFINITY; }
                }
                // ================= online softmax (log2 domain) =================
                // The warp-wide maximum is only formed when some score exceeds the running maximum.
                if (__any_sync(0xFFFFFFFFu, fmaxf(s0, s2) > m0[t] || fmaxf(s1, s3) > m1[t])) {
                    float mx0 = fmaxf(s0, s2), mx1 = fmaxf(s1, s3);
    #pragma unroll
                    for (int d = 4; d <= 16; d <<= 1) {
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, d));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, d));
                    }
                    const float mn0 = fmaxf(m0[t], mx0), mn1 = fmaxf(m1[t], mx1);
                    const float a0 = mn0 == -INFINITY ? 1.f : ex2f(m0[t] - mn0), a1 = mn1 == -INFINITY ? 1.f : ex2f(m1[t] - mn1);
                    m0[t] = mn0;
                    m1[t] = mn1;
                    lacc[t][0] *= a0; lacc[t][1] *= a1; lacc[t][2] *= a0; lacc[t][3] *= a1;
    #pragma unroll
                    for (int j = 0; j < 8; ++j) { o[t][j][0] *= a0; o[t][j][1] *= a1; o[t][j][2] *= a0; o[t][j][3] *= a1; }
                }
                // With several query tiles a tile may not have seen any token yet (its only token so far is masked): its
                // maximum is still -inf and every score is -inf; the weights must then be 0, not exp2(-inf + inf).
                const float r0 = (kQ > 1 && m0[t] == -INFINITY) ? 0.f : m0[t], r1 = (kQ > 1 && m1[t] == -INFINITY) ? 0.f : m1[t];
                // weights as FP16, transposed from (token, head) accumulator layout to the B-operand layout
                pb0[t] = movmatrix_trans(pack_half2(ex2f(s0 - r0), ex2f(s1 - r1)));   // tokens 2*t4, 2*t4+1 of head gq
                pb1[t] = movmatrix_trans(pack_half2(ex2f(s2 - r0), ex2f(s3 - r1)));   // tokens 2*t4+8, 2*t4+9
                const uint32_t ones[4] = {0x3C003C00u, 0x3C003C00u, 0x3C003C00u, 0x3C003C00u};
                mma_f16_acc(lacc[t], ones, pb0[t], pb1[t]);
            }
            // ================= P.V =================
            {
                uint4 vs[4];           // (f01, f89) of blocks 2c, 2c+1
    #pragma unroll
                for (int c = 0; c < 4; ++c) vs[c] = lds128(scrV + c * 64 + t4 * 16);
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
    #pragma unroll
                    for (int t = 0; t < kQ; ++t) mma_f16_acc(o[t][j], af, hmul2_u32(pb0[t], f01), hmul2_u32(pb1[t], f89));
                }
            }
            __syncwarp();      // every lane is done with the scratch tables
        } else {
            // ================= BF16 cache: the dequant-free baseline of section 3.3 =================
            // Q.K^T: tokens on M, BF16 operands straight from the record, two accumulators to shorten the chain
            float sca[4] = {0.f, 0.f, 0.f, 0.f}, scb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int jp = 0; jp < 4; ++jp) {
                const uint4 klo = lds128(sp + (2 * jp) * 512 + lane * 16);       // token gq: blocks 2jp, 2jp+1
                const uint4 khi = lds128(sp + (2 * jp + 1) * 512 + lane * 16);   // token gq+8
                const uint32_t a0[4] = {klo.x, khi.x, klo.y, khi.y}, a1[4] = {klo.z, khi.z, klo.w, khi.w};
                mma_bf16_acc(sca, a0, qf[0][2 * jp][0], qf[0][2 * jp][1]);
                mma_bf16_acc(scb, a1, qf[0][2 * jp + 1][0], qf[0][2 * jp + 1][1]);
            }
            // the V words go to registers now, so that the ring slot can be re-armed while softmax and P.V run
            uint4 vm[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) vm[j] = lds128(sp + kBf16Half + j * 512 + lane * 16);
            if (nvalid < kPageTokens) {
                // whatever the tail of the last page holds (NaN patterns included) must not reach the MMA: 0 * NaN = NaN
                const uint32_t mlo = (2 * t4 < nvalid ? 0xFFFFu : 0u) | (2 * t4 + 1 < nvalid ? 0xFFFF0000u : 0u);
                const uint32_t mhi = (2 * t4 + 8 < nvalid ? 0xFFFFu : 0u) | (2 * t4 + 9 < nvalid ? 0xFFFF0000u : 0u);
#pragma unroll
                for (int j = 0; j < 8; ++j) { vm[j].x &= mlo; vm[j].y &= mlo; vm[j].z &= mhi; vm[j].w &= mhi; }
            }
            __syncwarp();
            if (k + kDepth < Rw) {
                if (lane == 0) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // reads above, bulk write below
                issue();
            }
            float s0 = (sca[0] + scb[0]) * cs0[0], s1 = (sca[1] + scb[1]) * cs1[0], s2 = (sca[2] + scb[2]) * cs0[0], s3 = (sca[3] + scb[3]) * cs1[0];
            if (nvalid < kPageTokens) {
                if (gq >= nvalid) { s0 = -INFINITY; s1 = -INFINITY; }
                if (gq + 8 >= nvalid) { s2 = -INFINITY; s3 = -INFINITY; }
            }
            if (__any_sync(0xFFFFFFFFu, fmaxf(s0, s2) > m0[0] || fmaxf(s1, s3) > m1[0])) {
                float mx0 = fmaxf(s0, s2), mx1 = fmaxf(s1, s3);
#pragma unroll
                for (int d = 4; d <= 16; d <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xFFFFFFFFu, mx0, d));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xFFFFFFFFu, mx1, d));
                }
                const float mn0 = fmaxf(m0[0], mx0), mn1 = fmaxf(m1[0], mx1);
                const float a0 = mn0 == -INFINITY ? 1.f : ex2f(m0[0] - mn0), a1 = mn1 == -INFINITY ? 1.f : ex2f(m1[0] - mn1);
                m0[0] = mn0;
                m1[0] = mn1;
                lacc[0][0] *= a0; lacc[0][1] *= a1; lacc[0][2] *= a0; lacc[0][3] *= a1;
#pragma unroll
                for (int j = 0; j < 8; ++j) { o[0][j][0] *= a0; o[0][j][1] *= a1; o[0][j][2] *= a0; o[0][j][3] *= a1; }
            }
            // weights as BF16 hi + lo (16 significant bits): BF16-rounded weights alone would cost 1e-3 of relative error
            const float p0 = ex2f(s0 - m0[0]), p1 = ex2f(s1 - m1[0]), p2 = ex2f(s2 - m0[0]), p3 = ex2f(s3 - m1[0]);
            const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
            const uint32_t l01 = pack_bf16x2(p0 - __uint_as_float(h01 << 16), p1 - __uint_as_float(h01 & 0xFFFF0000u));
            const uint32_t l23 = pack_bf16x2(p2 - __uint_as_float(h23 << 16), p3 - __uint_as_float(h23 & 0xFFFF0000u));
            const uint32_t ph0 = movmatrix_trans(h01), ph1 = movmatrix_trans(h23);
            const uint32_t pl0 = movmatrix_trans(l01), pl1 = movmatrix_trans(l23);
            {
                const uint32_t ones[4] = {0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u};
                mma_bf16_acc(lacc[0], ones, ph0, ph1);
                mma_bf16_acc(lacc[0], ones, pl0, pl1);
            }
            // P.V: channels on M, tokens on K; one 16-byte word per lane is one operand fragment
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t af[4] = {vm[j].x, vm[j].y, vm[j].z, vm[j].w};
                mma_bf16_acc(o[0][j], af, ph0, ph1);
                mma_bf16_acc(o[0][j], af, pl0, pl1);
            }
        }
    }
    HMA_TRACE_STAMP(a, u, 4, trace_now());
    if (alive) {
        finish_segment(true);
        if (tail_seg >= 0 && kAttn) {
            // the last tail tile this warp wrote (it can only be shared with other warps if it was the warp's first
            // segment, and a warp writes at most one such) comes back from L2 into ring slot 1, same layout
            __syncwarp();
#pragma unroll
            for (int t = 0; t < kQ; ++t) {
                const uint4 *src = reinterpret_cast<const uint4 *>(a.tails + (tail_seg * kQ + t) * kTileFloats);
                const uint32_t dst = ring0 + (kQ + t) * kRecord;
                uint4 v[(kTileFloats * 4 / 16 + 31) / 32];
#pragma unroll
                for (int i = 0; i < (kTileFloats * 4 / 16 + 31) / 32; ++i)
                    if (lane + 32 * i < kTileFloats * 4 / 16) v[i] = __ldcg(src + lane + 32 * i);
#pragma unroll
                for (int i = 0; i < (kTileFloats * 4 / 16 + 31) / 32; ++i)
                    if (lane + 32 * i < kTileFloats * 4 / 16) sts128(dst + (lane + 32 * i) * 16, v[i].x, v[i].y, v[i].z, v[i].w);
            }
        }
    }
    HMA_TRACE_STAMP(a, u, 5, trace_now());
    if (!alive && lane == 0 && kMode != 2) {
        // a wait ran out: give the copies still in flight a bounded chance to land before the warp leaves
        for (int s = 0; s < kDepth; ++s)
            for (uint32_t it = 0; it < (1u << 16) && !mbar_try_wait(full0 + 8 * s, 0) && !mbar_try_wait(full0 + 8 * s, 1); ++it) {}
    }
    } while (0);

    if (kExtra) asm volatile("griddepcontrol.wait;" ::: "memory");     // the other cache's tiles are read from here on
    __syncthreads();
    if constexpr (kPlanOnly) {
        int *pg = reinterpret_cast<int *>(a.plan + plan_groups_off(B)) + (size_t)blockIdx.x * kPlanGroupInts;
        const int used = gstate[0] * kGroupInts;
        for (int i = tid; i < kPlanGroupInts; i += kThreads) pg[i] = i < used ? gdesc[i] : i == kMaxGroups * kGroupInts ? gstate[0] : 0;
        if (blockIdx.x == 0) {
            int *pc = reinterpret_cast<int *>(a.plan + plan_cum_off(B));
            for (int i = tid; i < 2 * (B + 1); i += kThreads) pc[i] = cum[i];
            if (tid == 0)
                *reinterpret_cast<PlanHeader *>(a.plan) =
                    PlanHeader{kPlanMagic, B, Hkv, kWarps, (int)gridDim.x, kQ, kFmt, a.q_len, a.max_pages, (int32_t)a.cv.num_pages};
        }
        return;
    }
    if (kAttn) {
        EpilogueArgs e;
        e.out = a.out; e.tiles = a.tiles; e.tails = a.tails; e.counters = a.counters;
        e.out_dtype = a.out_dtype; e.batch = a.batch;
        e.q_len = a.q_len; e.rows_per_seq = a.rows_per_seq;
        e.cv.num_kv_heads = a.cv.num_kv_heads; e.cv.num_q_heads = a.cv.num_q_heads;
        e.extra = a.extra;
        e.ctx = a.ctx; e.cum = cum; e.flags = a.cv.flags; e.max_pages = a.max_pages;
#ifdef HMA_TRACE
        e.trace = a.trace + (((int64_t)blockIdx.x < sp.ctas ? (int64_t)blockIdx.x * sp.nwk / sp.ctas : 0) + warp) * kTraceWords;
#endif
        cta_epilogue<kFmt, kQ, kExtra, kEmit, kPlanned>(e, ring, misc, gdesc, gstate);
    }
}

template <int kFmt, int kQ = 1>
static size_t attn_smem_bytes(int batch)
{
    using G = Geo<kFmt, kQ>;
    return (size_t)G::stages * G::record + (size_t)G::warps * G::scratch + G::stages * 8 + G::stages * 4 + (16 + 64) * 4 +
           (size_t)G::warps * 24 + (kMaxGroups * kGroupInts + 4) * 4 + ((size_t)batch + 1) * 8;
}

// Workspace layout: arrival counters | a reserved region | per-CTA tiles | per-segment tiles [| trace]
static size_t cum_bytes(int batch) { return (((size_t)batch + 1) * 8 + 255) & ~(size_t)255; }
// The counters sit at the head of the workspace in a region of one size for every call, whatever its batch and head
// count, so that calls of different shapes can share a workspace without one's tiles landing on the other's counters.
static size_t counter_bytes(int, int) { return (size_t)kMaxBatch * kMaxKvHeads * 4; }
static size_t cta_tiles(int batch, int hkv) { return 2 * (size_t)kMaxCtas + (size_t)batch * hkv; }     // enough for two query tiles per row

}  // namespace hma

extern "C" size_t hma_decode_attention_workspace_bytes(const hma_cache_desc_t *desc, int32_t batch)
{
    if (!desc || batch < 0 || desc->num_kv_heads <= 0) return 0;
    const int hkv = desc->num_kv_heads;
    size_t bytes = hma::counter_bytes(batch, hkv) + hma::cum_bytes(batch) +
                   (hma::cta_tiles(batch, hkv) + (size_t)batch * hkv) * hma::kTileFloats * 4;
#ifdef HMA_TRACE
    bytes += (size_t)hma::kMaxCtas * hma::kWarps * hma::kTraceWords * 8;
#endif
    return bytes;
}

#ifdef HMA_TRACE
// Instrumented build only: arms the timeout drill for the next attention launch of the calling process.
static long long g_drill_record = -1;
static uint32_t g_drill_spin_limit = 1000;
extern "C" hma_status_t hma_trace_arm_timeout_drill(int64_t record, uint32_t spin_limit)
{
    if (record < 0 || spin_limit == 0) return HMA_ERR_INVALID_ARG;
    g_drill_record = record;
    g_drill_spin_limit = spin_limit;
    return HMA_OK;
}
#endif

extern "C" hma_status_t hma_decode_attention_workspace_init(void *workspace, size_t workspace_bytes, void *stream)
{
    if (!workspace) return HMA_ERR_INVALID_ARG;
    if ((uintptr_t)workspace & 255u) return HMA_ERR_ALIGNMENT;
    HMA_CUDA_OK(cudaMemsetAsync(workspace, 0, workspace_bytes, (cudaStream_t)stream));
    return HMA_OK;
}

static hma_status_t launch_attention(const hma_cache_t *cache, int32_t layer, const void *q, void *out, int32_t out_dtype,
                                     const int32_t *block_table, int32_t max_pages_per_seq, const int32_t *context_lens,
                                     int32_t n_seqs, float sm_scale, void *workspace, size_t workspace_bytes, void *stream,
                                     int probe, int always_partial = 0, hma::AttnArgs *args_out = nullptr, int *ctas_out = nullptr,
                                     int32_t q_len = 1, const float *extra = nullptr, void *plan = nullptr, int plan_mode = 0)
{
    if (!cache || layer < 0 || layer >= cache->desc.num_layers || n_seqs < 0 || max_pages_per_seq < 0 || q_len < 1) return HMA_ERR_INVALID_ARG;
    if ((int64_t)n_seqs * q_len > hma::kMaxBatch) return HMA_ERR_UNSUPPORTED_SHAPE;
    const int32_t batch = n_seqs * q_len;         // rows of q and out
    if (out_dtype != HMA_OUT_BF16 && out_dtype != HMA_OUT_F32) return HMA_ERR_INVALID_ARG;
    if (batch == 0) return HMA_OK;
    if (!block_table || !context_lens || (!workspace && plan_mode != 5) || (!probe && plan_mode != 5 && (!q || !out))) return HMA_ERR_INVALID_ARG;
    if (((uintptr_t)q & 15u) || ((uintptr_t)out & 15u) || ((uintptr_t)workspace & 255u)) return HMA_ERR_ALIGNMENT;
    if (batch > hma::kMaxBatch || max_pages_per_seq > (1 << 26)) return HMA_ERR_UNSUPPORTED_SHAPE;
    if (plan_mode != 5 && workspace_bytes < hma_decode_attention_workspace_bytes(&cache->desc, batch)) return HMA_ERR_WORKSPACE_TOO_SMALL;
    if (plan_mode && (!plan || ((uintptr_t)plan & 255u))) return plan ? HMA_ERR_ALIGNMENT : HMA_ERR_INVALID_ARG;
    const bool bf16 = cache->desc.format != HMA_KV_BFP8;
    if (bf16 && probe == 2) return HMA_ERR_UNSUPPORTED_SHAPE;
    // Two query tokens per warp (they share the unpacked K and V operands) when the query count is even, on BFP8 caches;
    // otherwise every query token is a row of its own.
    const int kq = (!bf16 && probe == 0 && !always_partial && !extra && q_len % 2 == 0) ? 2 : 1;
    const int32_t rows = batch / kq;              // rows of the work list
    // per-device set-up, done by the first call on each device: SM count and the kernels' shared-memory opt-in
    static std::mutex setup_lock;
    static int sm_count[hma::kMaxDevices] = {};
    int dev = 0;
    HMA_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= hma::kMaxDevices) return HMA_ERR_UNSUPPORTED_SHAPE;
    if (dev != cache->device) return HMA_ERR_INVALID_ARG;     // the handle's pointers belong to the device it was made on
    {
        std::lock_guard<std::mutex> guard(setup_lock);
        if (!sm_count[dev]) {
            int n = 0;
            HMA_CUDA_OK(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<0, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<0, HMA_KV_BFP8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<1, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<2, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<0, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<1, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<3, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<3, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<4, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<4, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<5, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<5, HMA_KV_BFP8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<5, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<6, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<6, HMA_KV_BFP8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<6, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<7, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<7, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<8, HMA_KV_BFP8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            HMA_CUDA_OK(cudaFuncSetAttribute(hma::attn_kernel<8, HMA_KV_BF16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
            sm_count[dev] = n;
        }
    }
    const int n_sm = sm_count[dev];
    const size_t smem = bf16 ? hma::attn_smem_bytes<HMA_KV_BF16>(rows)
                             : kq == 2 ? hma::attn_smem_bytes<HMA_KV_BFP8, 2>(rows) : hma::attn_smem_bytes<HMA_KV_BFP8>(rows);
    if (smem > 227 * 1024) return HMA_ERR_UNSUPPORTED_SHAPE;
    hma::AttnArgs a;
    a.cv = hma::CacheView{(uint8_t *)cache->layers[layer], cache->desc.num_pages, cache->desc.num_kv_heads,
                          cache->desc.num_q_heads, cache->desc.format, cache->flags, cache->desc.key_layout};
    a.q = (const uint16_t *)q;
    a.out = out;
    a.out_dtype = out_dtype;
    a.block_table = block_table;
    a.max_pages = max_pages_per_seq;
    a.ctx = context_lens;
    a.batch = rows;
    a.q_len = q_len;
    a.rows_per_seq = q_len / kq;
    a.sm_scale = sm_scale;
    const int hkv = cache->desc.num_kv_heads;
    a.counters = (int32_t *)workspace;
    a.cum = nullptr;
    a.tiles = a.tails = nullptr;
    if (workspace) {
        a.cum = (int32_t *)((uint8_t *)workspace + hma::counter_bytes(batch, hkv));
        a.tiles = (float *)((uint8_t *)a.cum + hma::cum_bytes(batch));
        a.tails = a.tiles + hma::cta_tiles(batch, hkv) * hma::kTileFloats;      // batch = rows x query tiles per row
    }
    a.extra = extra;
    a.plan = (uint8_t *)plan;
#ifdef HMA_TRACE
    a.trace = workspace ? (unsigned long long *)(a.tails + (size_t)batch * hkv * hma::kTileFloats) : nullptr;
    a.drill_record = g_drill_record;
    a.spin_limit = g_drill_record >= 0 ? g_drill_spin_limit : hma::kSpinLimit;
    g_drill_record = -1;
#endif
    const int n_ctas = n_sm < hma::kMaxCtas ? n_sm : hma::kMaxCtas;
    cudaStream_t s = (cudaStream_t)stream;
    const int tb = kq == 2 ? hma::Geo<HMA_KV_BFP8, 2>::threads : hma::Geo<HMA_KV_BFP8>::threads, tf = hma::Geo<HMA_KV_BF16>::threads;
    // The kernel is launched with programmatic stream serialisation: it may be placed on the SMs while its
    // predecessor drains, and it waits on the grid dependency itself before it reads anything.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_ctas);
    cfg.blockDim = dim3((unsigned)(bf16 ? tf : tb));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (plan_mode == 5 && bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<5, HMA_KV_BF16, 1>, a));
    else if (plan_mode == 5 && kq == 2) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<5, HMA_KV_BFP8, 2>, a));
    else if (plan_mode == 5) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<5, HMA_KV_BFP8, 1>, a));
    else if (plan_mode == 6 && extra && bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<7, HMA_KV_BF16, 1>, a));
    else if (plan_mode == 6 && extra) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<7, HMA_KV_BFP8, 1>, a));
    else if (plan_mode == 6 && always_partial && bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<8, HMA_KV_BF16, 1>, a));
    else if (plan_mode == 6 && always_partial) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<8, HMA_KV_BFP8, 1>, a));
    else if (plan_mode == 6 && bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<6, HMA_KV_BF16, 1>, a));
    else if (plan_mode == 6 && kq == 2) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<6, HMA_KV_BFP8, 2>, a));
    else if (plan_mode == 6) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<6, HMA_KV_BFP8, 1>, a));
    else if (always_partial && bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<4, HMA_KV_BF16, 1>, a));
    else if (always_partial) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<4, HMA_KV_BFP8, 1>, a));
    else if (extra && bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<3, HMA_KV_BF16, 1>, a));
    else if (extra) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<3, HMA_KV_BFP8, 1>, a));
    else if (bf16 && probe == 0) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<0, HMA_KV_BF16, 1>, a));
    else if (bf16) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<1, HMA_KV_BF16, 1>, a));
    else if (probe == 0 && kq == 2) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<0, HMA_KV_BFP8, 2>, a));
    else if (probe == 0) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<0, HMA_KV_BFP8, 1>, a));
    else if (probe == 1) HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<1, HMA_KV_BFP8, 1>, a));
    else HMA_CUDA_OK(cudaLaunchKernelEx(&cfg, hma::attn_kernel<2, HMA_KV_BFP8, 1>, a));
    hma::count_launch();
    if (args_out) *args_out = a;
    if (ctas_out) *ctas_out = n_ctas;
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

extern "C" hma_status_t hma_decode_attention_multi(const hma_cache_t *cache, int32_t layer, const void *q, void *out,
                                                   int32_t out_dtype, const int32_t *block_table, int32_t max_pages_per_seq,
                                                   const int32_t *context_lens, int32_t batch, int32_t q_len, float sm_scale,
                                                   void *workspace, size_t workspace_bytes, void *stream)
{
    return launch_attention(cache, layer, q, out, out_dtype, block_table, max_pages_per_seq, context_lens, batch, sm_scale,
                            workspace, workspace_bytes, stream, 0, 0, nullptr, nullptr, q_len);
}

extern "C" size_t hma_decode_attention_plan_bytes(int32_t batch)
{
    return batch < 0 || batch > hma::kMaxBatch ? 0 : hma::plan_total_bytes(batch);
}

extern "C" hma_status_t hma_decode_attention_plan(const hma_cache_t *cache, const int32_t *block_table, int32_t max_pages_per_seq,
                                                  const int32_t *context_lens, int32_t batch, int32_t q_len, void *plan,
                                                  size_t plan_bytes, void *stream)
{
    if (q_len < 1 || batch < 0 || (int64_t)batch * q_len > hma::kMaxBatch) return batch < 0 || q_len < 1 ? HMA_ERR_INVALID_ARG : HMA_ERR_UNSUPPORTED_SHAPE;
    if (batch > 0 && plan_bytes < hma::plan_total_bytes(batch * q_len)) return HMA_ERR_WORKSPACE_TOO_SMALL;
    return launch_attention(cache, 0, nullptr, nullptr, HMA_OUT_BF16, block_table, max_pages_per_seq, context_lens, batch, 1.0f,
                            nullptr, 0, stream, 0, 0, nullptr, nullptr, q_len, nullptr, plan, 5);
}

extern "C" hma_status_t hma_decode_attention_planned(const hma_cache_t *cache, int32_t layer, const void *q, void *out,
                                                     int32_t out_dtype, const int32_t *block_table, int32_t max_pages_per_seq,
                                                     const int32_t *context_lens, int32_t batch, int32_t q_len, float sm_scale,
                                                     const void *plan, void *workspace, size_t workspace_bytes, void *stream)
{
    return launch_attention(cache, layer, q, out, out_dtype, block_table, max_pages_per_seq, context_lens, batch, sm_scale,
                            workspace, workspace_bytes, stream, 0, 0, nullptr, nullptr, q_len, nullptr, (void *)plan, 6);
}

static hma_status_t launch_mixed(const hma_cache_t *prefix, const hma_cache_t *tail, int32_t layer, const void *q, void *out,
                                 int32_t out_dtype, const int32_t *prefix_table, int32_t prefix_max_pages, const int32_t *prefix_lens,
                                 const int32_t *tail_table, int32_t tail_max_pages, const int32_t *tail_lens, int32_t batch,
                                 float sm_scale, const void *prefix_plan, const void *tail_plan, void *workspace,
                                 size_t workspace_bytes, void *stream)
{
    if (!prefix || !tail) return HMA_ERR_INVALID_ARG;
    if (prefix->desc.num_q_heads != tail->desc.num_q_heads || prefix->desc.num_kv_heads != tail->desc.num_kv_heads ||
        prefix->desc.key_layout != HMA_KEYS_AS_QUERIES || tail->desc.key_layout != HMA_KEYS_AS_QUERIES)
        return HMA_ERR_UNSUPPORTED_SHAPE;
    if (layer < 0 || layer >= tail->desc.num_layers) return HMA_ERR_INVALID_ARG;
    if (batch == 0) return HMA_OK;
    const size_t half = (hma_decode_attention_workspace_bytes(&prefix->desc, batch) + 255) & ~(size_t)255;
    if (!workspace) return HMA_ERR_INVALID_ARG;
    if (workspace_bytes < 2 * half) return HMA_ERR_WORKSPACE_TOO_SMALL;
    const int pm = prefix_plan ? 6 : 0;
    // The tail cache first: every finished segment leaves its unnormalised tile (vectors, maxima, sums) instead of an
    // output row.  Then the prefix cache, whose kernel folds that tile into the segment right before it writes it.  The
    // second kernel reads nothing of the first before a late grid-dependency wait: on the SMs that the first, usually
    // tiny, kernel leaves free it sets up and streams records at once.  (With plans: whatever made them ran before the
    // first kernel passed its own wait, so the second kernel may read its plan at once, too.)
    hma::AttnArgs ab;
    hma_status_t st = launch_attention(tail, layer, q, out, out_dtype, tail_table, tail_max_pages, tail_lens, batch, sm_scale,
                                       (uint8_t *)workspace + half, half, stream, 0, 1, &ab, nullptr, 1, nullptr, (void *)tail_plan, pm);
    if (st != HMA_OK) return st;
    return launch_attention(prefix, layer, q, out, out_dtype, prefix_table, prefix_max_pages, prefix_lens, batch, sm_scale,
                            workspace, half, stream, 0, 0, nullptr, nullptr, 1, ab.tails, (void *)prefix_plan, pm);
}

extern "C" hma_status_t hma_decode_attention_mixed(const hma_cache_t *prefix, const hma_cache_t *tail, int32_t layer,
                                                   const void *q, void *out, int32_t out_dtype,
                                                   const int32_t *prefix_table, int32_t prefix_max_pages, const int32_t *prefix_lens,
                                                   const int32_t *tail_table, int32_t tail_max_pages, const int32_t *tail_lens,
                                                   int32_t batch, float sm_scale, void *workspace, size_t workspace_bytes,
                                                   void *stream)
{
    return launch_mixed(prefix, tail, layer, q, out, out_dtype, prefix_table, prefix_max_pages, prefix_lens, tail_table, tail_max_pages,
                        tail_lens, batch, sm_scale, nullptr, nullptr, workspace, workspace_bytes, stream);
}

extern "C" hma_status_t hma_decode_attention_mixed_planned(const hma_cache_t *prefix, const hma_cache_t *tail, int32_t layer,
                                                           const void *q, void *out, int32_t out_dtype,
                                                           const int32_t *prefix_table, int32_t prefix_max_pages, const int32_t *prefix_lens,
                                                           const int32_t *tail_table, int32_t tail_max_pages, const int32_t *tail_lens,
                                                           int32_t batch, float sm_scale, const void *prefix_plan, const void *tail_plan,
                                                           void *workspace, size_t workspace_bytes, void *stream)
{
    if (!prefix_plan || !tail_plan) return HMA_ERR_INVALID_ARG;
    return launch_mixed(prefix, tail, layer, q, out, out_dtype, prefix_table, prefix_max_pages, prefix_lens, tail_table, tail_max_pages,
                        tail_lens, batch, sm_scale, prefix_plan, tail_plan, workspace, workspace_bytes, stream);
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

// ---------------------------------------------------------------- decode attention without a caller workspace
// Some callers cannot hand the library a workspace because they cannot allocate device memory at the point of
// the call: a serving loop whose memory pool was sized and frozen at start-up, a plug-in that runs inside
// another framework's allocator-free region, a host that has already given every byte to the KV cache.  For
// them the scratch lives in the library image itself.  Every GPU that loads the library carries the array
// below until the process exits.
namespace hma {
constexpr int kStaticMaxSegments = 512;       // batch * num_kv_heads
// counters | cum for up to 1000 rows | the per-CTA tiles and tail tiles of kStaticMaxSegments segments (the same sum as
// hma_decode_attention_workspace_bytes)
constexpr size_t kStaticWsBytes = (size_t)kMaxBatch * kMaxKvHeads * 4 + 8192 + (size_t)(2 * kMaxCtas + 2 * kStaticMaxSegments) * kTileFloats * 4;   // 5.8 MiB
static __device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];
static void *g_static_ws_ptr[kMaxDevices];    // device address of g_static_ws on each device, resolved on first use
}  // namespace hma

extern "C" size_t hma_decode_attention_static_limit_bytes(void) { return hma::kStaticWsBytes; }

extern "C" hma_status_t hma_decode_attention_static(const hma_cache_t *cache, int32_t layer, const void *q, void *out,
                                                    int32_t out_dtype, const int32_t *block_table, int32_t max_pages_per_seq,
                                                    const int32_t *context_lens, int32_t batch, float sm_scale, void *stream)
{
    if (!cache || batch < 0) return HMA_ERR_INVALID_ARG;
    if (hma_decode_attention_workspace_bytes(&cache->desc, batch) > hma::kStaticWsBytes) return HMA_ERR_STATIC_LIMIT;
    int dev = 0;
    HMA_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= hma::kMaxDevices) return HMA_ERR_STATIC_LIMIT;
    void *ws = nullptr;
    {
        static std::mutex static_lock;
        std::lock_guard<std::mutex> guard(static_lock);
        if (!hma::g_static_ws_ptr[dev]) {
            // In host code the array's name is only a handle: the device address has to be asked for, with the
            // device that will run the kernels current.
            void *p = nullptr;
            HMA_CUDA_OK(cudaGetSymbolAddress(&p, hma::g_static_ws));
            hma::g_static_ws_ptr[dev] = p;
        }
        ws = hma::g_static_ws_ptr[dev];
    }
    return launch_attention(cache, layer, q, out, out_dtype, block_table, max_pages_per_seq, context_lens, batch, sm_scale,
                            ws, hma::kStaticWsBytes, stream, 0);
}
