/*
 * hma.h -- C ABI of the decode-side BFP8 KV path (deferred dequantization, paper section 3.3).
 *
 * The prefill accelerator ships each layer's KV cache as raw Blocked-FP8 bytes; the decode GPU
 * keeps them as raw BFP8 pages in HBM and rebuilds BF16 values inside the paged attention kernel
 * (paper Fig. 2 step 3 and section 3.3).  This library is that decode-side path:
 *
 *   hma_kv_ingest_layer     scatter one layer of arriving wire bytes into the paged cache
 *                           (consumer half of the compute-transfer pipeline, section 3.2)
 *   hma_decode_attention    GQA paged decode attention reading raw BFP8 pages (section 3.3);
 *                           hma_decode_attention_plan once per decode step + hma_decode_attention_planned
 *                           per layer is the same computation with its set-up done once
 *   hma_bfp8_dequant_bf16   one-shot BFP8 -> BF16 rebuild of a request's KV (the whole-request
 *                           reconstruction kernel of section 3.3)
 *
 * BFP8 as read here (section 3.3 fixes only that a block shares one exponent and that mantissas
 * have 7 bits):
 * a block is 16 consecutive head-dim channels of one (token, kv head); it has one exponent byte E
 * (bias 127) and 16 element bytes b = s<<7 | m;  value = (-1)^s * m * 2^(E-133).  Every such
 * value with E <= 254 is exactly a BF16 number.
 *
 * Conventions for every call
 *   - plain C; all pointers are raw addresses; "device" = CUDA device memory of the current
 *     device, "host" = ordinary host memory, "pinned" = page-locked host memory mapped into the
 *     device address space.  `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - ownership: the caller owns every buffer (cache layers, wire, Q, output, tables, workspace);
 *     the library makes one small device allocation per cache handle (a flag word and a copy of the
 *     layer pointers) and nothing else.
 *   - asynchrony: a call validates its arguments on the host, enqueues work on `stream`, and
 *     returns; no call synchronises the device except hma_error_flags.
 *   - errors: invalid arguments return a status and enqueue nothing.  Device-side anomalies never
 *     trap: a page id outside [0, num_pages) is skipped and a bit is set in the cache's flag word.
 *   - supported geometry: head_dim 128, 16 tokens per page, 16-element blocks,
 *     num_q_heads / num_kv_heads in 1..8, at most 64 kv heads.
 */
#ifndef HMA_H
#define HMA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HMA_OK = 0,
    HMA_ERR_INVALID_ARG = 1,
    HMA_ERR_UNSUPPORTED_SHAPE = 2,
    HMA_ERR_ALIGNMENT = 3,
    HMA_ERR_WORKSPACE_TOO_SMALL = 4,
    HMA_ERR_CUDA = 5,
    /* 6 is not used */
    HMA_ERR_STATIC_LIMIT = 7      /* the request does not fit the library's built-in scratch array */
} hma_status_t;

typedef enum { HMA_KV_BFP8 = 0, HMA_KV_BF16 = 1 } hma_kv_format_t;
typedef enum { HMA_WIRE_TILE32 = 0, HMA_WIRE_ROWMAJOR = 1, HMA_WIRE_BF16_ROWS = 2 } hma_wire_layout_t;
typedef enum { HMA_OUT_BF16 = 0, HMA_OUT_F32 = 1 } hma_out_dtype_t;
/* Head-dim order of the cached keys relative to the queries (section 3.3: the prefill accelerator writes post-RoPE
 * keys with rotary pairs interleaved, (2i, 2i+1); FlashAttention-style decoders use the half-split order, (i, i+64)).
 * HMA_KEYS_AS_QUERIES: cached keys are in the queries' order.  HMA_KEYS_INTERLEAVED: cached key channel c is the
 * half-split channel (c >> 1) + 64 * (c & 1); queries (and the output of hma_bfp8_dequant_bf16 for K) are half-split.
 * Values carry no rotary embedding and are never re-ordered. */
typedef enum { HMA_KEYS_AS_QUERIES = 0, HMA_KEYS_INTERLEAVED = 1 } hma_key_layout_t;

/* bits of the device flag word (hma_error_flags) */
#define HMA_FLAG_BAD_PAGE_ATTENTION 1u  /* block table entry outside [0, num_pages): page skipped */
#define HMA_FLAG_BAD_PAGE_INGEST    2u  /* page id outside [0, num_pages): page not written      */
#define HMA_FLAG_BAD_PAGE_DEQUANT   4u  /* page id outside [0, num_pages): output rows zeroed    */
#define HMA_FLAG_WAIT_TIMEOUT       8u  /* a bounded wait inside a kernel ran out                */
#define HMA_FLAG_BAD_VALUE_ENCODE  16u  /* hma_bfp8_encode_rows met NaN/Inf: encoded as zero      */
#define HMA_FLAG_EXPONENT_RANGE   32u  /* attention met a V block exponent above 250, or a softmax
                                          sum that is not finite (K exponents that overflow fp32)   */
#define HMA_FLAG_BAD_PLAN         64u  /* hma_decode_attention_planned was given a plan made for another launch shape
                                         (nothing was computed) or for other page counts (results void) */

typedef struct {
    int32_t num_layers;
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;      /* must be 128 */
    int32_t page_tokens;   /* must be 16  */
    int32_t bfp_block;     /* must be 16  */
    int64_t num_pages;     /* physical pages per layer */
    int32_t format;        /* hma_kv_format_t */
    int32_t key_layout;    /* hma_key_layout_t */
} hma_cache_desc_t;

typedef struct hma_cache hma_cache_t;   /* opaque; host-side metadata only */

/*
 * Paged KV cache holding the arriving bytes undecoded (paper Fig. 2 step 3).
 *
 * One layer is `num_pages` pages; a page holds 16 tokens of every kv head; the record of one
 * (page, kv head) is contiguous: K part then V part.
 *   HMA_KV_BFP8: record = 4352 B = K[128 exponent bytes | 2048 element bytes] V[128 | 2048].
 *                The bytes are the wire bytes unchanged; only their positions inside the record
 *                are permuted so that one 16-byte shared-memory load feeds one tensor-core
 *                operand fragment:
 *                  K exponent (tok, blk j)  at  (tok%8)*16 + (tok/8)*8 + j
 *                  K element  (tok, ch)     at  128 + ((tok/8) + 2*(j/4))*512 + ((tok%8)*4 + (ch%16)/4)*16
 *                                               + (j%4)*4 + ch%4,              j = ch/16
 *                  V exponent (tok, blk j)  at  2176 + ((tok%8)/2)*32 + j*4 + k
 *                  V element  (tok, ch)     at  2304 + (j/2)*512 + ((ch%8)*4 + (tok%8)/2)*16
 *                                               + ((j%2)*2 + (ch%16)/8)*4 + k
 *                                               with k = tok%2 + 2*(tok/8)
 *   HMA_KV_BF16: record = 8192 B = K[16 x 128 BF16] V[16 x 128 BF16], positions permuted likewise
 *                (the dequant-free baseline cache, section 3.3 last sentence).
 * hma_cache_layer_bytes returns num_pages * num_kv_heads * record size, or 0 for a bad descriptor.
 * The caller allocates each layer (device memory, 256-byte aligned) and passes the pointers;
 * the handle copies the pointer array.  Layers are not touched by create/destroy.
 */
size_t hma_cache_layer_bytes(const hma_cache_desc_t *desc);
hma_status_t hma_cache_create(const hma_cache_desc_t *desc, void *const *layer_ptrs /* host array of device pointers */,
                              hma_cache_t **out);
void hma_cache_destroy(hma_cache_t *cache);

/*
 * Ingest one layer of one request (sections 3.2 and 3.3: host-to-device copy and the
 * tiled -> paged layout conversion that merges per-chip shards).  Pure byte movement on a BFP8
 * cache; on a BF16 cache the same call decodes while scattering (the separate consumer-side dequantization pass
 * of section 2.3, used to fill the baseline cache with identical values).
 *
 *   k_wire, v_wire  device or pinned: raw wire bytes of heads [head_begin, head_begin+head_count)
 *                   for tokens [token_begin, token_begin+n_tokens), wire token 0 = token_begin.
 *                   HMA_WIRE_ROWMAJOR: [head][token][8 exponent bytes | 128 element bytes]
 *                   HMA_WIRE_TILE32:   [head][ceil(n_tokens/32)][4][1088 B]: a 32-token x 32-channel
 *                     tile = four 16x16 faces ordered (row half, column half); exponents at
 *                     face*16 + row%16, elements at 64 + face*256 + (row%16)*16 + col%16.
 *                   HMA_WIRE_BF16_ROWS (BF16 caches only): [head][token][128] plain BF16 values, KV that was
 *                     made on the decode GPU itself (the paper keeps decode in BF16, section 3.1).
 *                   Both pointers 16-byte aligned (HMA_WIRE_ROWMAJOR: 8-byte aligned is enough, which is
 *                   what hma_bfp8_encode_rows asks of its output).
 *   page_ids        device int32: page_ids[i] = physical page of the request's logical page
 *                   floor(token_begin/16) + i; ceil((token_begin%16 + n_tokens)/16) entries.
 * Token slots outside the range, other heads and other pages keep their bytes.  Pages being
 * written must not be read by a concurrent hma_decode_attention; order with stream events.
 */
hma_status_t hma_kv_ingest_layer(hma_cache_t *cache, int32_t layer,
                                 const void *k_wire, const void *v_wire, int32_t wire_layout,
                                 int32_t head_begin, int32_t head_count,
                                 const int32_t *page_ids, int64_t token_begin, int64_t n_tokens,
                                 void *stream);

/* The same for several producer shards in one launch (the shard merge of section 3.3; Table 2
 * runs Qwen3-32B prefill as one TP=4 group, so a layer arrives as four head ranges).  k_wires, v_wires,
 * head_begins, head_counts are host arrays of n_shards (1..8) entries; shard i carries heads
 * [head_begins[i], head_begins[i]+head_counts[i]) in the wire layout described above; head ranges must not
 * overlap.  Everything else as hma_kv_ingest_layer. */
hma_status_t hma_kv_ingest_layer_shards(hma_cache_t *cache, int32_t layer, int32_t n_shards,
                                        const void *const *k_wires, const void *const *v_wires, int32_t wire_layout,
                                        const int32_t *head_begins, const int32_t *head_counts,
                                        const int32_t *page_ids, int64_t token_begin, int64_t n_tokens, void *stream);

/* Every layer of the cache in one call, for a request whose bytes have all arrived (the counterpart of
 * hma_bfp8_rebuild_request): layer l's wire of shard s starts l * layer_stride_bytes after k_wires[s] / v_wires[s]
 * (a multiple of 16).  Same contents as num_layers calls of hma_kv_ingest_layer_shards; whole pages of a tiled wire into a
 * BFP8 cache go through one launch of the streaming kernel (a 36-MB layer alone is too short a launch to reach the
 * memory system's rate), everything else layer by layer. */
hma_status_t hma_kv_ingest_request_shards(hma_cache_t *cache, int32_t n_shards, const void *const *k_wires,
                                          const void *const *v_wires, size_t layer_stride_bytes, int32_t wire_layout,
                                          const int32_t *head_begins, const int32_t *head_counts, const int32_t *page_ids,
                                          int64_t token_begin, int64_t n_tokens, void *stream);

/*
 * Decode attention over block tables (section 3.3; one query token per sequence, section 1).
 * For sequence b, q head h, kv head g = h / (num_q_heads/num_kv_heads), T = context_lens[b]:
 *   s_t = sm_scale * <q[b][h], K_t>,  p = softmax_t(s),  out[b][h] = sum_t p_t V_t,  t < T,
 * K_t, V_t being the exact BFP8 values of the cached bytes.  T = 0 gives zeros.  Tokens >= T are
 * masked whatever bytes the last page holds; table entries past ceil(T/16) are never read.
 *
 *   q            device, BF16 [batch][num_q_heads][128], 16-byte aligned
 *   out          device, [batch][num_q_heads][128] BF16 or F32 per out_dtype
 *   block_table  device int32 [batch][max_pages_per_seq]
 *   context_lens device int32 [batch]; every entry <= max_pages_per_seq*16
 *   workspace    device, 256-byte aligned, >= hma_decode_attention_workspace_bytes(...) bytes.  It must have been
 *                zero-filled once (hma_decode_attention_workspace_init, or any memset to 0) before the first call that
 *                uses it: it holds one arrival counter per (sequence, kv head) on which the CTAs that share a segment
 *                meet.  Every call leaves the counters at zero again, so one workspace serves any number of calls, of
 *                any shape it is large enough for; the rest of it is clobbered.  A call that reports
 *                HMA_FLAG_WAIT_TIMEOUT may leave counters behind: zero the workspace again before its next use.
 *                Calls that may overlap on the GPU need a workspace each.
 *   batch        at most 1024 (HMA_ERR_UNSUPPORTED_SHAPE beyond)
 * Accuracy: fp32 accumulation.  Block exponents above 250 (values beyond 2^117) are outside the supported
 * range: the call still returns, HMA_FLAG_EXPONENT_RANGE is raised and the affected rows are not meaningful.
 * Launches: one kernel per call (the cross-split reduction happens inside it), with programmatic stream
 * serialisation; it waits on the grid dependency before it reads any input, so the usual stream order holds
 * whatever kernel precedes the call.  The first call on a device sets the kernels' shared-memory attributes.
 */
size_t hma_decode_attention_workspace_bytes(const hma_cache_desc_t *desc, int32_t batch);
/* Zero-fills a workspace on `stream` (see hma_decode_attention: needed once per workspace, before its first use). */
hma_status_t hma_decode_attention_workspace_init(void *workspace, size_t workspace_bytes, void *stream);
hma_status_t hma_decode_attention(const hma_cache_t *cache, int32_t layer,
                                  const void *q, void *out, int32_t out_dtype,
                                  const int32_t *block_table, int32_t max_pages_per_seq,
                                  const int32_t *context_lens, int32_t batch, float sm_scale,
                                  void *workspace, size_t workspace_bytes, void *stream);

/*
 * Decode attention with q_len query tokens per sequence (speculative or chunked decode; section 1 describes decode as
 * one token per step, this is the widening of it).  The cache of sequence b already holds all context_lens[b] tokens,
 * the last q_len of which are the new tokens themselves; query i (0 .. q_len-1) attends causally, to tokens
 * t < context_lens[b] - (q_len - 1 - i).  A query that sees no token gives a row of zeros.
 *   q, out       [batch][q_len][num_q_heads][128]
 *   workspace    >= hma_decode_attention_workspace_bytes(desc, batch * q_len); batch * q_len <= 1024
 * Everything else as hma_decode_attention, of which this is the q_len = 1 case.  With an even q_len on a BFP8 cache
 * two query tokens are handled per warp and share the unpacked K and V operands (about 1.2x per query token); otherwise
 * every query token costs what a sequence of hma_decode_attention costs.
 */
hma_status_t hma_decode_attention_multi(const hma_cache_t *cache, int32_t layer,
                                        const void *q, void *out, int32_t out_dtype,
                                        const int32_t *block_table, int32_t max_pages_per_seq,
                                        const int32_t *context_lens, int32_t batch, int32_t q_len, float sm_scale,
                                        void *workspace, size_t workspace_bytes, void *stream);

/*
 * hma_decode_attention for callers that cannot allocate.  (The paper has no counterpart: this exists for
 * the way the library gets embedded, not for the method.)  A decode loop that fixed its memory pool at
 * start-up, or code running where the host framework forbids allocation, has no workspace to pass; here
 * the scratch is a 5.8 MiB array that is part of the library image on every GPU that loads it
 * (hma_decode_attention_static_limit_bytes returns the exact size).  The call allocates and frees nothing.
 *
 *   - same arguments and results as hma_decode_attention, without the workspace pair; the outputs of the
 *     two entry points are identical for identical inputs.
 *   - limit: hma_decode_attention_workspace_bytes(desc, batch) must not exceed the array, which holds for
 *     batch * num_kv_heads <= 512 with batch <= 1000; anything larger returns HMA_ERR_STATIC_LIMIT and
 *     enqueues nothing.
 *   - the first call on each device looks up the array's device address (with that device current) and sets
 *     kernel attributes; make that first call outside any stream capture.
 *   - all calls on a device share the one array.  Its arrival counters start at zero (the loader zero-fills the
 *     array) and every call returns them to zero; nothing else in it is read before it is written.  Two calls
 *     that overlap on the GPU (different streams) race on it: keep such calls on one stream or order them with
 *     events.
 */
size_t hma_decode_attention_static_limit_bytes(void);
hma_status_t hma_decode_attention_static(const hma_cache_t *cache, int32_t layer,
                                         const void *q, void *out, int32_t out_dtype,
                                         const int32_t *block_table, int32_t max_pages_per_seq,
                                         const int32_t *context_lens, int32_t batch, float sm_scale,
                                         void *stream);

/* Same contract, computed by a plain one-CTA-per-(sequence, kv head) CUDA-core kernel that decodes
 * every element to BF16 first (the elementwise reconstruction section 3.3 compares against).
 * Needs no workspace.  Kept as an on-device cross-check of the fast kernel. */
hma_status_t hma_decode_attention_simple(const hma_cache_t *cache, int32_t layer,
                                         const void *q, void *out, int32_t out_dtype,
                                         const int32_t *block_table, int32_t max_pages_per_seq,
                                         const int32_t *context_lens, int32_t batch, float sm_scale,
                                         void *stream);

/*
 * Plan once, run per layer.  Everything hma_decode_attention works out from the context lengths and the block table
 * alone (page prefixes, the cut of the work list into per-warp record ranges, every warp's first record addresses,
 * every CTA's reduction plan) is the same for all layers of one decode step; it costs each call about 4 us before
 * its first record is even requested.  hma_decode_attention_plan runs that set-up once (one small launch) and writes it
 * to `plan`; hma_decode_attention_planned is hma_decode_attention_multi with the set-up read from the plan.
 *
 *   plan         device, 256-byte aligned, >= hma_decode_attention_plan_bytes(batch * q_len) bytes.  Valid for calls with
 *                the same cache geometry (format, head counts, num_pages), batch, q_len, max_pages_per_seq, on the same GPU
 *                model, while the block table holds what it held when the plan was made and every sequence still has
 *                the same number of pages: context lengths may grow inside their last pages (the lengths themselves are
 *                read at every call), so a plan lasts until a sequence starts a new page or the batch changes.  A plan
 *                made for another launch shape is detected and the call computes nothing; page counts that no longer
 *                match are detected while the call runs and its results are void; both raise HMA_FLAG_BAD_PLAN.  Changed
 *                table entries under unchanged page counts are not detectable.
 *   results      identical, bit for bit, to hma_decode_attention_multi with the same arguments, except when no sequence
 *                is longer than 8 pages: such a plan gives every (sequence, kv head) to one warp (nothing to combine at
 *                the end of the kernel), the softmax weights (FP16) are rounded against other
 *                running maxima and the sums are formed in another order: the results agree within the kernel's own error.
 * The plan call is ordinary stream work: later planned calls on the same stream see it without further synchronisation.
 */
size_t hma_decode_attention_plan_bytes(int32_t rows);
hma_status_t hma_decode_attention_plan(const hma_cache_t *cache, const int32_t *block_table, int32_t max_pages_per_seq,
                                       const int32_t *context_lens, int32_t batch, int32_t q_len, void *plan,
                                       size_t plan_bytes, void *stream);
hma_status_t hma_decode_attention_planned(const hma_cache_t *cache, int32_t layer, const void *q, void *out,
                                          int32_t out_dtype, const int32_t *block_table, int32_t max_pages_per_seq,
                                          const int32_t *context_lens, int32_t batch, int32_t q_len, float sm_scale,
                                          const void *plan, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Decode attention over two caches: the first prefix_lens[b] tokens of sequence b are pages of `prefix` (the BFP8
 * KV that arrived from the prefill accelerator), the next tail_lens[b] tokens are pages of `tail` (a BF16 cache
 * holding the KV of tokens generated since, which the paper's decode side produces in BF16, section 3.1; the
 * paper does not say where those live, this is one answer, hma_bfp8_encode_rows the other).  One softmax over
 * both.  Same q/out/sm_scale conventions as hma_decode_attention; both caches must have the same head counts and
 * HMA_KEYS_AS_QUERIES.  workspace: 2 * hma_decode_attention_workspace_bytes(desc, batch), rounded up to 256 each,
 * under the same zero-once contract as hma_decode_attention's (hma_decode_attention_workspace_init over all of it).
 * Two launches: the tail cache first, every finished (sequence, kv head) segment leaving its unnormalised tile (vectors,
 * maxima, sums) in the workspace's second half; then the prefix cache, whose kernel folds that tile into the segment
 * right before it writes it.  The second kernel waits for the first only when it first needs a tile, so it sets up
 * and streams records on every SM the first, usually tiny, kernel leaves free.
 */
hma_status_t hma_decode_attention_mixed(const hma_cache_t *prefix, const hma_cache_t *tail, int32_t layer,
                                        const void *q, void *out, int32_t out_dtype,
                                        const int32_t *prefix_table, int32_t prefix_max_pages, const int32_t *prefix_lens,
                                        const int32_t *tail_table, int32_t tail_max_pages, const int32_t *tail_lens,
                                        int32_t batch, float sm_scale, void *workspace, size_t workspace_bytes,
                                        void *stream);
/* The same with both launches' set-up taken from plans: prefix_plan from hma_decode_attention_plan(prefix, prefix_table,
 * prefix_max_pages, prefix_lens, batch, 1, ..), tail_plan likewise for the tail cache (two plan buffers).  Same results (to
 * the bit, or within the kernel's own error where a plan of short segments cuts the work differently); the rules for a plan's lifetime
 * are those of hma_decode_attention_planned. */
hma_status_t hma_decode_attention_mixed_planned(const hma_cache_t *prefix, const hma_cache_t *tail, int32_t layer,
                                                const void *q, void *out, int32_t out_dtype,
                                                const int32_t *prefix_table, int32_t prefix_max_pages, const int32_t *prefix_lens,
                                                const int32_t *tail_table, int32_t tail_max_pages, const int32_t *tail_lens,
                                                int32_t batch, float sm_scale, const void *prefix_plan, const void *tail_plan,
                                                void *workspace, size_t workspace_bytes, void *stream);

/*
 * One-shot reconstruction (section 3.3): tokens [token_begin, token_begin+n_tokens) of a request,
 * tensor `which` (0 = K, 1 = V), all kv heads -> row-major BF16 [n_tokens][num_kv_heads][128].
 * Bit-exact: each output is the BFP8 value rounded to BF16 (exact for E <= 254; E = 255 with
 * m >= 64 gives +-Inf; m = 0 keeps its sign).  page_ids as in hma_kv_ingest_layer.
 * On a BF16 cache the call is a gather.  out_bf16: device, 16-byte aligned.
 */
hma_status_t hma_bfp8_dequant_bf16(const hma_cache_t *cache, int32_t layer, int32_t which,
                                   const int32_t *page_ids, int64_t token_begin, int64_t n_tokens,
                                   void *out_bf16, void *stream);

/* The whole request in one launch (the whole-request reconstruction of section 3.3): every layer, K and V,
 * -> out_bf16 [num_layers][2 (K, V)][n_tokens][num_kv_heads][128] (device, 16-byte aligned), with the same decode,
 * key re-layout and page_ids convention as hma_bfp8_dequant_bf16. */
hma_status_t hma_bfp8_rebuild_request(const hma_cache_t *cache, const int32_t *page_ids, int64_t token_begin,
                                      int64_t n_tokens, void *out_bf16, void *stream);

/* The elementwise strawman that section 3.3 measures the fused rebuild against (72 ms vs 1.5 ms on the
 * paper's A100): same arguments and the same bits as hma_bfp8_dequant_bf16, computed one thread per element with byte
 * loads.  A comparison point for the benchmark, not a product path. */
hma_status_t hma_bfp8_dequant_bf16_naive(const hma_cache_t *cache, int32_t layer, int32_t which,
                                         const int32_t *page_ids, int64_t token_begin, int64_t n_tokens,
                                         void *out_bf16, void *stream);

/* Flat variant: n_blocks blocks, exps[i] with mants[16*i .. 16*i+15] -> out_bf16[16*i ..] (device pointers). */
hma_status_t hma_bfp8_dequant_blocks_bf16(const uint8_t *exps, const uint8_t *mants, int64_t n_blocks,
                                          void *out_bf16, void *stream);

/*
 * BFP8 encode on the GPU: n_rows rows of 128 channels (FP32, or BF16 when x_is_bf16 = 1; device, 16-byte aligned)
 * -> HMA_WIRE_ROWMAJOR rows of 136 bytes (device, 8-byte aligned), ready for hma_kv_ingest_layer.  This is the
 * format the prefill accelerator produces (sections 3.1, 3.3); the paper does not say how KV made on the decode GPU
 * (freshly generated tokens) joins a BFP8 cache, and this call is this library's answer: encode the token's K and V
 * rows here, then ingest them at token_begin = current length.  Shared exponent = largest FP32 exponent field of the
 * block; significands rounded to nearest-even onto 7 bits, a carry saturates at 127; FP32 subnormals encode as zero;
 * the sign is always copied.  NaN/Inf encode as zero and raise HMA_FLAG_BAD_VALUE_ENCODE in the cache's flag word
 * (`cache` is used for nothing else). */
hma_status_t hma_bfp8_encode_rows(const hma_cache_t *cache, const void *x, int32_t x_is_bf16, int64_t n_rows,
                                  void *wire_rowmajor, void *stream);

/* Copies the cache's device flag word to *host_out and clears it.  Synchronises `stream`. */
hma_status_t hma_error_flags(const hma_cache_t *cache, uint32_t *host_out, void *stream);

const char *hma_status_string(int32_t status);

/* Text of the CUDA runtime error behind the calling thread's most recent HMA_ERR_CUDA. */
const char *hma_last_cuda_error(void);

/* Number of kernels this library has launched in the calling process (for launch accounting). */
int64_t hma_launch_count(void);

/* ------------------------------------------------------------------------------------------------
 * Instrumentation.  Nothing below is on the decode path; the benchmark uses these entry points to
 * say which ceiling binds (the paper has no counterpart; section 2.2 only states that decode is
 * memory-bound).
 * ------------------------------------------------------------------------------------------------ */

/* Bandwidth probe: streams exactly the page records hma_decode_attention would read (same block
 * tables, same work split, same bulk-copy ring) and does no arithmetic and no output.  Its time is
 * the ceiling the attention kernel's memory pipeline can reach (section 2.2: decode is memory-bound).
 * BFP8 caches only.  Workspace as for hma_decode_attention. */
hma_status_t hma_kv_read_probe(const hma_cache_t *cache, int32_t layer, const int32_t *block_table,
                               int32_t max_pages_per_seq, const int32_t *context_lens, int32_t batch,
                               void *workspace, size_t workspace_bytes, void *stream);

/* Diagnostic twin of the probe: the arithmetic of every record on whatever shared memory holds, with no
 * loads and no output; its time is the attention kernel's instruction-issue floor.  The paper has no
 * counterpart; it exists so that the benchmark can say which of the two floors binds. */
hma_status_t hma_attention_alu_probe(const hma_cache_t *cache, int32_t layer, const int32_t *block_table,
                                     int32_t max_pages_per_seq, const int32_t *context_lens, int32_t batch,
                                     void *workspace, size_t workspace_bytes, void *stream);

/* A plain contiguous read of `bytes` bytes of device memory (16-byte aligned) with streaming loads: the simplest
 * read-only ceiling of the GPU's memory system, for comparison with hma_kv_read_probe.  `sink4` is a device word
 * the kernel may add to (it practically never does; it keeps the loads alive). */
hma_status_t hma_hbm_read_probe(const void *src, size_t bytes, void *sink4, void *stream);

/* A streaming read of read_bytes from `src` mixed with a streaming write of write_bytes to `dst` (both device,
 * 16-byte aligned, read_bytes <= write_bytes; the written data is the source stretched to the output's length): the
 * simplest kernel with the byte counts of a conversion that expands its input, for comparison with
 * hma_bfp8_rebuild_request (17 bytes in for 32 out) and the ingest (1:1). */
hma_status_t hma_hbm_copy_probe(const void *src, size_t read_bytes, void *dst, size_t write_bytes, void *stream);


#ifdef HMA_TRACE
/* Only in the instrumented build of the library (compiled with -DHMA_TRACE; the default build has neither this entry
 * point nor the per-warp time stamps).  Failure drill for the bounded waits inside the attention kernel: in the next
 * hma_decode_attention launch of this process, record number `record` of the launch's work list (records are counted
 * sequence by sequence, kv head by kv head, page by page) is announced to its arrival barrier as 16 bytes longer than
 * the copy that fills it, and waits give up after `spin_limit` polls.  The copy lands in full, the barrier never
 * completes, the waiting warp gives up, raises HMA_FLAG_WAIT_TIMEOUT and the kernel returns: nothing faults and nothing
 * hangs.  Outputs of the segments that CTA worked on are void. */
hma_status_t hma_trace_arm_timeout_drill(int64_t record, uint32_t spin_limit);
#endif

#ifdef __cplusplus
}
#endif
#endif /* HMA_H */
