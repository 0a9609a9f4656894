/*
 * CPU oracle for BFP8 paged decode attention.  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 restatement of what the decode-side hot path of deferred
 * dequantization (paper section 3.3) computes.  It shares no code, header, table
 * or constant with the CUDA library; only tests, the smoke check and the CPU
 * baseline leg of the benchmark may call it.
 *
 * The paper fixes only "per-block shared exponent" and "7-bit mantissa" (section 3.3)
 * and a 32x32 tiled producer layout (sections 1 and 2.3).  Everything else below is the
 * reading this build takes:
 *   block     = 16 consecutive head-dim channels of one (token, kv head)
 *   E         = one byte, bias 127 (as in FP32 / BF16)
 *   element   = s<<7 | m, s = sign, m in [0,127], leading one explicit
 *   value     = (-1)^s * m * 2^(E-133)
 * Pins: tests/test_oracle_*.py (hand-worked blocks, exhaustive decode table, closed
 * forms of attention, float64 library attention, brute force).
 *
 * Build: gcc -O2 -fopenmp -shared -fPIC -o liboracle.so hma_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_BLOCK 16   /* elements per BFP8 block */
#define ORC_HEAD_DIM 128
#define ORC_BLOCKS_PER_ROW (ORC_HEAD_DIM / ORC_BLOCK)          /* 8 */
#define ORC_ROW_BYTES (ORC_BLOCKS_PER_ROW + ORC_HEAD_DIM)      /* 136: 8 exponents then 128 mantissas */
#define ORC_TILE_BYTES 1088                                    /* 64 exponents + 1024 mantissas */

/* ---------------------------------------------------------------- BF16 */

/* fp64 -> BF16 bit pattern, IEEE round-to-nearest-even, with subnormals, overflow to Inf. */
uint16_t orc_f64_to_bf16(double x)
{
    uint16_t sign = signbit(x) ? 0x8000u : 0u;
    if (isnan(x)) return 0x7FC0u;
    double a = fabs(x);
    if (a == 0.0) return sign;
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    int e = ilogb(a);                       /* floor(log2 a) */
    /* spacing of BF16 numbers around a: 2^(e-7) for normals, 2^-133 below 2^-126 */
    int qexp = (e < -126) ? -133 : e - 7;
    double n = ldexp(a, -qexp);             /* exact: scaling by a power of two */
    double r = nearbyint(n);                /* default rounding mode = ties to even */
    double v = ldexp(r, qexp);              /* the rounded value, exact in fp64 */
    if (v == 0.0) return sign;
    if (v >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7F80u);
    int ev = ilogb(v);
    if (ev < -126) {
        unsigned mant = (unsigned)ldexp(v, 133);      /* 1..127 */
        return (uint16_t)(sign | mant);
    }
    unsigned mant = (unsigned)(ldexp(v, 7 - ev)) - 128u;   /* 0..127 */
    unsigned ef = (unsigned)(ev + 127);
    return (uint16_t)(sign | (ef << 7) | mant);
}

/* BF16 bit pattern -> fp64 (exact). */
double orc_bf16_to_f64(uint16_t h)
{
    unsigned s = h >> 15, ef = (h >> 7) & 0xFFu, mant = h & 0x7Fu;
    double v;
    if (ef == 0xFF) v = mant ? NAN : INFINITY;
    else if (ef == 0) v = ldexp((double)mant, -133);
    else v = ldexp((double)(128u + mant), (int)ef - 134);
    return s ? -v : v;
}

/* ---------------------------------------------------------------- BFP8 decode (section 3.3, block-float decode) */

/* value of one element: (-1)^s * m * 2^(E-133) */
static double bfp8_value(uint8_t E, uint8_t b)
{
    double v = ldexp((double)(b & 0x7F), (int)E - 133);
    return (b & 0x80) ? -v : v;
}

void orc_bfp8_decode_f64(const uint8_t *exps, const uint8_t *mants, int64_t n_blocks, double *out)
{
    for (int64_t i = 0; i < n_blocks; ++i)
        for (int j = 0; j < ORC_BLOCK; ++j)
            out[i * ORC_BLOCK + j] = bfp8_value(exps[i], mants[i * ORC_BLOCK + j]);
}

/* decode to BF16 = the real value rounded to BF16 by RNE (always exact for E <= 254) */
void orc_bfp8_decode_bf16(const uint8_t *exps, const uint8_t *mants, int64_t n_blocks, uint16_t *out)
{
    for (int64_t i = 0; i < n_blocks; ++i)
        for (int j = 0; j < ORC_BLOCK; ++j)
            out[i * ORC_BLOCK + j] = orc_f64_to_bf16(bfp8_value(exps[i], mants[i * ORC_BLOCK + j]));
}

/* ---------------------------------------------------------------- BFP8 encode (producer side; used to make test inputs) */

/* FP32 -> BFP8.  Shared exponent = largest FP32 exponent field in the block; each
 * significand is shifted to that exponent and rounded to nearest, ties to even; a
 * carry to 128 saturates at 127; FP32 subnormals encode as zero; the sign bit is
 * always copied.  Returns the number of NaN/Inf inputs met (their bytes are 0). */
int64_t orc_bfp8_encode(const float *x, int64_t n_blocks, uint8_t *exps, uint8_t *mants)
{
    int64_t bad = 0;
    for (int64_t i = 0; i < n_blocks; ++i) {
        uint32_t bits[ORC_BLOCK];
        memcpy(bits, x + i * ORC_BLOCK, sizeof bits);
        unsigned E = 0;
        for (int j = 0; j < ORC_BLOCK; ++j) {
            unsigned e = (bits[j] >> 23) & 0xFFu;
            if (e == 0xFF) { ++bad; bits[j] &= 0x80000000u; e = 0; }
            if (e > E) E = e;
        }
        exps[i] = (uint8_t)E;
        for (int j = 0; j < ORC_BLOCK; ++j) {
            unsigned e = (bits[j] >> 23) & 0xFFu;
            unsigned s = bits[j] >> 31;
            unsigned q = 0;
            if (e != 0) {
                uint64_t sig = (1u << 23) | (bits[j] & 0x7FFFFFu);
                unsigned sh = 17u + (E - e);
                if (sh < 40) {
                    uint64_t quo = sig >> sh;
                    uint64_t rem = sig & ((1ull << sh) - 1);
                    uint64_t half = 1ull << (sh - 1);
                    if (rem > half || (rem == half && (quo & 1))) ++quo;
                    q = (unsigned)quo;
                }
                if (q > 127) q = 127;
            }
            mants[i * ORC_BLOCK + j] = (uint8_t)((s << 7) | q);
        }
    }
    return bad;
}

/* ---------------------------------------------------------------- wire layouts (ingest source formats) */

/* ROWMAJOR: [head][token][8 exponent bytes | 128 mantissa bytes].
 * TILE32:   [head][ceil(n/32) tile rows][4 tile cols][1088 B]; a tile covers 32 tokens x 32 channels
 *           as four 16x16 faces in the order (row-half, col-half) = (0,0),(0,1),(1,0),(1,1);
 *           bytes 0..63 hold exponents at face*16 + row%16, bytes 64.. hold mantissas at
 *           64 + face*256 + (row%16)*16 + col%16.  The paper says only "32x32 tiled" (section 1);
 *           the order inside a tile is this build's reading. */
static int64_t tile_rows(int64_t n_tokens) { return (n_tokens + 31) / 32; }

int64_t orc_tile32_bytes(int64_t n_tokens, int32_t heads)
{
    return (int64_t)heads * tile_rows(n_tokens) * 4 * ORC_TILE_BYTES;
}

void orc_pack_tile32(const uint8_t *rowmajor, int64_t n_tokens, int32_t heads, uint8_t *tiles)
{
    int64_t tr = tile_rows(n_tokens);
    memset(tiles, 0, (size_t)orc_tile32_bytes(n_tokens, heads));
    for (int32_t h = 0; h < heads; ++h)
        for (int64_t t = 0; t < n_tokens; ++t) {
            const uint8_t *row = rowmajor + ((int64_t)h * n_tokens + t) * ORC_ROW_BYTES;
            for (int c = 0; c < ORC_HEAD_DIM; ++c) {
                int64_t trow = t / 32; int tcol = c / 32;
                int r = (int)(t % 32), cc = c % 32;
                int face = (r / 16) * 2 + (cc / 16);
                uint8_t *tile = tiles + (((int64_t)h * tr + trow) * 4 + tcol) * ORC_TILE_BYTES;
                tile[64 + face * 256 + (r % 16) * 16 + (cc % 16)] = row[ORC_BLOCKS_PER_ROW + c];
                if (cc % 16 == 0) tile[face * 16 + (r % 16)] = row[c / 16];
            }
        }
}

void orc_unpack_tile32(const uint8_t *tiles, int64_t n_tokens, int32_t heads, uint8_t *rowmajor)
{
    int64_t tr = tile_rows(n_tokens);
    for (int32_t h = 0; h < heads; ++h)
        for (int64_t t = 0; t < n_tokens; ++t) {
            uint8_t *row = rowmajor + ((int64_t)h * n_tokens + t) * ORC_ROW_BYTES;
            for (int c = 0; c < ORC_HEAD_DIM; ++c) {
                int64_t trow = t / 32; int tcol = c / 32;
                int r = (int)(t % 32), cc = c % 32;
                int face = (r / 16) * 2 + (cc / 16);
                const uint8_t *tile = tiles + (((int64_t)h * tr + trow) * 4 + tcol) * ORC_TILE_BYTES;
                row[ORC_BLOCKS_PER_ROW + c] = tile[64 + face * 256 + (r % 16) * 16 + (cc % 16)];
                if (cc % 16 == 0) row[c / 16] = tile[face * 16 + (r % 16)];
            }
        }
}

/* ---------------------------------------------------------------- decode attention, fp64 */

/* One query token per sequence (decode).  For sequence b, q head h, kv head g = h / (Hq/Hkv),
 * T = ctx_lens[b]:  s_t = sm_scale * <q_h, K_t>,  p = softmax(s) (two passes, max subtracted),
 * o = sum_t p_t V_t.   K_t, V_t are the exact BFP8 values of the wire bytes.
 *
 *   q_bf16   [B][Hq][128]   BF16 bit patterns
 *   k_wire, v_wire          ROWMAJOR wire bytes; sequence b starts at byte wire_off[b] and is
 *                           laid out [Hkv][T_b][136]
 *   out_f64  [B][Hq][128]   fp64 result (may be NULL)
 *   out_bf16 [B][Hq][128]   the same rounded to BF16 by RNE (may be NULL)
 *   probs    if not NULL: fp64 softmax weights of sequence 0, head 0 (ctx_lens[0] values); for tests
 * T = 0 gives a row of zeros. */
/* Position, in the half-split head-dim order (rotary pairs (i, i+64)), of channel c of the interleaved order
 * (rotary pairs (2i, 2i+1)): the key re-layout of section 3.3. */
int32_t orc_half_split_index(int32_t c) { return (c >> 1) + 64 * (c & 1); }

/* keys_interleaved != 0: the wire keys are in interleaved rotary order while the queries are half-split, so key
 * channel c meets query channel orc_half_split_index(c). */
void orc_decode_attention(const uint16_t *q_bf16, const uint8_t *k_wire, const uint8_t *v_wire,
                          const int64_t *wire_off, const int32_t *ctx_lens,
                          int32_t B, int32_t Hq, int32_t Hkv, double sm_scale, int32_t keys_interleaved,
                          double *out_f64, uint16_t *out_bf16, double *probs)
{
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b)
        for (int32_t h = 0; h < Hq; ++h) {
            const int64_t T = ctx_lens[b];
            const int32_t g = h / G;
            double q[ORC_HEAD_DIM], o[ORC_HEAD_DIM];
            for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                q[d] = orc_bf16_to_f64(q_bf16[((int64_t)b * Hq + h) * ORC_HEAD_DIM + d]);
                o[d] = 0.0;
            }
            if (T > 0) {
                const uint8_t *kr = k_wire + wire_off[b] + (int64_t)g * T * ORC_ROW_BYTES;
                const uint8_t *vr = v_wire + wire_off[b] + (int64_t)g * T * ORC_ROW_BYTES;
                double *s = (double *)malloc((size_t)T * sizeof(double));
                double smax = -INFINITY;
                for (int64_t t = 0; t < T; ++t) {
                    const uint8_t *row = kr + t * ORC_ROW_BYTES;
                    double acc = 0.0;
                    for (int d = 0; d < ORC_HEAD_DIM; ++d)
                        acc += q[keys_interleaved ? orc_half_split_index(d) : d] * bfp8_value(row[d / ORC_BLOCK], row[ORC_BLOCKS_PER_ROW + d]);
                    s[t] = sm_scale * acc;
                    if (s[t] > smax) smax = s[t];
                }
                double denom = 0.0;
                for (int64_t t = 0; t < T; ++t) { s[t] = exp(s[t] - smax); denom += s[t]; }
                for (int64_t t = 0; t < T; ++t) {
                    const uint8_t *row = vr + t * ORC_ROW_BYTES;
                    double p = s[t] / denom;
                    if (probs && b == 0 && h == 0) probs[t] = p;
                    for (int d = 0; d < ORC_HEAD_DIM; ++d)
                        o[d] += p * bfp8_value(row[d / ORC_BLOCK], row[ORC_BLOCKS_PER_ROW + d]);
                }
                free(s);
            }
            for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                int64_t idx = ((int64_t)b * Hq + h) * ORC_HEAD_DIM + d;
                if (out_f64) out_f64[idx] = o[d];
                if (out_bf16) out_bf16[idx] = orc_f64_to_bf16(o[d]);
            }
        }
}

/* Decode attention over a context whose first prefix_lens[b] tokens are BFP8 wire bytes (as above) and whose
 * last tail_lens[b] tokens are plain BF16 values: KV made on the decode GPU, which the paper keeps in BF16
 * (section 3.1), appended to the prefix that arrived from the prefill accelerator.  One softmax over all tokens.
 *   k_tail, v_tail  BF16 bit patterns; sequence b starts at element tail_off[b], laid out [Hkv][tail_lens[b]][128]
 * Keys of both parts are in the queries' head-dim order. */
void orc_decode_attention_mixed(const uint16_t *q_bf16, const uint8_t *k_wire, const uint8_t *v_wire,
                                const int64_t *wire_off, const int32_t *prefix_lens,
                                const uint16_t *k_tail, const uint16_t *v_tail, const int64_t *tail_off,
                                const int32_t *tail_lens, int32_t B, int32_t Hq, int32_t Hkv, double sm_scale,
                                double *out_f64, uint16_t *out_bf16)
{
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b)
        for (int32_t h = 0; h < Hq; ++h) {
            const int64_t T = prefix_lens[b], S = tail_lens[b], N = T + S;
            const int32_t g = h / G;
            double q[ORC_HEAD_DIM], o[ORC_HEAD_DIM];
            for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                q[d] = orc_bf16_to_f64(q_bf16[((int64_t)b * Hq + h) * ORC_HEAD_DIM + d]);
                o[d] = 0.0;
            }
            if (N > 0) {
                const uint8_t *kr = k_wire + wire_off[b] + (int64_t)g * T * ORC_ROW_BYTES;
                const uint8_t *vr = v_wire + wire_off[b] + (int64_t)g * T * ORC_ROW_BYTES;
                const uint16_t *kt = k_tail + tail_off[b] + (int64_t)g * S * ORC_HEAD_DIM;
                const uint16_t *vt = v_tail + tail_off[b] + (int64_t)g * S * ORC_HEAD_DIM;
                double *s = (double *)malloc((size_t)N * sizeof(double));
                double smax = -INFINITY;
                for (int64_t t = 0; t < N; ++t) {
                    double acc = 0.0;
                    for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                        double kv = t < T ? bfp8_value(kr[t * ORC_ROW_BYTES + d / ORC_BLOCK], kr[t * ORC_ROW_BYTES + ORC_BLOCKS_PER_ROW + d])
                                          : orc_bf16_to_f64(kt[(t - T) * ORC_HEAD_DIM + d]);
                        acc += q[d] * kv;
                    }
                    s[t] = sm_scale * acc;
                    if (s[t] > smax) smax = s[t];
                }
                double denom = 0.0;
                for (int64_t t = 0; t < N; ++t) { s[t] = exp(s[t] - smax); denom += s[t]; }
                for (int64_t t = 0; t < N; ++t) {
                    double p = s[t] / denom;
                    for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                        double vv = t < T ? bfp8_value(vr[t * ORC_ROW_BYTES + d / ORC_BLOCK], vr[t * ORC_ROW_BYTES + ORC_BLOCKS_PER_ROW + d])
                                          : orc_bf16_to_f64(vt[(t - T) * ORC_HEAD_DIM + d]);
                        o[d] += p * vv;
                    }
                }
                free(s);
            }
            for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                int64_t idx = ((int64_t)b * Hq + h) * ORC_HEAD_DIM + d;
                if (out_f64) out_f64[idx] = o[d];
                if (out_bf16) out_bf16[idx] = orc_f64_to_bf16(o[d]);
            }
        }
}

/* Decode attention with several query tokens per sequence (speculative or chunked decode; the paper's decode loop,
 * section 1, generates one token per step, this is the widening named in its place).  The cache of sequence b holds
 * T = ctx_lens[b] tokens, the last q_len of which are the new tokens themselves; query i (0 .. q_len-1) is the i-th
 * new token and attends causally: to tokens t < T - (q_len - 1 - i).  A query that sees no token gives zeros.
 *   q_bf16   [B][q_len][Hq][128]
 *   out      [B][q_len][Hq][128]
 * Everything else as orc_decode_attention (keys in the queries' head-dim order). */
void orc_decode_attention_multi(const uint16_t *q_bf16, const uint8_t *k_wire, const uint8_t *v_wire,
                                const int64_t *wire_off, const int32_t *ctx_lens,
                                int32_t B, int32_t q_len, int32_t Hq, int32_t Hkv, double sm_scale,
                                double *out_f64, uint16_t *out_bf16)
{
    const int G = Hq / Hkv;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int32_t b = 0; b < B; ++b)
        for (int32_t i = 0; i < q_len; ++i)
            for (int32_t h = 0; h < Hq; ++h) {
                const int64_t T = ctx_lens[b];
                const int64_t visible = T - (q_len - 1 - i);       /* causal: the later new tokens are masked */
                const int32_t g = h / G;
                const int64_t row = ((int64_t)b * q_len + i) * Hq + h;
                double q[ORC_HEAD_DIM], o[ORC_HEAD_DIM];
                for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                    q[d] = orc_bf16_to_f64(q_bf16[row * ORC_HEAD_DIM + d]);
                    o[d] = 0.0;
                }
                if (visible > 0) {
                    const uint8_t *kr = k_wire + wire_off[b] + (int64_t)g * T * ORC_ROW_BYTES;
                    const uint8_t *vr = v_wire + wire_off[b] + (int64_t)g * T * ORC_ROW_BYTES;
                    double *s = (double *)malloc((size_t)T * sizeof(double));
                    double smax = -INFINITY;
                    for (int64_t t = 0; t < T; ++t) {
                        if (t >= visible) { s[t] = -INFINITY; continue; }
                        const uint8_t *kv = kr + t * ORC_ROW_BYTES;
                        double acc = 0.0;
                        for (int d = 0; d < ORC_HEAD_DIM; ++d) acc += q[d] * bfp8_value(kv[d / ORC_BLOCK], kv[ORC_BLOCKS_PER_ROW + d]);
                        s[t] = sm_scale * acc;
                        if (s[t] > smax) smax = s[t];
                    }
                    double denom = 0.0;
                    for (int64_t t = 0; t < T; ++t) { s[t] = exp(s[t] - smax); denom += s[t]; }      /* exp(-inf) = 0 for masked tokens */
                    for (int64_t t = 0; t < T; ++t) {
                        const uint8_t *vv = vr + t * ORC_ROW_BYTES;
                        double p = s[t] / denom;
                        for (int d = 0; d < ORC_HEAD_DIM; ++d) o[d] += p * bfp8_value(vv[d / ORC_BLOCK], vv[ORC_BLOCKS_PER_ROW + d]);
                    }
                    free(s);
                }
                for (int d = 0; d < ORC_HEAD_DIM; ++d) {
                    if (out_f64) out_f64[row * ORC_HEAD_DIM + d] = o[d];
                    if (out_bf16) out_bf16[row * ORC_HEAD_DIM + d] = orc_f64_to_bf16(o[d]);
                }
            }
}

int orc_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}
