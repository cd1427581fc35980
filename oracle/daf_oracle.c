/*
 * DAF activation compress / decompress -- CPU ORACLE (test infrastructure only).
 *
 * A plain, slow, step-by-step restatement of the hot path of the Dynamic
 * Activation Framework paper, written from the paper's definitions:
 *   - Eq. 1 (Sec. 2.3): scale = (max - min) / (2^b - 1), Q = round((X - min) / scale)
 *   - Sec. 2.3: stored activations are dequantized before the backward pass
 *   - Sec. 3.2: min / max reductions feed the scale and the importance metric
 *   - Sec. 3.4.1: greedy bit-width choice, candidates ordered by importance per
 *     unit of memory footprint, under a memory budget
 *   - Sec. 3.3 / Eq. 5: float <-> uint conversion through a power-of-two offset,
 *     and compact concatenation of the codes ("eight uint4 per uint32")
 * The paper works per activation tensor with one width per tensor; this
 * restatement applies the same formulas to contiguous groups of G elements,
 * chooses widths per window of groups, rounds stochastically from a Philox4x32-10
 * stream and packs LSB-first.  Each function names the passage it follows.
 *
 * This file is NOT part of the product: nothing in the CUDA library includes,
 * links or calls it, and it shares no code, table or constant generator with it.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Arithmetic: IEEE-754 binary32, round-to-nearest-even, subnormals honoured,
 * no contraction (build with -ffp-contract=off -fno-fast-math); fmaf() only
 * where a fused multiply-add is written.
 *
 * Parity pins (tests, CPU only): Philox against the published Random123
 * known-answer vectors; min/max, offsets and bit order against numpy library
 * routines; bit choice against a worked example, brute force and an
 * independently written heap greedy; codes against Eq. 1 evaluated in float64,
 * the exhaustive mean over all 2^15 rounding offsets, and worked vectors; decode
 * against closed forms.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_NONFINITE 2
#define ORACLE_ERR_BUDGET 3
#define ORACLE_ERR_CAPACITY 4

enum { ORACLE_F32 = 0, ORACLE_F16 = 1, ORACLE_BF16 = 2 };
enum { ORACLE_ROUND_STOCHASTIC = 0, ORACLE_ROUND_NEAREST = 1 };

static uint32_t f2u(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float u2f(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* ------------------------------------------------------------------ */
/* Widening of 16-bit inputs (exact) and narrowing of outputs (RNE).   */
/* ------------------------------------------------------------------ */

/* binary16 -> binary32, exact. */
float daf_oracle_half_to_float(uint16_t h)
{
    uint32_t sign = (uint32_t)(h >> 15) << 31;
    uint32_t e = (h >> 10) & 0x1F;
    uint32_t m = h & 0x3FF;
    if (e == 0) {
        /* zero or subnormal: value = m * 2^-24 */
        float v = (float)m * 0x1p-24f;          /* exact: m < 2^10 */
        return u2f(f2u(v) | sign);
    }
    if (e == 31) return u2f(sign | 0x7F800000u | (m << 13));
    return u2f(sign | ((e + 112) << 23) | (m << 13));
}

/* bfloat16 -> binary32, exact (bfloat16 is the upper half of binary32). */
float daf_oracle_bf16_to_float(uint16_t b) { return u2f((uint32_t)b << 16); }

/* binary32 -> bfloat16, round to nearest even. */
uint16_t daf_oracle_float_to_bf16(float f)
{
    uint32_t u = f2u(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40); /* NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* binary32 -> binary16, round to nearest even (overflow -> inf, gradual underflow). */
uint16_t daf_oracle_float_to_half(float f)
{
    uint32_t u = f2u(f);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t a = u & 0x7FFFFFFFu;
    if (a > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);        /* NaN */
    if (a >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u);       /* >= 65520 -> inf */
    if (a < 0x33000001u) return sign;                               /* <= 2^-25 -> 0 (tie to even) */
    int e = (int)(a >> 23) - 127;                                   /* unbiased exponent */
    uint32_t m = (a & 0x7FFFFFu) | 0x800000u;                       /* 24-bit significand */
    int shift = (e < -14) ? (13 + (-14 - e)) : 13;                  /* bits dropped */
    uint32_t kept = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t halfway = 1u << (shift - 1);
    if (rem > halfway || (rem == halfway && (kept & 1u))) kept++;
    uint32_t h;
    if (e < -14) h = kept;                                          /* subnormal (may carry into normal) */
    else h = (uint32_t)((e + 15) << 10) + (kept - 0x400u);          /* carry propagates into exponent */
    return (uint16_t)(sign | h);
}

/* Step 1 -- widen the input to binary32 (exact for fp16 / bf16). */
int daf_oracle_widen(int dtype, const void *in, uint64_t n, float *x)
{
    if (dtype == ORACLE_F32) { memcpy(x, in, n * 4); return ORACLE_OK; }
    const uint16_t *p = (const uint16_t *)in;
    if (dtype == ORACLE_F16) { for (uint64_t i = 0; i < n; i++) x[i] = daf_oracle_half_to_float(p[i]); return ORACLE_OK; }
    if (dtype == ORACLE_BF16) { for (uint64_t i = 0; i < n; i++) x[i] = daf_oracle_bf16_to_float(p[i]); return ORACLE_OK; }
    return ORACLE_ERR_ARG;
}

/* ------------------------------------------------------------------ */
/* Step 2 -- per-group min / max (Sec. 3.2: the reductions behind Eq. 1) */
/* ------------------------------------------------------------------ */

/* Total order on finite floats in which -0.0 < +0.0: map to an unsigned key. */
static uint32_t order_key(float f)
{
    uint32_t u = f2u(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

/* mn, mx per group; R = fl(mx - mn), set to 0 when below 2^-118 (degenerate group). */
int daf_oracle_stats(const float *x, uint64_t n, uint32_t G, float *mn, float *mx, float *R)
{
    if (G == 0 || n % G) return ORACLE_ERR_ARG;
    uint64_t ng = n / G;
    for (uint64_t g = 0; g < ng; g++) {
        const float *p = x + g * G;
        float lo = p[0], hi = p[0];
        for (uint32_t i = 0; i < G; i++) {
            if (!isfinite(p[i])) return ORACLE_ERR_NONFINITE;
            if (order_key(p[i]) < order_key(lo)) lo = p[i];
            if (order_key(p[i]) > order_key(hi)) hi = p[i];
        }
        float r = hi - lo;
        if (!isfinite(r)) return ORACLE_ERR_NONFINITE;
        if (r < 0x1p-118f) r = 0.0f;
        mn[g] = lo; mx[g] = hi; R[g] = r;
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
/* Step 3 -- greedy bit-width choice per window (Sec. 3.4.1)           */
/* ------------------------------------------------------------------ */

/* Allowed widths of a mask (bit b set <=> width b allowed), ascending. */
static int widths_of(uint32_t mask, int *S)
{
    int m = 0;
    for (int b = 1; b <= 8; b++) if (mask & (1u << b)) S[m++] = b;
    return m;
}

/* Importance-per-bit factor of the raise b_lo -> b_hi: a group of range R has
 * rounding-error variance proportional to R^2 / (2^b - 1)^2 (uniform quantizer,
 * Eq. 1); the factor is the square root of the variance removed per added bit,
 * evaluated in double and rounded once to binary32. */
float daf_oracle_raise_factor(int b_lo, int b_hi)
{
    double c_lo = 1.0 / ((ldexp(1.0, b_lo) - 1.0) * (ldexp(1.0, b_lo) - 1.0));
    double c_hi = 1.0 / ((ldexp(1.0, b_hi) - 1.0) * (ldexp(1.0, b_hi) - 1.0));
    return (float)sqrt((c_lo - c_hi) / (double)(b_hi - b_lo));
}

typedef struct { uint32_t key; uint32_t level; uint32_t group; uint32_t cost; } cand_t;

static int cand_cmp(const void *pa, const void *pb)
{
    const cand_t *a = (const cand_t *)pa, *b = (const cand_t *)pb;
    if (a->key != b->key) return (a->key > b->key) ? -1 : 1;      /* key descending   */
    if (a->level != b->level) return (a->level < b->level) ? -1 : 1; /* level ascending  */
    if (a->group != b->group) return (a->group < b->group) ? -1 : 1; /* group ascending  */
    return 0;
}

/* One window of n groups.  Every group starts at the smallest width; candidate
 * raises are sorted by importance per bit and accepted while the window's bit
 * budget T = floor(beta_q8 * n / 256) holds; the walk stops at the first raise
 * that does not fit. */
static int choose_bits_window(const float *R, uint32_t n, const int *S, int m,
                              uint32_t beta_q8, uint8_t *bits)
{
    uint64_t T = ((uint64_t)beta_q8 * n) >> 8;
    if (T < (uint64_t)S[0] * n) return ORACLE_ERR_BUDGET;
    uint64_t rem = T - (uint64_t)S[0] * n;
    uint32_t nc = n * (uint32_t)(m - 1);
    cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (nc ? nc : 1));
    uint8_t *level = (uint8_t *)calloc(n, 1);
    if (!c || !level) { free(c); free(level); return ORACLE_ERR_ARG; }
    uint32_t q = 0;
    for (uint32_t g = 0; g < n; g++)
        for (int k = 0; k + 1 < m; k++) {
            float v = daf_oracle_raise_factor(S[k], S[k + 1]);
            float key = R[g] * v;                       /* one binary32 multiply */
            c[q].key = f2u(key); c[q].level = (uint32_t)k; c[q].group = g;
            c[q].cost = (uint32_t)(S[k + 1] - S[k]); q++;
        }
    qsort(c, nc, sizeof(cand_t), cand_cmp);
    uint64_t cum = 0;
    for (uint32_t i = 0; i < nc; i++) {
        cum += c[i].cost;
        if (cum > rem) break;                           /* prefix rule: no skipping */
        level[c[i].group]++;
    }
    for (uint32_t g = 0; g < n; g++) bits[g] = (uint8_t)S[level[g]];
    free(c); free(level);
    return ORACLE_OK;
}

/* All windows: groups_per_window groups each, the last window may be shorter. */
int daf_oracle_choose_bits(const float *R, uint64_t n_groups, uint32_t groups_per_window,
                           uint32_t width_mask, uint32_t beta_q8, uint8_t *bits)
{
    int S[8];
    if (width_mask & ~0x116u) return ORACLE_ERR_ARG;    /* subset of {1,2,4,8} */
    int m = widths_of(width_mask, S);
    if (m == 0 || groups_per_window == 0) return ORACLE_ERR_ARG;
    for (uint64_t g0 = 0; g0 < n_groups; g0 += groups_per_window) {
        uint64_t n = n_groups - g0 < groups_per_window ? n_groups - g0 : groups_per_window;
        int rc = choose_bits_window(R + g0, (uint32_t)n, S, m, beta_q8, bits + g0);
        if (rc) return rc;
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
/* Step 4 -- group parameters (Eq. 1: scale = (max - min) / (2^b - 1)) */
/* ------------------------------------------------------------------ */
void daf_oracle_group_params(const float *R, const uint8_t *bits, uint64_t n_groups,
                             float *scale, float *inv)
{
    for (uint64_t g = 0; g < n_groups; g++) {
        float L = (float)((1u << bits[g]) - 1u);
        scale[g] = R[g] > 0.0f ? R[g] / L : 0.0f;       /* IEEE division */
        inv[g] = R[g] > 0.0f ? L / R[g] : 0.0f;         /* IEEE division */
    }
}

/* ------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al., "Parallel random numbers: as easy as  */
/* 1, 2, 3", SC'11): counter-based generator, 10 rounds.               */
/* ------------------------------------------------------------------ */
void daf_oracle_philox_round(uint32_t c[4], uint32_t k[2])
{
    uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
    uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
    uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
    uint32_t n0 = hi1 ^ c[1] ^ k[0];
    uint32_t n1 = lo1;
    uint32_t n2 = hi0 ^ c[3] ^ k[1];
    uint32_t n3 = lo0;
    c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
    k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u;           /* key bumped after each round */
}

void daf_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c[4] = { ctr[0], ctr[1], ctr[2], ctr[3] };
    uint32_t k[2] = { key[0], key[1] };
    for (int r = 0; r < 10; r++) daf_oracle_philox_round(c, k);
    memcpy(out, c, 16);
}

/* 15 random bits for global element index j: block j>>3, 16-bit lane j&7, top 15 bits of it. */
uint32_t daf_oracle_r15(uint64_t seed, uint64_t j)
{
    uint64_t blk = j >> 3;
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t o[4];
    daf_oracle_philox4x32_10(ctr, key, o);
    uint32_t e = (uint32_t)(j & 7u);
    uint32_t word = o[e >> 1];
    uint32_t half = (e & 1u) ? (word >> 16) : (word & 0xFFFFu);
    return half >> 1;
}

/* ------------------------------------------------------------------ */
/* Step 5 -- codes (Eq. 1 with the division folded into a multiply,    */
/* the float -> uint step done as in Eq. 5 read backwards)             */
/* ------------------------------------------------------------------ */
/* Core of step 5 with the 15-bit rounding offsets given: r15[i] in [0, 2^15). */
int daf_oracle_codes_r15(const float *x, uint64_t n, uint32_t G, const float *mn, const float *inv,
                         const uint8_t *bits, const uint16_t *r15, uint8_t *codes)
{
    if (G == 0 || n % G) return ORACLE_ERR_ARG;
    for (uint64_t i = 0; i < n; i++) {
        uint64_t g = i / G;
        uint32_t L = (1u << bits[g]) - 1u;
        float d = x[i] - mn[g];
        float s = fmaf(d, inv[g], 256.0f);              /* in [256, 512): ulp 2^-15 */
        uint32_t fixed = f2u(s) - 0x43800000u;          /* (s - 256) * 2^15 exactly  */
        uint32_t q = (fixed + (uint32_t)r15[i]) >> 15;
        codes[i] = (uint8_t)(q < L ? q : L);
    }
    return ORACLE_OK;
}

/* Step 5: offsets from the Philox stream (stochastic) or the constant 2^14 (nearest, half up). */
int daf_oracle_codes(const float *x, uint64_t n, uint32_t G, const float *mn, const float *inv,
                     const uint8_t *bits, int rounding, uint64_t seed, uint64_t elem_index_base,
                     uint8_t *codes)
{
    uint16_t *r = (uint16_t *)malloc((n ? n : 1) * 2);
    if (!r) return ORACLE_ERR_ARG;
    for (uint64_t i = 0; i < n; i++)
        r[i] = rounding == ORACLE_ROUND_NEAREST ? (uint16_t)0x4000u
                                                : (uint16_t)daf_oracle_r15(seed, elem_index_base + i);
    int rc = daf_oracle_codes_r15(x, n, G, mn, inv, bits, r, codes);
    free(r);
    return rc;
}

/* ------------------------------------------------------------------ */
/* Step 6 -- offsets and packing (Sec. 3.3: compact concatenation)     */
/* ------------------------------------------------------------------ */

/* Exclusive prefix sum of group byte lengths G*b/8; off has n_groups+1 entries. */
void daf_oracle_offsets(const uint8_t *bits, uint64_t n_groups, uint32_t G, uint64_t *off)
{
    uint64_t acc = 0;
    for (uint64_t g = 0; g < n_groups; g++) { off[g] = acc; acc += (uint64_t)G * bits[g] / 8u; }
    off[n_groups] = acc;
}

/* Bit t of code i (i within its group) is bit n = i*b + t of the group's stream;
 * stream bit n lives in byte off_g + (n >> 3), bit position n & 7. */
int daf_oracle_pack(const uint8_t *codes, uint64_t n, uint32_t G, const uint8_t *bits,
                    const uint64_t *off, uint8_t *packed, uint64_t capacity)
{
    if (G == 0 || n % G) return ORACLE_ERR_ARG;
    uint64_t ng = n / G;
    if (off[ng] > capacity) return ORACLE_ERR_CAPACITY;
    memset(packed, 0, off[ng]);
    for (uint64_t g = 0; g < ng; g++) {
        uint32_t b = bits[g];
        for (uint32_t i = 0; i < G; i++)
            for (uint32_t t = 0; t < b; t++) {
                uint64_t nb = (uint64_t)i * b + t;
                if ((codes[g * G + i] >> t) & 1u) packed[off[g] + (nb >> 3)] |= (uint8_t)(1u << (nb & 7u));
            }
    }
    return ORACLE_OK;
}

int daf_oracle_unpack(const uint8_t *packed, uint64_t n, uint32_t G, const uint8_t *bits,
                      const uint64_t *off, uint8_t *codes)
{
    if (G == 0 || n % G) return ORACLE_ERR_ARG;
    uint64_t ng = n / G;
    for (uint64_t g = 0; g < ng; g++) {
        uint32_t b = bits[g];
        for (uint32_t i = 0; i < G; i++) {
            uint32_t q = 0;
            for (uint32_t t = 0; t < b; t++) {
                uint64_t nb = (uint64_t)i * b + t;
                q |= (uint32_t)((packed[off[g] + (nb >> 3)] >> (nb & 7u)) & 1u) << t;
            }
            codes[g * G + i] = (uint8_t)q;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
/* Step 8 -- decode (Sec. 2.3: dequantize to the original precision)   */
/* ------------------------------------------------------------------ */
int daf_oracle_decode(const uint8_t *codes, uint64_t n, uint32_t G, const float *mn,
                      const float *scale, int dtype, void *out)
{
    if (G == 0 || n % G) return ORACLE_ERR_ARG;
    for (uint64_t i = 0; i < n; i++) {
        uint64_t g = i / G;
        float xh = fmaf((float)codes[i], scale[g], mn[g]);
        if (dtype == ORACLE_F32) ((float *)out)[i] = xh;
        else if (dtype == ORACLE_F16) ((uint16_t *)out)[i] = daf_oracle_float_to_half(xh);
        else if (dtype == ORACLE_BF16) ((uint16_t *)out)[i] = daf_oracle_float_to_bf16(xh);
        else return ORACLE_ERR_ARG;
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------ */
/* Whole path, the steps above in order.  A range of whole windows may */
/* be processed at a time so that callers can run windows on several   */
/* host threads (windows are independent once the widths are known):   */
/* that is a timing convenience of the caller, not part of the method. */
/* ------------------------------------------------------------------ */
typedef struct {
    int dtype;
    uint64_t numel;
    uint32_t group_size;
    uint32_t window_elems;
    uint32_t width_mask;
    float bit_budget;
    int rounding;
    uint64_t seed;
    uint64_t elem_index_base;
} oracle_params;

uint32_t daf_oracle_beta_q8(float bit_budget) { return (uint32_t)floorf(bit_budget * 256.0f); }

static size_t dtype_size(int dtype) { return dtype == ORACLE_F32 ? 4 : 2; }

/* Compress: fills bits / mn / scale (per group), window_offsets (n_windows+1,
 * bytes), packed (capacity bytes), and optionally mx / codes when non-NULL. */
int daf_oracle_compress(const oracle_params *p, const void *in, uint8_t *packed, uint64_t capacity,
                        uint8_t *bits, float *mn, float *scale, uint64_t *window_offsets,
                        float *mx_out, uint8_t *codes_out)
{
    uint32_t G = p->group_size, We = p->window_elems ? p->window_elems : 16384u;
    uint64_t n = p->numel;
    if (G == 0 || G % 32 || G > We || We % G || n == 0 || n % G) return ORACLE_ERR_ARG;
    uint64_t ng = n / G;
    uint32_t W = We / G;
    uint64_t nw = (ng + W - 1) / W;
    int rc = ORACLE_OK;
    float *x = (float *)malloc(n * 4);
    float *mx = (float *)malloc(ng * 4), *R = (float *)malloc(ng * 4), *inv = (float *)malloc(ng * 4);
    uint64_t *off = (uint64_t *)malloc((ng + 1) * 8);
    uint8_t *codes = (uint8_t *)malloc(n);
    if (!x || !mx || !R || !inv || !off || !codes) rc = ORACLE_ERR_ARG;
    if (!rc) rc = daf_oracle_widen(p->dtype, in, n, x);
    if (!rc) rc = daf_oracle_stats(x, n, G, mn, mx, R);
    if (!rc) rc = daf_oracle_choose_bits(R, ng, W, p->width_mask, daf_oracle_beta_q8(p->bit_budget), bits);
    if (!rc) {
        daf_oracle_group_params(R, bits, ng, scale, inv);
        rc = daf_oracle_codes(x, n, G, mn, inv, bits, p->rounding, p->seed, p->elem_index_base, codes);
    }
    if (!rc) {
        daf_oracle_offsets(bits, ng, G, off);
        for (uint64_t w = 0; w < nw; w++) window_offsets[w] = off[w * W];
        window_offsets[nw] = off[ng];
        rc = daf_oracle_pack(codes, n, G, bits, off, packed, capacity);
    }
    if (!rc && mx_out) memcpy(mx_out, mx, ng * 4);
    if (!rc && codes_out) memcpy(codes_out, codes, n);
    free(x); free(mx); free(R); free(inv); free(off); free(codes);
    return rc;
}

/* Decompress: per-group offsets are rebuilt from bits (they must agree with
 * window_offsets at every window boundary), then unpack and decode. */
int daf_oracle_decompress(const oracle_params *p, const uint8_t *packed, const uint8_t *bits,
                          const float *mn, const float *scale, const uint64_t *window_offsets,
                          void *out)
{
    uint32_t G = p->group_size, We = p->window_elems ? p->window_elems : 16384u;
    uint64_t n = p->numel;
    if (G == 0 || G % 32 || G > We || We % G || n == 0 || n % G) return ORACLE_ERR_ARG;
    uint64_t ng = n / G;
    uint32_t W = We / G;
    uint64_t nw = (ng + W - 1) / W;
    uint64_t *off = (uint64_t *)malloc((ng + 1) * 8);
    uint8_t *codes = (uint8_t *)malloc(n);
    int rc = (!off || !codes) ? ORACLE_ERR_ARG : ORACLE_OK;
    if (!rc) {
        daf_oracle_offsets(bits, ng, G, off);
        for (uint64_t w = 0; w < nw && !rc; w++) if (window_offsets[w] != off[w * W]) rc = ORACLE_ERR_ARG;
        if (!rc && window_offsets[nw] != off[ng]) rc = ORACLE_ERR_ARG;
    }
    if (!rc) rc = daf_oracle_unpack(packed, n, G, bits, off, codes);
    if (!rc) rc = daf_oracle_decode(codes, n, G, mn, scale, p->dtype, out);
    free(off); free(codes);
    (void)dtype_size;
    return rc;
}
