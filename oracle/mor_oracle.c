/*
 * mor_oracle.c -- plain, slow CPU statement of the MoR analyse-and-quantise pass.
 *
 * TEST INFRASTRUCTURE.  This file is the checker, not the product: only the tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.  It shares no code,
 * header, table or constant generator with the CUDA library and includes none of its
 * files; it is written from the paper alone:
 *
 *   - FP8 formats E4M3 / E5M2            Section 1 (bit split), Section 2 (ranges 2^-9..448,
 *                                         2^-16..57344), Section 3.2 (E5M2 min normal 2^-14)
 *   - Group Amax Mantissa scaling        Section 2, Algorithm 1
 *   - ordered fallback over formats      Section 3, Algorithm 2
 *   - tensor mean relative error         Section 3.1, Eq. 1-2  (threshold 4.5 %, Section 4.1.1)
 *   - block test E4M3 vs E5M2            Section 3.2, Eq. 3
 *   - E5M2 dynamic-range test            Section 3.2, Eq. 4
 *
 * The method is its own definition (it approximates nothing else), so the oracle takes
 * the algorithm's steps in the paper's order, one element at a time, with every sum in
 * double.  Two quantities are FP32 by the paper's wording (Section 2 calls the scaling factor
 * an FP32 number): the scale q_amax/amax and the scaled value x*scale that is then rounded
 * to FP8.  Both are formed here as one correctly rounded FP32 operation.
 *
 * FP8 encoding is done from the format definition: the table of finite values is built
 * from the bit fields, and a value is encoded by finding the nearest table entry, ties
 * to the entry with an even code, magnitudes above the largest finite entry saturating
 * to it.
 *
 * Readings where the paper is silent (each is restated next to the code that takes it):
 *   R1  formats are OCP E4M3 (bias 7, no infinities, S.1111.111 = NaN) and E5M2 (bias 15,
 *       IEEE-like): the only variants with the printed ranges.  Round to nearest even,
 *       saturate to the largest finite value.
 *   R2  mantissa()/exponent() in Algorithm 1 are the binary32 fraction and biased exponent
 *       fields; the E8M0 byte is that biased exponent; "- 1" acts on it.
 *   R3  Q(x) in Eq. 1-3 is the FP8 value de-scaled exactly; the ratio is formed in the
 *       scaled domain, |y - q| / |y| with y = fl32(x * scale).
 *   R4  a non-zero element whose FP8 value is zero contributes exactly 1.
 *   R5  all-zero block: exponent field 127; all-zero tensor: group mantissa 0;
 *       q_amax/amax overflowing FP32 is clamped to the largest finite FP32.
 *   R6  Eq. 3 accepts E4M3 on a tie (flag STRICT_TIES gives the literal '<').
 *   R7  min|b| in Eq. 4 runs over non-zero elements (flag RANGE_MIN_INCLUDES_ZERO gives
 *       the literal minimum); no non-zero element: the minimum is +infinity.
 *   R8  the E5M2 scale shares the group mantissa and uses the E4M3 block exponent + 7
 *       (57344 = 448 * 2^7), capped at 254.
 *   R9  NaN and +-infinity inputs are ignored by every amax, count and sum, are counted in
 *       n_nonfinite, encode as NaN -> 0x7F, +-inf -> +-largest finite, and force their
 *       block (and the tensor-level decision) to BF16.  PARITY UNPINNED: nothing in the
 *       paper fixes this case.
 *   R10 blocks that overhang the tensor edge are filled with absent elements, which take
 *       part in nothing.
 *   R11 fake quantisation (Section 4: "quantise, dequantise, de-scale", BF16 out): the FP8
 *       value divided by the scale in one binary32 division, then rounded to BF16 (nearest
 *       even).  A block that stays in BF16, and any NaN/inf element, is copied unchanged.  Where
 *       the decision is taken for the whole tensor (tensor-level criterion, per-tensor
 *       partition) the E4M3 values are written and the caller keeps the input when the tensor
 *       falls back.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_FMT_E4M3 = 0, ORC_FMT_E5M2 = 1, ORC_FMT_BF16 = 2 };
enum { ORC_CRIT_TENSOR_MEAN_REL = 0, ORC_CRIT_BLOCK_VS_E5M2 = 1, ORC_CRIT_BLOCK_MEAN_REL = 2 };
enum { ORC_SCALE_GAM = 0, ORC_SCALE_E8M0 = 1, ORC_SCALE_FP32_AMAX = 2 };
enum { ORC_FLAG_STRICT_TIES = 1u, ORC_FLAG_RANGE_MIN_INCLUDES_ZERO = 2u };

typedef struct {
    int64_t rows, cols, ld;          /* ld in elements                                   */
    int32_t block_rows, block_cols;  /* (0,0) = the whole tensor is one block             */
    int32_t n_formats;               /* 2: [E4M3, BF16]   3: [E4M3, E5M2, BF16]           */
    int32_t criterion;
    double  threshold;
    int32_t scale_mode;
    uint32_t flags;
    int32_t have_group_amax;         /* 0: compute it; 1: use group_amax as given         */
    float   group_amax;
} orc_cfg_t;

typedef struct {
    double  amax;            /* max |x| over finite elements of the block                 */
    double  min_abs_nz;      /* min |x| over finite non-zero elements, +inf if none       */
    int64_t nnz;             /* finite non-zero elements                                  */
    double  sum_rel_e4m3;    /* left side of Eq. 3                                        */
    double  sum_rel_e5m2;    /* right side of Eq. 3                                       */
    int64_t n_nonfinite;
    float   scale_e4m3;      /* FP32 scale applied before the E4M3 cast                   */
    float   scale_e5m2;
    int32_t exp_e4m3;        /* biased exponent byte of scale_e4m3                        */
    int32_t exp_e5m2;
    int32_t sel;             /* chosen format of the block                                */
    int32_t has_zero;        /* the block holds at least one (finite) zero                */
} orc_block_t;

typedef struct {
    double   sum_rel_e4m3;   /* numerator of Eq. 2 (sum over blocks, block order)         */
    int64_t  nnz;            /* n of Eq. 1                                                */
    double   mean_rel_e4m3;  /* error of Eq. 2, 0 when n = 0                              */
    float    group_amax;
    uint32_t group_mantissa; /* m_g of Algorithm 1: 23 fraction bits                      */
    int32_t  tensor_format;  /* Eq. 2 decision for the whole tensor                       */
    int64_t  n_blocks, n_e4m3, n_e5m2, n_bf16, n_nonfinite;
} orc_tensor_t;

/* ------------------------------------------------------------------ bit helpers ---- */

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* BF16 is the upper half of a binary32. */
float orc_bf16_to_float(uint16_t h) { return bits_f32((uint32_t)h << 16); }

static int bf16_is_nonfinite(uint16_t h) { return (h & 0x7F80u) == 0x7F80u; }
static int bf16_is_zero(uint16_t h) { return (h & 0x7FFFu) == 0; }

/* ------------------------------------------------------------------ FP8 formats ---- */
/* Reading R1.  E4M3: sign, 4 exponent bits (bias 7), 3 mantissa bits; exponent 15 with
 * mantissa 7 is NaN, every other code is finite (largest 1.75 * 2^8 = 448, smallest
 * positive 2^-3 * 2^-6 = 2^-9: the range printed in Section 2).  E5M2: sign, 5 exponent
 * bits (bias 15), 2 mantissa bits; exponent 31 is infinity (mantissa 0) or NaN (largest
 * finite 1.75 * 2^15 = 57344, smallest positive 2^-2 * 2^-14 = 2^-16, smallest normal
 * 2^-14: Sections 2 and 3.2). */

double orc_decode_e4m3(uint8_t c)
{
    int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else        v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -v : v;
}

double orc_decode_e5m2(uint8_t c)
{
    int s = c >> 7, e = (c >> 2) & 31, m = c & 3;
    double v;
    if (e == 31) return m == 0 ? (s ? -INFINITY : INFINITY) : NAN;
    if (e == 0) v = ldexp((double)m / 4.0, -14);
    else        v = ldexp(1.0 + (double)m / 4.0, e - 15);
    return s ? -v : v;
}

#define E4M3_NFINITE 127 /* codes 0x00..0x7E */
#define E5M2_NFINITE 124 /* codes 0x00..0x7B */

static double tab_e4m3[E4M3_NFINITE], tab_e5m2[E5M2_NFINITE];
static int tabs_ready = 0;

static void build_tables(void)
{
    if (tabs_ready) return;
    for (int c = 0; c < E4M3_NFINITE; ++c) tab_e4m3[c] = orc_decode_e4m3((uint8_t)c);
    for (int c = 0; c < E5M2_NFINITE; ++c) tab_e5m2[c] = orc_decode_e5m2((uint8_t)c);
    tabs_ready = 1;
}

/* Nearest finite value of the table, ties to the even code, saturating.  `exhaustive`
 * walks every code (the definition, used by the pins); otherwise the bracketing pair is
 * found by bisection of the same increasing table. */
static uint8_t encode_with_table(float y, const double* tab, int n, int exhaustive)
{
    build_tables();
    if (isnan(y)) return 0x7F;                       /* R9: one canonical NaN code      */
    uint8_t sign = (uint8_t)(signbit(y) ? 0x80 : 0x00);
    double a = fabs((double)y);
    int code;
    if (a >= tab[n - 1]) {
        code = n - 1;                                /* saturate (also +-infinity)      */
    } else if (exhaustive) {
        double best = INFINITY; code = 0;
        for (int c = 0; c < n; ++c) {
            double d = fabs(a - tab[c]);
            if (d < best || (d == best && (c & 1) == 0)) { best = d; code = c; }
        }
    } else {
        int lo = 0, hi = n - 1;                      /* tab[lo] <= a < tab[hi]          */
        while (hi - lo > 1) {
            int mid = (lo + hi) / 2;
            if (tab[mid] <= a) lo = mid; else hi = mid;
        }
        double dlo = a - tab[lo], dhi = tab[hi] - a; /* both exact in double            */
        if (dlo < dhi) code = lo;
        else if (dhi < dlo) code = hi;
        else code = (lo & 1) == 0 ? lo : hi;
    }
    return (uint8_t)(sign | code);
}

uint8_t orc_encode_e4m3(float y) { return encode_with_table(y, tab_e4m3, E4M3_NFINITE, 0); }
uint8_t orc_encode_e5m2(float y) { return encode_with_table(y, tab_e5m2, E5M2_NFINITE, 0); }
uint8_t orc_encode_e4m3_exhaustive(float y) { return encode_with_table(y, tab_e4m3, E4M3_NFINITE, 1); }
uint8_t orc_encode_e5m2_exhaustive(float y) { return encode_with_table(y, tab_e5m2, E5M2_NFINITE, 1); }

/* --------------------------------------------------------------- Algorithm 1 (GAM) -- */

#define Q_AMAX_E4M3 448.0f

/* Algorithm 1's FP32 scaling factor q_amax / amax: one binary32 division.  R5: an overflowing
 * quotient is replaced by the largest finite binary32. */
static float ideal_scale(float q_amax, float amax)
{
    float s = q_amax / amax;
    if (!(s <= 3.4028234663852886e38f)) s = 3.4028234663852886e38f;
    return s;
}

/* Algorithm 1, group part: s_g = q_amax / g_amax, m_g = mantissa(s_g).  R5: g_amax = 0
 * gives m_g = 0.  Scale mode E8M0 has no mantissa at all (m_g = 0). */
uint32_t orc_group_mantissa(float g_amax, int scale_mode)
{
    if (scale_mode != ORC_SCALE_GAM) return 0;
    if (!(g_amax > 0.0f)) return 0;
    return f32_bits(ideal_scale(Q_AMAX_E4M3, g_amax)) & 0x7FFFFFu;
}

/* Algorithm 1, block part.  s_b = q_amax / b_amax; keep exponent(s_b), lowered by one
 * when m_g > m_b so that b_amax * scale cannot exceed q_amax; the scale applied is the
 * shared mantissa joined to the block exponent.  Scale mode FP32_AMAX applies s_b itself
 * (the ablation's "per-block FP32 amax scaling", Section 4.1.2). */
void orc_block_scale(float b_amax, uint32_t m_g, int scale_mode,
                     float* scale_e4m3, int32_t* exp_e4m3, float* scale_e5m2, int32_t* exp_e5m2)
{
    uint32_t e, m;
    if (!(b_amax > 0.0f)) {                 /* R5: nothing to scale                    */
        e = 127; m = (scale_mode == ORC_SCALE_FP32_AMAX) ? 0 : m_g;
    } else {
        uint32_t sb = f32_bits(ideal_scale(Q_AMAX_E4M3, b_amax));
        uint32_t m_b = sb & 0x7FFFFFu;
        e = sb >> 23;                       /* s_b > 0: no sign bit                    */
        if (scale_mode == ORC_SCALE_FP32_AMAX) {
            m = m_b;
        } else {
            if (!(m_g <= m_b)) e -= 1;
            m = m_g;
        }
    }
    uint32_t e5 = e + 7 > 254 ? 254 : e + 7; /* R8                                     */
    *scale_e4m3 = bits_f32((e << 23) | m);
    *exp_e4m3 = (int32_t)e;
    *scale_e5m2 = bits_f32((e5 << 23) | m);
    *exp_e5m2 = (int32_t)e5;
}

/* ------------------------------------------------------- one element, one format ---- */

/* y = fl32(x * scale): the product of an 8-bit and a 24-bit significand is exact in
 * double, so the cast below is the single rounding to binary32. */
static float scale_value(float x, float scale) { return (float)((double)x * (double)scale); }

/* |y - q| / |y| in double; R4: q = 0 (which includes y = 0) gives 1. */
static double rel_err(float y, double q)
{
    if (q == 0.0) return 1.0;
    return fabs((double)y - q) / fabs((double)y);
}

/* ------------------------------------------------------------------- one block ------ */

/* Elements of block (bi, bj): rows [r0, r1) x cols [c0, c1) of the tensor (R10). */
static void block_bounds(const orc_cfg_t* cfg, int64_t bi, int64_t bj,
                         int64_t* r0, int64_t* r1, int64_t* c0, int64_t* c1)
{
    if (cfg->block_rows == 0 && cfg->block_cols == 0) {
        *r0 = 0; *r1 = cfg->rows; *c0 = 0; *c1 = cfg->cols;
        return;
    }
    *r0 = bi * cfg->block_rows; *r1 = *r0 + cfg->block_rows; if (*r1 > cfg->rows) *r1 = cfg->rows;
    *c0 = bj * cfg->block_cols; *c1 = *c0 + cfg->block_cols; if (*c1 > cfg->cols) *c1 = cfg->cols;
}

static void grid_dims(const orc_cfg_t* cfg, int64_t* nbr, int64_t* nbc)
{
    if (cfg->block_rows == 0 && cfg->block_cols == 0) {
        *nbr = (cfg->rows > 0 && cfg->cols > 0) ? 1 : 0; *nbc = *nbr;
        return;
    }
    *nbr = (cfg->rows + cfg->block_rows - 1) / cfg->block_rows;
    *nbc = (cfg->cols + cfg->block_cols - 1) / cfg->block_cols;
    if (cfg->rows == 0 || cfg->cols == 0) { *nbr = 0; *nbc = 0; }
}

int64_t orc_num_blocks(const orc_cfg_t* cfg)
{
    int64_t a, b; grid_dims(cfg, &a, &b); return a * b;
}

/* Block-level decision of Algorithm 2 for the per-block criteria (the tensor-level
 * criterion is decided after all blocks are known). */
static int32_t decide_block(const orc_cfg_t* cfg, const orc_block_t* b)
{
    if (b->n_nonfinite > 0) return ORC_FMT_BF16;                       /* R9 */
    if (cfg->criterion == ORC_CRIT_BLOCK_VS_E5M2) {
        /* M_1, Eq. 3.  R6: a tie keeps the preferred format unless STRICT_TIES. */
        int ok = (cfg->flags & ORC_FLAG_STRICT_TIES) ? (b->sum_rel_e4m3 < b->sum_rel_e5m2)
                                                     : (b->sum_rel_e4m3 <= b->sum_rel_e5m2);
        if (ok) return ORC_FMT_E4M3;
        if (cfg->n_formats == 3) {
            /* M_2, Eq. 4: max|b| / min|b| < 57344 / 2^-14, written without the division.
             * 57344 * 2^14 = 939524096; the product with a BF16 value is exact in double. */
            double mn = b->min_abs_nz;                                  /* R7 */
            if ((cfg->flags & ORC_FLAG_RANGE_MIN_INCLUDES_ZERO) && b->has_zero) mn = 0.0;
            if (b->amax < 939524096.0 * mn) return ORC_FMT_E5M2;
        }
        return ORC_FMT_BF16;
    }
    if (cfg->criterion == ORC_CRIT_BLOCK_MEAN_REL) {
        /* Eq. 1-2 on the block alone: mean over its non-zeros below the threshold. */
        double err = b->nnz > 0 ? b->sum_rel_e4m3 / (double)b->nnz : 0.0;
        return err < cfg->threshold ? ORC_FMT_E4M3 : ORC_FMT_BF16;
    }
    return ORC_FMT_E4M3; /* tensor criterion: placeholder, overwritten by the caller */
}

/* Steps of one block in the paper's order: block amax (Alg. 1), scale (Alg. 1), cast to
 * E4M3 and to E5M2, per-element relative errors and their sums (Eq. 1-3), range
 * statistics (Eq. 4), decision (Alg. 2).  Codes of both formats go to scratch so that
 * the caller can keep the ones of the chosen format. */
static void do_block(const orc_cfg_t* cfg, const uint16_t* x, int64_t bi, int64_t bj, uint32_t m_g,
                     orc_block_t* out, uint8_t* c43, uint8_t* c52 /* each (r1-r0)*(c1-c0) */)
{
    int64_t r0, r1, c0, c1;
    block_bounds(cfg, bi, bj, &r0, &r1, &c0, &c1);
    memset(out, 0, sizeof(*out));

    float amax = 0.0f; int has_zero = 0;
    for (int64_t r = r0; r < r1; ++r)
        for (int64_t c = c0; c < c1; ++c) {
            uint16_t h = x[r * cfg->ld + c];
            if (bf16_is_nonfinite(h)) { out->n_nonfinite++; continue; }   /* R9 */
            float a = fabsf(orc_bf16_to_float(h));
            if (a > amax) amax = a;
            if (bf16_is_zero(h)) has_zero = 1;
        }
    out->amax = amax;
    orc_block_scale(amax, m_g, cfg->scale_mode, &out->scale_e4m3, &out->exp_e4m3,
                    &out->scale_e5m2, &out->exp_e5m2);

    double mn = INFINITY, e43 = 0.0, e52 = 0.0; int64_t n = 0, k = 0;
    for (int64_t r = r0; r < r1; ++r)
        for (int64_t c = c0; c < c1; ++c, ++k) {
            uint16_t h = x[r * cfg->ld + c];
            float xv = orc_bf16_to_float(h);
            if (bf16_is_nonfinite(h)) {                                   /* R9 */
                uint8_t s = (uint8_t)((h >> 8) & 0x80);
                int is_nan = (h & 0x7F) != 0;
                c43[k] = is_nan ? 0x7F : (uint8_t)(s | 0x7E);
                c52[k] = is_nan ? 0x7F : (uint8_t)(s | 0x7B);
                continue;
            }
            float y43 = scale_value(xv, out->scale_e4m3);
            float y52 = scale_value(xv, out->scale_e5m2);
            c43[k] = orc_encode_e4m3(y43);
            c52[k] = orc_encode_e5m2(y52);
            if (bf16_is_zero(h)) continue;          /* sums of Eq. 1-3 run over x != 0 */
            n++;
            e43 += rel_err(y43, orc_decode_e4m3(c43[k]));
            e52 += rel_err(y52, orc_decode_e5m2(c52[k]));
            double a = fabs((double)xv);
            if (a < mn) mn = a;
        }
    out->nnz = n; out->sum_rel_e4m3 = e43; out->sum_rel_e5m2 = e52; out->min_abs_nz = mn;
    out->has_zero = has_zero;
    out->sel = decide_block(cfg, out);
}

/* -------------------------------------------------------------- whole tensor -------- */

/* g_amax of Algorithm 1 with the whole tensor as the single group (Section 2: "a single
 * group for the entire tensor"). */
float orc_tensor_amax(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld)
{
    float amax = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            uint16_t h = x[r * ld + c];
            if (bf16_is_nonfinite(h)) continue;                           /* R9 */
            float a = fabsf(orc_bf16_to_float(h));
            if (a > amax) amax = a;
        }
    return amax;
}

static void write_codes(const orc_cfg_t* cfg, int64_t bi, int64_t bj, const uint8_t* src,
                        uint8_t* codes, int64_t codes_ld)
{
    int64_t r0, r1, c0, c1, k = 0;
    block_bounds(cfg, bi, bj, &r0, &r1, &c0, &c1);
    for (int64_t r = r0; r < r1; ++r)
        for (int64_t c = c0; c < c1; ++c, ++k) codes[r * codes_ld + c] = src[k];
}

/* Analyse the blocks listed in `ids` (linear index bi * nbc + bj), or all blocks when
 * ids == NULL.  Outputs that are NULL are skipped.  `blocks` receives one record per
 * listed block.  Codes are written only for listed blocks.  With the tensor-level
 * criterion, and for `tensor` in general, all blocks must be listed (ids == NULL) for
 * the aggregate to be the tensor's; with a subset the aggregate covers the subset.
 * Returns 0, or -1 on an unsupported recipe. */
int orc_run_blocks(const orc_cfg_t* cfg, const uint16_t* x, const int64_t* ids, int64_t n_ids,
                   uint8_t* codes, int64_t codes_ld, uint8_t* scale_e8m0, uint8_t* sel,
                   float* scale_f32, orc_block_t* blocks, orc_tensor_t* tensor, int n_threads)
{
    if (cfg->n_formats != 2 && cfg->n_formats != 3) return -1;
    if (cfg->n_formats == 3 && cfg->criterion != ORC_CRIT_BLOCK_VS_E5M2) return -1;
    if ((cfg->block_rows == 0) != (cfg->block_cols == 0)) return -1;
    build_tables();

    int64_t nbr, nbc; grid_dims(cfg, &nbr, &nbc);
    int64_t total = nbr * nbc, n = ids ? n_ids : total;

    /* Algorithm 1: group amax first, then the shared mantissa. */
    float g_amax = cfg->have_group_amax ? cfg->group_amax
                                        : orc_tensor_amax(x, cfg->rows, cfg->cols, cfg->ld);
    uint32_t m_g = orc_group_mantissa(g_amax, cfg->scale_mode);

    int64_t bel = (cfg->block_rows == 0) ? cfg->rows * cfg->cols
                                         : (int64_t)cfg->block_rows * cfg->block_cols;
    orc_block_t* recs = blocks ? blocks : (orc_block_t*)malloc((size_t)(n > 0 ? n : 1) * sizeof(orc_block_t));
    if (!recs) return -2;

    (void)n_threads;
#ifdef _OPENMP
#pragma omp parallel num_threads(n_threads > 0 ? n_threads : 1)
#endif
    {
        uint8_t* c43 = (uint8_t*)malloc((size_t)(bel > 0 ? bel : 1));
        uint8_t* c52 = (uint8_t*)malloc((size_t)(bel > 0 ? bel : 1));
#ifdef _OPENMP
#pragma omp for schedule(static)
#endif
        for (int64_t i = 0; i < n; ++i) {
            int64_t id = ids ? ids[i] : i, bi = id / nbc, bj = id % nbc;
            do_block(cfg, x, bi, bj, m_g, &recs[i], c43, c52);
            /* Codes kept: the chosen FP8 format's; E4M3 codes for BF16 blocks (their data
             * stays in the input).  For the tensor criterion E4M3 is the only FP8 format. */
            if (codes) write_codes(cfg, bi, bj, recs[i].sel == ORC_FMT_E5M2 ? c52 : c43, codes, codes_ld);
        }
        free(c43); free(c52);
    }

    /* Eq. 1-2 over the whole tensor: local sums aggregated into the global error
     * (Section 3.1), in block order. */
    orc_tensor_t t; memset(&t, 0, sizeof(t));
    t.group_amax = g_amax; t.group_mantissa = m_g; t.n_blocks = n;
    for (int64_t i = 0; i < n; ++i) {
        t.sum_rel_e4m3 += recs[i].sum_rel_e4m3;
        t.nnz += recs[i].nnz;
        t.n_nonfinite += recs[i].n_nonfinite;
    }
    t.mean_rel_e4m3 = t.nnz > 0 ? t.sum_rel_e4m3 / (double)t.nnz : 0.0;
    t.tensor_format = (t.n_nonfinite == 0 && t.mean_rel_e4m3 < cfg->threshold) ? ORC_FMT_E4M3 : ORC_FMT_BF16;

    for (int64_t i = 0; i < n; ++i) {
        int64_t id = ids ? ids[i] : i;
        if (cfg->criterion == ORC_CRIT_TENSOR_MEAN_REL) recs[i].sel = t.tensor_format;
        int32_t s = recs[i].sel;
        if (s == ORC_FMT_E4M3) t.n_e4m3++; else if (s == ORC_FMT_E5M2) t.n_e5m2++; else t.n_bf16++;
        if (sel) sel[id] = (uint8_t)s;
        if (scale_e8m0) scale_e8m0[id] = (uint8_t)(s == ORC_FMT_E5M2 ? recs[i].exp_e5m2 : recs[i].exp_e4m3);
        if (scale_f32) scale_f32[id] = s == ORC_FMT_E5M2 ? recs[i].scale_e5m2 : recs[i].scale_e4m3;
    }
    if (tensor) *tensor = t;
    if (!blocks) free(recs);
    return 0;
}

/* The whole tensor. */
int orc_run(const orc_cfg_t* cfg, const uint16_t* x, uint8_t* codes, int64_t codes_ld,
            uint8_t* scale_e8m0, uint8_t* sel, float* scale_f32, orc_block_t* blocks,
            orc_tensor_t* tensor, int n_threads)
{
    return orc_run_blocks(cfg, x, NULL, 0, codes, codes_ld, scale_e8m0, sel, scale_f32, blocks, tensor, n_threads);
}

/* ------------------------------------------------------------- fake quantisation --- */

static uint16_t f32_to_bf16_rne(float f)
{
    uint32_t u = f32_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u);   /* NaN stays NaN */
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/* R11.  `sel` and `scale_f32` are the per-block results of orc_run (selected format and its
 * scale).  out has the layout of x with leading dimension out_ld. */
/* Section 4.1.3: the relative-error histogram has bins of 0.5 %: bin k holds errors in
 * [0.5 k %, 0.5 (k+1) %), the twelfth and last bin everything from 5.5 % up.  One tensor and
 * mini-batch contribute one count. */
int orc_error_bin(double mean_rel)
{
    int k = 0;
    while (k < 11 && mean_rel >= 0.005 * (double)(k + 1)) ++k;
    return k;
}

int orc_fake_quant(const orc_cfg_t* cfg, const uint16_t* x, const uint8_t* sel, const float* scale_f32,
                   uint16_t* out, int64_t out_ld)
{
    build_tables();
    int64_t nbr, nbc; grid_dims(cfg, &nbr, &nbc);
    int whole = cfg->criterion == ORC_CRIT_TENSOR_MEAN_REL || (cfg->block_rows == 0 && cfg->block_cols == 0);
    for (int64_t bi = 0; bi < nbr; ++bi)
        for (int64_t bj = 0; bj < nbc; ++bj) {
            int64_t r0, r1, c0, c1, id = bi * nbc + bj;
            block_bounds(cfg, bi, bj, &r0, &r1, &c0, &c1);
            int fmt = whole ? ORC_FMT_E4M3 : sel[id];
            float s = scale_f32[id];
            for (int64_t r = r0; r < r1; ++r)
                for (int64_t c = c0; c < c1; ++c) {
                    uint16_t h = x[r * cfg->ld + c];
                    if (fmt == ORC_FMT_BF16 || bf16_is_nonfinite(h)) { out[r * out_ld + c] = h; continue; }
                    float y = scale_value(orc_bf16_to_float(h), s);
                    float q = fmt == ORC_FMT_E5M2 ? (float)orc_decode_e5m2(orc_encode_e5m2(y))
                                                  : (float)orc_decode_e4m3(orc_encode_e4m3(y));
                    out[r * out_ld + c] = f32_to_bf16_rne(q / s);      /* one binary32 division */
                }
        }
    return 0;
}

/* Element-level helpers exported for the pins. */
float orc_scale_value(float x, float scale) { return scale_value(x, scale); }
uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }
double orc_rel_err_e4m3(float y) { return rel_err(y, orc_decode_e4m3(orc_encode_e4m3(y))); }
double orc_rel_err_e5m2(float y) { return rel_err(y, orc_decode_e5m2(orc_encode_e5m2(y))); }
int orc_sizeof_cfg(void) { return (int)sizeof(orc_cfg_t); }
int orc_sizeof_block(void) { return (int)sizeof(orc_block_t); }
int orc_sizeof_tensor(void) { return (int)sizeof(orc_tensor_t); }
