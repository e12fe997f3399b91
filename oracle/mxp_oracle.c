/*
 * MX+ CPU oracle -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, step-by-step restatement of the MXFP4 / MXFP4+ block format of
 * "MX+: Pushing the Limits of Microscaling Formats for Efficient LLM Serving"
 * (Sec. 2 Eq. 1, Sec. 4.1-4.2, Sec. 5 Eq. 3 and Eq. 4).  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it.  It shares no code,
 * table or constant with the CUDA library and must never be reached from the
 * product path.
 *
 * Arithmetic is done on doubles (every bf16 / fp32 input converts exactly).
 *
 * Pinned by tests (see tests/test_oracle_*.py): element table, scale, NBM and BM
 * rounding, flush rule, layout, Eq. 4 split, decode, fp64 GEMM; the MXFP6(+) / MXFP8(+)
 * functions at the end of the file likewise (element tables, casts against a library cast
 * and a closed form, BM grid, flush thresholds, 6-bit packing, round trips).
 * Parity unpinned: blocks holding Inf/NaN (the paper does not define them).
 *
 * Readings of the paper taken here (each is listed in the design notes):
 *   - rounding of the element cast: round to nearest, ties to the even code;
 *   - a BM whose scaled value rounds up to 8 keeps the scale and clamps to 7.5;
 *   - several equal maxima: the lowest index is the BM;
 *   - the sign bit of the input is kept even when the magnitude rounds to zero;
 *   - element 2j sits in the low nibble of byte j; three separate row-major planes;
 *   - the flush rule and the reserved scale byte 0 apply in plain MXFP4 mode too;
 *   - MX++ (Sec. 4.3): the scale byte keeps the BM's shared exponent, the three reserved
 *     bits of the index byte hold delta = shared_exp - shared_exp_new; "second-largest
 *     exponent" is the largest exponent among the non-zero NBM elements (the block
 *     without its BM); a block whose NBMs are all zero takes the lower clip (delta = 7).
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_MODE_MXFP4 0
#define ORACLE_MODE_MXFP4_PLUS 1
#define ORACLE_MODE_MXFP4_PP 2 /* MX++ (Sec. 4.3): NBMs get their own, smaller shared exponent */

/* Sec. 2: FP4 element = 1 sign, 2 exponent bits (bias 1), 1 mantissa bit,
 * implicit leading one, IEEE-like subnormals; emax = 3 - 1 = 2. */
#define EMAX 2
#define EXP_BIAS 1

static int g_threads = 1;

void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int oracle_get_threads(void) { return g_threads; }
int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Value of a 3-bit E2M1 magnitude code, from the definition of the type. */
double oracle_e2m1_value(int code)
{
    int e = (code >> 1) & 3;
    int m = code & 1;
    if (e == 0) /* subnormal: 2^(1-bias) * 0.m */
        return ldexp((double)m * 0.5, 1 - EXP_BIAS);
    return ldexp(1.0 + (double)m * 0.5, e - EXP_BIAS);
}

/* Nearest E2M1 magnitude to r >= 0.  Ties go to the even code.  Anything beyond
 * the largest magnitude saturates to it (Sec. 4.3 example: 7.92 -> 6.0). */
static int e2m1_nearest(double r)
{
    /* saturation first: beyond 2^53 the distances to 4 and to 6 round to the same double and
     * the search below could no longer tell them apart */
    if (r >= 6.0)
        return 7;
    int best = 0;
    double best_d = fabs(r - oracle_e2m1_value(0));
    for (int c = 1; c < 8; ++c) {
        double d = fabs(r - oracle_e2m1_value(c));
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    /* 7.0 is midway between 6 and the next binade value 8 (which has an even
     * mantissa): it rounds to 8 and then saturates, i.e. still code 7. */
    return best;
}

/* BM mantissa code in MX+ mode: v in [4, 8), grid 4 + m/2, m = 0..7 (E0M3 stored,
 * E2M3 effective with the implied exponent emax).  Round to nearest, ties to even
 * m; a value that would round up to 8 clamps to m = 7. */
static int bm_code(double v)
{
    double t = (v - 4.0) * 2.0; /* in [0, 8) */
    double fl = floor(t);
    double frac = t - fl;
    int m = (int)fl;
    if (frac > 0.5 || (frac == 0.5 && (m & 1)))
        m += 1;
    if (m > 7)
        m = 7;
    return m;
}

/* floor(log2(a)) for finite a > 0, exact. */
static int floor_log2(double a)
{
    int ex;
    (void)frexp(a, &ex); /* a = f * 2^ex, f in [0.5, 1) */
    return ex - 1;
}

/*
 * One block of k elements (k even, k <= 32; the format uses k = 32).
 * Outputs: k/2 nibble bytes, one scale byte, one index byte.
 */
static void quantize_block(const double *x, int k, int mode, uint8_t *nib,
                           uint8_t *scale, uint8_t *index)
{
    /* Sec. 3.2: BM = the absolute maximum of the block; first one wins. */
    double amax = 0.0;
    int bm = 0;
    int nonfinite = 0;
    for (int i = 0; i < k; ++i) {
        double a = fabs(x[i]);
        if (!(a <= 1.79769313486231570815e+308))
            nonfinite = 1;
        if (a > amax) {
            amax = a;
            bm = i;
        }
    }
    memset(nib, 0, (size_t)k / 2);
    if (nonfinite) { /* not defined by the paper: E8M0 NaN byte, data zero */
        *scale = 0xFF;
        *index = 0;
        return;
    }
    /* Sec. 4.1 flush rule: floor(log2 BM) <= -127 + emax -> whole block is zero,
     * signalled by the reserved biased scale 0. */
    if (amax == 0.0 || floor_log2(amax) <= -127 + EMAX) {
        *scale = 0;
        *index = 0;
        return;
    }
    /* Eq. 1: shared_exp = max floor(log2|x|) - emax; E8M0 bias 127. */
    int se = floor_log2(amax) - EMAX;
    *scale = (uint8_t)(se + 127);
    int plus = (mode == ORACLE_MODE_MXFP4_PLUS || mode == ORACLE_MODE_MXFP4_PP);
    int se_nbm = se;
    if (mode == ORACLE_MODE_MXFP4_PP) {
        /* Sec. 4.3: e = max2(floor(log2|x|)) - emax + 1 over the block without its BM,
         * shared_exp_new = CLIP(e, {shared_exp - 7, shared_exp}). */
        int have = 0, max2 = 0;
        for (int i = 0; i < k; ++i) {
            if (i == bm || x[i] == 0.0)
                continue;
            int ex = floor_log2(fabs(x[i]));
            if (!have || ex > max2) {
                max2 = ex;
                have = 1;
            }
        }
        se_nbm = se - 7; /* nothing but zeros beside the BM: the lower clip */
        if (have) {
            int e = max2 - EMAX + 1;
            se_nbm = e < se - 7 ? se - 7 : (e > se ? se : e);
        }
    }
    *index = (uint8_t)(plus ? (bm | ((se - se_nbm) << 5)) : 0);
    for (int i = 0; i < k; ++i) {
        int code;
        if (plus && i == bm)
            code = bm_code(ldexp(fabs(x[i]), -se)); /* Sec. 4.1: exponent bits reused as mantissa */
        else
            code = e2m1_nearest(ldexp(fabs(x[i]), -se_nbm)); /* exact scaling */
        int sign = signbit(x[i]) ? 1 : 0;
        uint8_t n = (uint8_t)((sign << 3) | code);
        if (i & 1)
            nib[i / 2] |= (uint8_t)(n << 4);
        else
            nib[i / 2] |= n;
    }
}

static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/*
 * src_kind: 0 = float32, 1 = bfloat16 bit patterns (uint16), 2 = float64.
 * Planes: nibbles rows*cols/2, scales rows*cols/k, bm_index rows*cols/k (written
 * in both modes; all zero in MXFP4 mode).  Returns 0, or -1 on a bad argument.
 */
int oracle_quantize(const void *src, int src_kind, int64_t rows, int64_t cols,
                    int64_t ld_src, int k, int mode, uint8_t *nibbles,
                    uint8_t *scales, uint8_t *bm_index)
{
    if (k < 2 || k > 32 || (k & 1) || cols % k != 0 || rows < 0 || cols < 0)
        return -1;
    if (mode != ORACLE_MODE_MXFP4 && mode != ORACLE_MODE_MXFP4_PLUS && mode != ORACLE_MODE_MXFP4_PP)
        return -1;
    int64_t bpr = cols / k;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < bpr; ++b) {
            double x[32];
            for (int i = 0; i < k; ++i) {
                int64_t off = r * ld_src + b * k + i;
                if (src_kind == 0)
                    x[i] = (double)((const float *)src)[off];
                else if (src_kind == 1)
                    x[i] = bf16_to_double(((const uint16_t *)src)[off]);
                else
                    x[i] = ((const double *)src)[off];
            }
            quantize_block(x, k, mode, nibbles + (r * cols + b * k) / 2,
                           scales + r * bpr + b, bm_index + r * bpr + b);
        }
    }
    return 0;
}

/* Eq. 3.  Scale byte 0 -> zeros (reserved encoding); 0xFF -> NaN (unpinned). */
int oracle_dequantize(const uint8_t *nibbles, const uint8_t *scales,
                      const uint8_t *bm_index, int64_t rows, int64_t cols, int k,
                      int mode, double *dst, int64_t ld_dst)
{
    if (k < 2 || k > 32 || (k & 1) || cols % k != 0)
        return -1;
    int64_t bpr = cols / k;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < bpr; ++b) {
            int sb = scales[r * bpr + b];
            int plus = (mode == ORACLE_MODE_MXFP4_PLUS || mode == ORACLE_MODE_MXFP4_PP);
            int bm = plus ? (bm_index[r * bpr + b] & 31) : -1;
            /* MX++: the NBMs' shared exponent lies delta below the BM's */
            int delta = (mode == ORACLE_MODE_MXFP4_PP) ? (bm_index[r * bpr + b] >> 5) : 0;
            for (int i = 0; i < k; ++i) {
                uint8_t byte = nibbles[(r * cols + b * k + i) / 2];
                int n = (i & 1) ? (byte >> 4) : (byte & 15);
                int s = n >> 3;
                int code = n & 7;
                double out;
                if (sb == 0) {
                    out = 0.0;
                } else if (sb == 0xFF) {
                    out = NAN;
                } else {
                    if (i == bm) /* "MX+ addition": 2^emax * 1.mmm */
                        out = ldexp(ldexp(1.0 + (double)code / 8.0, EMAX), sb - 127);
                    else
                        out = ldexp(oracle_e2m1_value(code), sb - 127 - delta);
                    if (s)
                        out = -out;
                }
                dst[r * ld_dst + b * k + i] = out;
            }
        }
    }
    return 0;
}

/* Eq. 4: BM = BM_H + BM_L on the scaled grid, um[3:0] = 1 m2 m1 m0.
 *   BM_H = 2^emax * um[3:2]     -> 4 or 6      (E2M1 magnitude codes 6, 7)
 *   BM_L = 2^(emax-2) * um[1:0] -> 0 .. 1.5    (E2M1 magnitude codes 0 .. 3)
 * Returns the two E2M1 magnitude codes. */
void oracle_bm_split(int m, int *code_h, int *code_l)
{
    int m2 = (m >> 2) & 1, m1 = (m >> 1) & 1, m0 = m & 1;
    /* um[3:2] read as the fixed-point number 1.m2; um[1:0] as m1.m0 */
    double h = ldexp(1.0 + (double)m2 * 0.5, EMAX);
    double l = ldexp((double)m1 + (double)m0 * 0.5, EMAX - 2);
    *code_h = e2m1_nearest(h);
    *code_l = e2m1_nearest(l);
}

/* ------------------------------------------------------------------------------------------
 * MXFP6 / MXFP6+ (E2M3 elements) and MXFP8 / MXFP8+ (E4M3 elements): Sec. 2 Table "Concrete
 * MX-compliant formats", Sec. 4.1 (BM re-encoding), Sec. 4.2 (layout).  Same scheme as MXFP4+:
 * shared_exp = floor(log2 BM) - emax with emax = 2 (E2M3) or 8 (E4M3); the BM keeps its sign
 * bit and spends every other bit on mantissa (E0M5: 4 + m/8, m = 0..31; E0M7: 256 + 2 m,
 * m = 0..127), its exponent being emax by construction.
 *
 * Readings taken here (the paper gives no worked example at these widths):
 *   - element casts round to nearest, ties to the even code, and saturate at the largest
 *     finite magnitude (7.5; 448: the E4M3 code S.1111.111 is NaN and never produced);
 *   - a BM whose scaled value rounds up to 2^(emax+1) clamps to the largest m;
 *   - flush rule with the format's own emax: floor(log2 BM) <= -127 + emax;
 *   - codes are produced one per byte here (sign in bit 5 resp. 7); oracle_pack6 gives the
 *     6-bit storage order: code i of a row in bits 6 i .. 6 i + 5 of the little-endian bit
 *     stream, so four codes fill three bytes.
 * ------------------------------------------------------------------------------------------ */
#define ORACLE_FMT_E2M3 6
#define ORACLE_FMT_E4M3 8

static int fmt_ebits(int fmt) { return fmt == ORACLE_FMT_E2M3 ? 2 : 4; }
static int fmt_mbits(int fmt) { return 3; (void)fmt; }
static int fmt_bias(int fmt) { return fmt == ORACLE_FMT_E2M3 ? 1 : 7; }
static int fmt_emax(int fmt) { return fmt == ORACLE_FMT_E2M3 ? 2 : 8; }
/* number of finite magnitude codes: all 32 for E2M3; E4M3 loses 1111.111 (NaN) */
static int fmt_ncodes(int fmt) { return fmt == ORACLE_FMT_E2M3 ? 32 : 127; }

/* Value of a magnitude code (exponent and mantissa bits, no sign), from the definition of
 * the type: subnormals 2^(1-bias) * 0.mmm, normals 2^(e-bias) * 1.mmm. */
double oracle_elem_value(int fmt, int code)
{
    int mb = fmt_mbits(fmt);
    int e = code >> mb;
    int m = code & ((1 << mb) - 1);
    (void)fmt_ebits;
    if (e == 0)
        return ldexp((double)m / (double)(1 << mb), 1 - fmt_bias(fmt));
    return ldexp(1.0 + (double)m / (double)(1 << mb), e - fmt_bias(fmt));
}

/* Nearest magnitude code to r >= 0 by exhaustive search; ties go to the even code; beyond
 * the largest finite magnitude the search returns that magnitude (saturation). */
static int elem_nearest(int fmt, double r)
{
    int n = fmt_ncodes(fmt);
    int best = 0;
    double best_d = fabs(r - oracle_elem_value(fmt, 0));
    for (int c = 1; c < n; ++c) {
        double d = fabs(r - oracle_elem_value(fmt, c));
        if (d < best_d || (d == best_d && (c & 1) == 0)) {
            best = c;
            best_d = d;
        }
    }
    return best;
}

/* BM mantissa: v in [2^emax, 2^(emax+1)), grid 2^emax * (1 + m / 2^mb) with mb = 5 or 7. */
static int bm_code_wide(int fmt, double v)
{
    int mb = fmt - 1; /* every bit but the sign */
    double t = (ldexp(v, -fmt_emax(fmt)) - 1.0) * (double)(1 << mb); /* in [0, 2^mb) */
    double fl = floor(t);
    double frac = t - fl;
    int m = (int)fl;
    if (frac > 0.5 || (frac == 0.5 && (m & 1)))
        m += 1;
    if (m > (1 << mb) - 1)
        m = (1 << mb) - 1;
    return m;
}

/* One block of k elements -> k code bytes (sign above the magnitude code), scale, index. */
static void quantize_block_wide(const double *x, int k, int fmt, int plus, uint8_t *codes,
                                uint8_t *scale, uint8_t *index)
{
    double amax = 0.0;
    int bm = 0, nonfinite = 0;
    int emax = fmt_emax(fmt);
    for (int i = 0; i < k; ++i) {
        double a = fabs(x[i]);
        if (!(a <= 1.79769313486231570815e+308))
            nonfinite = 1;
        if (a > amax) { /* Sec. 3.2: the absolute maximum, first one wins */
            amax = a;
            bm = i;
        }
    }
    if (k < 1 || k > 32)
        return;
    memset(codes, 0, (size_t)k);
    *index = 0;
    if (nonfinite) { /* not defined by the paper */
        *scale = 0xFF;
        return;
    }
    if (amax == 0.0 || floor_log2(amax) <= -127 + emax) { /* Sec. 4.1 flush rule */
        *scale = 0;
        return;
    }
    int se = floor_log2(amax) - emax; /* Eq. 1 */
    *scale = (uint8_t)(se + 127);
    if (plus)
        *index = (uint8_t)bm;
    for (int i = 0; i < k; ++i) {
        int code;
        if (plus && i == bm)
            code = bm_code_wide(fmt, ldexp(fabs(x[i]), -se));
        else
            code = elem_nearest(fmt, ldexp(fabs(x[i]), -se));
        int sign = signbit(x[i]) ? 1 : 0;
        codes[i] = (uint8_t)((sign << (fmt - 1)) | code);
    }
}

/* src_kind as in oracle_quantize; fmt 6 (E2M3) or 8 (E4M3); codes: rows*cols bytes. */
int oracle_quantize_wide(const void *src, int src_kind, int64_t rows, int64_t cols,
                         int64_t ld_src, int k, int fmt, int plus, uint8_t *codes,
                         uint8_t *scales, uint8_t *bm_index)
{
    if (k < 1 || k > 32 || cols % k != 0 || rows < 0 || cols < 0)
        return -1;
    if (fmt != ORACLE_FMT_E2M3 && fmt != ORACLE_FMT_E4M3)
        return -1;
    int64_t bpr = cols / k;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < bpr; ++b) {
            double x[32];
            for (int i = 0; i < k; ++i) {
                int64_t off = r * ld_src + b * k + i;
                if (src_kind == 0)
                    x[i] = (double)((const float *)src)[off];
                else if (src_kind == 1)
                    x[i] = bf16_to_double(((const uint16_t *)src)[off]);
                else
                    x[i] = ((const double *)src)[off];
            }
            quantize_block_wide(x, k, fmt, plus, codes + r * cols + b * k, scales + r * bpr + b,
                                bm_index + r * bpr + b);
        }
    }
    return 0;
}

/* Eq. 3 at the wider formats.  Scale byte 0 -> zeros; 0xFF -> NaN (unpinned). */
int oracle_dequantize_wide(const uint8_t *codes, const uint8_t *scales, const uint8_t *bm_index,
                           int64_t rows, int64_t cols, int k, int fmt, int plus, double *dst,
                           int64_t ld_dst)
{
    if (k < 1 || k > 32 || cols % k != 0)
        return -1;
    if (fmt != ORACLE_FMT_E2M3 && fmt != ORACLE_FMT_E4M3)
        return -1;
    int64_t bpr = cols / k;
    int mb = fmt - 1;
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < bpr; ++b) {
            int sb = scales[r * bpr + b];
            int bm = plus ? (bm_index[r * bpr + b] & 31) : -1;
            for (int i = 0; i < k; ++i) {
                int c = codes[r * cols + b * k + i];
                int s = (c >> mb) & 1;
                int mag = c & ((1 << mb) - 1);
                double out;
                if (sb == 0)
                    out = 0.0;
                else if (sb == 0xFF)
                    out = NAN;
                else {
                    if (i == bm) /* 2^emax * 1.m with every non-sign bit as mantissa */
                        out = ldexp(ldexp(1.0 + (double)mag / (double)(1 << mb), fmt_emax(fmt)), sb - 127);
                    else
                        out = ldexp(oracle_elem_value(fmt, mag), sb - 127);
                    if (s)
                        out = -out;
                }
                dst[r * ld_dst + b * k + i] = out;
            }
        }
    }
    return 0;
}

/* 6-bit storage order: code i in bits 6 i .. 6 i + 5 of the little-endian bit stream.
 * n codes (n % 4 == 0) -> 3 n / 4 bytes. */
void oracle_pack6(const uint8_t *codes, int64_t n, uint8_t *out)
{
    memset(out, 0, (size_t)(n / 4 * 3));
    for (int64_t i = 0; i < n; ++i) {
        int64_t bit = 6 * i;
        unsigned v = (unsigned)(codes[i] & 63) << (bit & 7);
        out[bit >> 3] |= (uint8_t)(v & 0xFF);
        if ((bit & 7) > 2)
            out[(bit >> 3) + 1] |= (uint8_t)(v >> 8);
    }
}

/* ------------------------------------------------------------------------------------------
 * NVFP4 / NVFP4+ (Sec. 8, "Applicability of MX+ to NVFP4"): E2M1 elements in blocks of 16
 * with an E4M3 block scale on top of one fp32 scale for the whole tensor.  The scale maps the
 * block's largest magnitude (the BM) onto the largest E2M1 magnitude, 6, so the BM's exponent
 * field is at its maximum and, as in MX+, can be spent on mantissa: NVFP4+ stores the BM as
 * sign + three mantissa bits, value 4 + m/2, and adds a 4-bit BM index per block.  Blocks whose
 * scale byte is 00000010b or smaller keep the plain NVFP4 form (their scale is too coarse for
 * the BM to land in [4, 8) reliably); their index nibble is 0.
 *
 * The passage says that the scale maps the BM as closely as possible onto the largest E2M1
 * magnitude and that elements are the inputs divided by the scale; it fixes neither the
 * rounding nor the layout.  Readings taken here (the definition, in real numbers):
 *       q = amax / (6 * ts);  scale byte = the E4M3 value nearest to q, ties to the even
 *       byte, saturating at 448;  d = value(scale byte) * ts  (exact);
 *       code_i = the E2M1 value nearest to abs(x_i) / d, ties to the even code, saturating at 6;
 *       the sign bit of the input is kept even when the magnitude rounds to zero;
 *   - scale byte 0 (amax too small for the tensor scale): all codes 0, index 0;
 *   - BM = first element with the largest magnitude; m = nearest integer to (v - 4) * 2, ties to
 *     the even m, with v = amax / d clamped to [4, 8] and m to 0..7 (v leaves [4, 8) only when
 *     the scale saturated);
 *   - element 2j in the low nibble of byte j; one scale byte per block; index nibbles two per
 *     byte, block 2j of a row in the low nibble (cols % 32 == 0 keeps rows byte aligned);
 *   - decode: x_i = +-E_i * d, E_i the E2M1 value or 4 + m/2 for the BM (exact; a consumer
 *     rounds it once to its output type).
 * Arithmetic: doubles.  6 * ts (26 bits), value(byte) * ts (28 bits) and every decoded value
 * (at most 32 bits) are exact.  The two quotients are rounded at 2^-53; that cannot move a
 * value across a rounding boundary or onto one: a quotient of a 24-bit by a 28-bit number (or
 * its boundary t, at most 5 bits, cross-multiplied: x vs t * d, at most 33 bits) is either
 * exactly the boundary -- then the division is exact -- or differs from it by more than
 * 2^-34 of its size.
 * Parity unpinned: Inf / NaN inputs, ts <= 0.
 * ------------------------------------------------------------------------------------------ */

/* E4M3 byte (sign 0) nearest to q >= 0, saturating: the search over the type's 127 finite
 * magnitudes used for MXFP8 elements above. */
int oracle_e4m3_round(double q) { return elem_nearest(ORACLE_FMT_E4M3, q); }

static void nvfp4_block(const double *x, double ts, int plus, uint8_t *nib, uint8_t *scale,
                        int *index)
{
    double amax = 0.0;
    int bm = 0;
    for (int i = 0; i < 16; ++i) {
        double a = fabs(x[i]);
        if (a > amax) {
            amax = a;
            bm = i;
        }
    }
    int sb = oracle_e4m3_round(amax / (6.0 * ts));
    *scale = (uint8_t)sb;
    *index = 0;
    memset(nib, 0, 8);
    if (sb == 0)
        return;
    double d = oracle_elem_value(ORACLE_FMT_E4M3, sb) * ts;
    int extend = plus && sb > 2;
    for (int i = 0; i < 16; ++i) {
        double v = fabs(x[i]) / d;
        int code;
        if (extend && i == bm)
            code = bm_code(fmin(fmax(v, 4.0), 8.0));
        else
            code = e2m1_nearest(v);
        if (signbit(x[i]))
            code |= 8;
        nib[i / 2] |= (uint8_t)(code << (4 * (i & 1)));
    }
    if (extend)
        *index = bm;
}

/* src_kind as in oracle_quantize (0 float32, 1 bfloat16 bits).  Planes: nibbles rows*cols/2,
 * scales rows*cols/16, bm_index rows*cols/32 (written in both modes; zero for NVFP4). */
int oracle_nvfp4_quantize(const void *src, int src_kind, int64_t rows, int64_t cols, float ts,
                          int plus, uint8_t *nibbles, uint8_t *scales, uint8_t *bm_index)
{
    if (rows < 0 || cols < 0 || cols % 32 != 0 || (src_kind != 0 && src_kind != 1))
        return -1;
    int64_t nb = cols / 16;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < nb; ++b) {
            double x[16];
            for (int i = 0; i < 16; ++i) {
                int64_t e = r * cols + b * 16 + i;
                x[i] = src_kind == 0 ? (double)((const float *)src)[e]
                                     : bf16_to_double(((const uint16_t *)src)[e]);
            }
            int idx;
            nvfp4_block(x, (double)ts, plus, nibbles + (r * nb + b) * 8, scales + r * nb + b,
                        &idx);
            uint8_t *ib = bm_index + (r * nb + b) / 2;
            if (b & 1)
                *ib = (uint8_t)((*ib & 0x0F) | (idx << 4));
            else
                *ib = (uint8_t)idx;
        }
    }
    return 0;
}

/* Decoded values as doubles (exact). */
int oracle_nvfp4_dequantize(const uint8_t *nibbles, const uint8_t *scales,
                            const uint8_t *bm_index, int64_t rows, int64_t cols, float ts,
                            int plus, double *out)
{
    if (rows < 0 || cols < 0 || cols % 32 != 0)
        return -1;
    int64_t nb = cols / 16;
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (int64_t r = 0; r < rows; ++r) {
        for (int64_t b = 0; b < nb; ++b) {
            int sb = scales[r * nb + b];
            double d = oracle_elem_value(ORACLE_FMT_E4M3, sb & 127) * (double)ts;
            int extend = plus && sb > 2;
            int bm = (bm_index[(r * nb + b) / 2] >> (4 * (b & 1))) & 15;
            for (int i = 0; i < 16; ++i) {
                int code = (nibbles[(r * nb + b) * 8 + i / 2] >> (4 * (i & 1))) & 15;
                double mag = (extend && i == bm) ? 4.0 + 0.5 * (code & 7)
                                                 : oracle_e2m1_value(code & 7);
                double v = mag * d;
                out[r * cols + b * 16 + i] = (code & 8) ? -v : v;
            }
        }
    }
    return 0;
}

/* D[m][n] = sum_k A[m][k] * B[n][k], fp64, k ascending.  A is M x K, B is N x K. */
void oracle_gemm_fp64(const double *A, int64_t lda, const double *B, int64_t ldb,
                      int64_t M, int64_t N, int64_t K, double *D, int64_t ldd)
{
#ifdef _OPENMP
#pragma omp parallel for num_threads(g_threads) schedule(static)
#endif
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int64_t kk = 0; kk < K; ++kk)
                acc += A[m * lda + kk] * B[n * ldb + kk];
            D[m * ldd + n] = acc;
        }
    }
}
