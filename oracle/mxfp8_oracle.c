/*
 * MXFP8 conversion oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, scalar CPU statement of what the MXFP8 conversion of the paper
 * "Recipes for Pre-training LLMs with MXFP8" computes.  It exists so that tests,
 * the smoke check and the benchmark's CPU-baseline leg can compare the CUDA
 * library against something written independently from the paper.  It shares no
 * code, header, table or constant generator with the CUDA path and nothing in
 * the product may call it.
 *
 * Every value is carried in double precision: an FP32 input times a power of
 * two in 2^-127..2^127 is always exact in binary64, so the only rounding is the
 * single round-to-nearest-even onto the FP8 grid that the paper asks for.
 *
 * Parity status of each function (what pins it, in tests/test_oracle_*.py):
 *   orc_fp8_decode / orc_fp8_encode   pinned: Table 1 constants, all 256 codes,
 *                                     midpoints, an independent library cast.
 *   orc_scale_byte (paper, ocp)       pinned: exact-rational brute force of the
 *                                     definition, no-overflow invariant (Sec. 3.3),
 *                                     hand-worked blocks in tests/golden/.
 *   orc_quantize / orc_dequantize     pinned: the above plus metamorphic
 *                                     invariants and exhaustive ldexp decode.
 *   NaN / Inf handling                parity unpinned: Sec. 3.3 only says that
 *                                     "special care" is taken; the reading used
 *                                     here is stated at orc_block_amax below.
 *
 * Build: gcc -O2 -std=c11 -fPIC -shared (never -ffast-math).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#define ORC_E4M3 0
#define ORC_E5M2 1
#define ORC_RULE_PAPER 0
#define ORC_RULE_OCP 1
#define ORC_ROW 1
#define ORC_COL 2

/* Element formats (Table 1 and Sec. 2): E4M3 is 1-4-3 with one NaN pattern and
 * no infinity, max 1.75*2^8, min subnormal 2^-9; E5M2 is 1-5-2 with IEEE
 * specials, max 1.75*2^15, min subnormal 2^-16.
 * The 6- and 4-bit element formats of Table 1 (MXFP6: E2M3, E3M2; MXFP4: E2M1)
 * have a sign bit, no infinity and no NaN: E2M3 (bias 1) max 1.875*2^2, min
 * subnormal 2^-3; E3M2 (bias 3) max 1.75*2^4, min subnormal 2^-4 (Table 1
 * prints 2^-3 there, which no 1-3-2 format with that maximum has; the bias-3
 * format of the OCP MX specification the paper builds on is taken); E2M1
 * (bias 1) max 1.5*2^2, min subnormal 2^-1.  A code sits in the low bits of
 * its byte. */
#define ORC_E2M3 3
#define ORC_E3M2 4
#define ORC_E2M1 5
typedef struct {
    int ebits;       /* exponent bits                                  */
    int mbits;       /* mantissa bits                                  */
    int bias;        /* exponent bias                                  */
    int emin;        /* exponent of the smallest normal                */
    int emax;        /* exponent of the largest normal (of destmax)    */
    double destmax;  /* largest finite magnitude                       */
    int max_code;    /* code of +destmax                               */
    int nan_code;    /* the NaN code this oracle emits                 */
} orc_fmt;

static orc_fmt orc_format(int elem)
{
    orc_fmt f;
    if (elem == ORC_E5M2) {
        f.ebits = 5; f.mbits = 2; f.bias = 15; f.emin = -14; f.emax = 15;
        f.destmax = 57344.0; f.max_code = 0x7B; f.nan_code = 0x7F;
    } else if (elem == ORC_E2M3) {
        f.ebits = 2; f.mbits = 3; f.bias = 1; f.emin = 0; f.emax = 2;
        f.destmax = 7.5; f.max_code = 0x1F; f.nan_code = 0x1F;     /* no NaN: see orc_fp8_encode */
    } else if (elem == ORC_E3M2) {
        f.ebits = 3; f.mbits = 2; f.bias = 3; f.emin = -2; f.emax = 4;
        f.destmax = 28.0; f.max_code = 0x1F; f.nan_code = 0x1F;
    } else if (elem == ORC_E2M1) {
        f.ebits = 2; f.mbits = 1; f.bias = 1; f.emin = 0; f.emax = 2;
        f.destmax = 6.0; f.max_code = 0x07; f.nan_code = 0x07;
    } else {
        f.ebits = 4; f.mbits = 3; f.bias = 7; f.emin = -6; f.emax = 8;
        f.destmax = 448.0; f.max_code = 0x7E; f.nan_code = 0x7F;
    }
    return f;
}

/* Decoded value of one FP8 code (Sec. 2, Table 1). */
double orc_fp8_decode(int code, int elem)
{
    orc_fmt f = orc_format(elem);
    int sbit = f.ebits + f.mbits;                         /* position of the sign bit */
    int sign = (code >> sbit) & 1;
    int mag = code & ((1 << sbit) - 1);                   /* bits above the sign are ignored */
    int efield = mag >> f.mbits;
    int mfield = mag & ((1 << f.mbits) - 1);
    double v;
    if (elem == ORC_E4M3) {
        if (mag == 0x7F) return NAN;                      /* the single NaN pattern */
    } else if (elem == ORC_E5M2) {
        if (efield == 31) return mfield ? NAN : (sign ? -INFINITY : INFINITY);
    }                                                     /* the 6- and 4-bit formats have no specials */
    if (efield == 0)
        v = ldexp((double)mfield, f.emin - f.mbits);      /* subnormal: 0.m * 2^emin */
    else
        v = ldexp((double)((1 << f.mbits) + mfield), efield - f.bias - f.mbits);
    return sign ? -v : v;
}

/* Quantize_to_fp8 (Sec. 3.3, App. A.2): round-to-nearest-ties-to-even onto the
 * element grid, subnormals included, then saturate: magnitudes above destmax
 * (infinity too) become +-destmax.  NaN stays NaN where the format has one; the
 * 6- and 4-bit formats have none and the paper does not say what a NaN element
 * becomes there: this oracle emits +destmax (the saturating hardware convert's
 * choice), parity unpinned for that case.  The sign of zero and of values that
 * round to zero is kept. */
int orc_fp8_encode(double x, int elem)
{
    orc_fmt f = orc_format(elem);
    int sign, code, ex;
    double a, k;
    if (isnan(x)) return f.nan_code;
    sign = signbit(x) ? (1 << (f.ebits + f.mbits)) : 0;
    a = fabs(x);
    if (a >= f.destmax) return sign | f.max_code;
    if (a < ldexp(1.0, f.emin)) {
        /* subnormal range: multiples of 2^(emin-mbits); k == 2^mbits is the
         * smallest normal, whose code is exactly k as well */
        k = rint(ldexp(a, -(f.emin - f.mbits)));         /* rint: ties to even */
        return sign | (int)k;
    }
    (void)frexp(a, &ex);
    ex -= 1;                                             /* a = 1.xxx * 2^ex */
    k = rint(ldexp(a, -(ex - f.mbits)));                 /* in [2^mbits, 2^(mbits+1)] */
    if (k == (double)(1 << (f.mbits + 1))) { ex += 1; k = (double)(1 << f.mbits); }
    code = ((ex + f.bias) << f.mbits) | ((int)k - (1 << f.mbits));
    if (code > f.max_code) code = f.max_code;            /* saturate after rounding */
    return sign | code;
}

/* Block amax (Sec. 3.3): max |V_i| over the block.  Reading taken for the
 * "special care" the paper leaves open: NaN and +-Inf elements are left out of
 * the maximum so the block's scale stays finite and the other elements keep
 * their values; a block without a finite non-zero element has amax 0. */
static float orc_block_amax(const float *v, ptrdiff_t stride, int n)
{
    float amax = 0.0f;
    for (int i = 0; i < n; i++) {
        float a = fabsf(v[(ptrdiff_t)i * stride]);
        if (isfinite(a) && a > amax) amax = a;
    }
    return amax;
}

/* UE8M0 scale byte b; the scale is X = 2^(b-127) (Sec. 2, Algorithm 1).
 *
 * paper rule (Algorithm 1 with the order of App. A.1): X is amax/destmax
 *   rounded UP to a power of two, never below 2^-127: the smallest n in
 *   [-127,127] with amax <= destmax * 2^n.  Evaluated by direct search with
 *   exact binary64 comparisons, not with log2 (App. A.1 warns that a rounded
 *   log2 gives wrong ceilings).
 * ocp rule (the OCP MX v1.0 suggestion the paper compares against, which
 *   "rounds down"): n = floor(log2(amax)) - emax, clamped to [-127,127];
 *   amax == 0 gives -127.
 */
int orc_scale_byte(float amax, int elem, int rule)
{
    orc_fmt f = orc_format(elem);
    double a = (double)amax;
    int n;
    if (rule == ORC_RULE_PAPER) {
        for (n = -127; n < 127; n++)
            if (a <= ldexp(f.destmax, n)) break;
    } else {
        if (a == 0.0) {
            n = -127;
        } else {
            int ex;
            (void)frexp(a, &ex);                         /* a = f * 2^ex, f in [0.5,1) */
            n = (ex - 1) - f.emax;
            if (n < -127) n = -127;
            if (n > 127) n = 127;
        }
    }
    return n + 127;
}

/* Conversion of a row-major [rows, cols] FP32 tensor (Sec. 2, 3.2, 3.3).
 * orientation ORC_ROW: blocks are 32 consecutive elements of a row, scales are
 * [rows, cols/32] row-major.  ORC_COL: blocks are 32 consecutive rows of one
 * column, scales are [rows/32, cols] row-major.  q has the shape of src in both
 * cases.  Returns 0, or -1 when the blocked dimension is not a multiple of 32. */
int orc_quantize(const float *src, int64_t rows, int64_t cols, int orientation,
                 int rule, int elem, uint8_t *q, uint8_t *s)
{
    orc_fmt f = orc_format(elem);
    if (orientation == ORC_ROW) {
        if (cols % 32) return -1;
        for (int64_t r = 0; r < rows; r++)
            for (int64_t cb = 0; cb < cols / 32; cb++) {
                const float *v = src + r * cols + cb * 32;
                int b = orc_scale_byte(orc_block_amax(v, 1, 32), elem, rule);
                s[r * (cols / 32) + cb] = (uint8_t)b;
                for (int i = 0; i < 32; i++) {
                    double x = (double)v[i];
                    int code;
                    if (isnan(x)) code = f.nan_code;
                    else if (isinf(x)) code = (x < 0 ? (1 << (f.ebits + f.mbits)) : 0) | f.max_code;
                    else code = orc_fp8_encode(ldexp(x, -(b - 127)), elem);   /* V_i / X */
                    q[r * cols + cb * 32 + i] = (uint8_t)code;
                }
            }
    } else {
        if (rows % 32) return -1;
        for (int64_t rb = 0; rb < rows / 32; rb++)
            for (int64_t c = 0; c < cols; c++) {
                const float *v = src + rb * 32 * cols + c;
                int b = orc_scale_byte(orc_block_amax(v, cols, 32), elem, rule);
                s[rb * cols + c] = (uint8_t)b;
                for (int i = 0; i < 32; i++) {
                    double x = (double)v[(int64_t)i * cols];
                    int code;
                    if (isnan(x)) code = f.nan_code;
                    else if (isinf(x)) code = (x < 0 ? (1 << (f.ebits + f.mbits)) : 0) | f.max_code;
                    else code = orc_fp8_encode(ldexp(x, -(b - 127)), elem);
                    q[(rb * 32 + i) * cols + c] = (uint8_t)code;
                }
            }
    }
    return 0;
}

/* Decoded value Q_i * X in binary64 (Sec. 2); scale byte 0xFF encodes NaN. */
int orc_dequantize(const uint8_t *q, const uint8_t *s, int64_t rows, int64_t cols,
                   int orientation, int elem, double *out)
{
    if (orientation == ORC_ROW ? (cols % 32) : (rows % 32)) return -1;
    for (int64_t r = 0; r < rows; r++)
        for (int64_t c = 0; c < cols; c++) {
            int b = (orientation == ORC_ROW) ? s[r * (cols / 32) + c / 32]
                                             : s[(r / 32) * cols + c];
            double d = orc_fp8_decode(q[r * cols + c], elem);
            out[r * cols + c] = (b == 0xFF) ? NAN : ldexp(d, b - 127);
        }
    return 0;
}

/* binary64 -> binary32, round-to-nearest-even (the C conversion under the
 * default rounding mode), overflow to infinity, gradual underflow. */
void orc_round_to_f32(const double *x, int64_t n, float *out)
{
    for (int64_t i = 0; i < n; i++) out[i] = (float)x[i];
}

/* binary64 -> bfloat16 bit pattern with a single round-to-nearest-even.
 * bfloat16: 8 exponent bits (bias 127), 7 mantissa bits, subnormals down to
 * 2^-133, overflow to infinity. */
void orc_round_to_bf16(const double *x, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; i++) {
        double v = x[i], a = fabs(v), k;
        uint16_t sign = signbit(v) ? 0x8000 : 0;
        int ex;
        if (isnan(v)) { out[i] = 0x7FC0; continue; }
        if (isinf(v)) { out[i] = sign | 0x7F80; continue; }
        if (a < ldexp(1.0, -126)) {
            k = rint(ldexp(a, 133));                     /* multiples of 2^-133 */
            out[i] = sign | (uint16_t)k;                 /* k == 128 is the min normal */
            continue;
        }
        (void)frexp(a, &ex);
        ex -= 1;
        k = rint(ldexp(a, 7 - ex));                      /* in [128, 256] */
        if (k == 256.0) { ex += 1; k = 128.0; }
        if (ex > 127) { out[i] = sign | 0x7F80; continue; }
        out[i] = sign | (uint16_t)(((ex + 127) << 7) | ((int)k - 128));
    }
}
