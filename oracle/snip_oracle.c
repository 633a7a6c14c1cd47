/*
 * snip_oracle.c -- plain CPU oracle for the SNIP mixed-precision linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of what the
 * hot path computes.  It shares no code with the CUDA library and must never be called from the
 * product path: only the tests, the smoke check and the benchmark's cpu_baseline / reference
 * arm may load it.
 *
 * What it follows (paper sections, not code):
 *   - Sec. 2.3 "Quantization", scaling rule:  scale = FPX_MAX / max(abs(x));
 *     y = Op(Quant(x * scale)) / scale.
 *   - Sec. 2.3 "Quantization granularity": 1x128 tiles for activations and gradients,
 *     128x128 blocks for weights.  The tile runs along the contraction dimension of the GEMM
 *     that consumes the operand, which gives the three tile kinds ROW, COL and BLK below.
 *   - Sec. 2.3 "Quantization format": FP8 E4M3 (OCP variant, max 448, no infinities) and
 *     FP4 E2M1 (MX specification, max 6).
 *   - Sec. 2.2 "Mixed Precision Training" / Fig. 5: quantize X, W, dY, run the GEMM in low
 *     precision, keep the GEMM output in BF16.  Tensor shapes X[M,K], W[N,K], dY[M,N] follow
 *     Sec. 4.2 / 4.3 (Y = X W^T, dX = dY W, dW = dY^T X).
 *   - Sec. 3.1 (Step 1): Frobenius norms of the tensors and of their quantization errors;
 *     Sec. 4.1: q(x) = x + delta_x, so the error tensor is x - dequant(quant(x)).
 *
 * Arithmetic contract (readings where the paper is silent are listed in the design notes):
 *   amax  : exact maximum of |x| over the tile (inputs are bf16, so float compares are exact)
 *   S     : binary32 division FPX_MAX / amax, round-to-nearest; S = 1 for an all-zero tile;
 *           S clamped to FLT_MAX if the division overflows
 *   t     : binary32 product x * S (rounded once, no fused multiply-add)
 *   code  : t rounded to the target format, round-to-nearest ties-to-even, saturating to
 *           +-FPX_MAX, sign bit taken from t (so -0 and negative underflow keep their sign)
 *   xhat  : value(code) / S evaluated in binary64
 *   stats : sum x^2 and sum (x - xhat)^2 in binary64
 *   GEMM  : plain binary64 triple loop over dequantized operands
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 * "parity unpinned": none of the functions in this file; every one has a pin in tests/.
 */
#include <float.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_FMT_BF16 = 0, ORC_FMT_FP8_E4M3 = 1, ORC_FMT_FP4_E2M1 = 2 };
enum { ORC_BLOCK_ROW = 0, ORC_BLOCK_COL = 1, ORC_BLOCK_BLK = 2,
       /* added option (the paper lets further quantization methods plug in as options, Sec. 3.2): 32-long tiles as in
        * the microscaling formats the paper cites; meant for the power-of-two scale rule */
       ORC_BLOCK_ROW32 = 3, ORC_BLOCK_COL32 = 4 };
#define ORC_TILE 128
#define ORC_SUBTILE 32

/* ---------------------------------------------------------------------------------------- */
/* Number formats                                                                            */
/* ---------------------------------------------------------------------------------------- */

/* A small binary floating-point format with `ebits` exponent bits, `mbits` mantissa bits and
 * exponent bias `bias`; `max_value` is the largest finite magnitude that is used. */
typedef struct {
    int ebits, mbits, bias;
    double max_value;
} orc_minifloat_t;

static const orc_minifloat_t ORC_E4M3 = {4, 3, 7, 448.0};
static const orc_minifloat_t ORC_E2M1 = {2, 1, 1, 6.0};

static const orc_minifloat_t *orc_format(int fmt)
{
    if (fmt == ORC_FMT_FP8_E4M3) return &ORC_E4M3;
    if (fmt == ORC_FMT_FP4_E2M1) return &ORC_E2M1;
    return NULL;
}

double orc_fpx_max(int fmt)
{
    const orc_minifloat_t *f = orc_format(fmt);
    return f ? f->max_value : 0.0;
}

/* bf16 is the upper half of a binary32 word. */
float orc_bf16_to_float(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* binary64 -> bf16, round-to-nearest ties-to-even, done arithmetically (no bit tricks on the
 * double): find the binade, round the significand to 8 bits with rint().  Finite inputs only;
 * overflow goes to infinity as IEEE rounding does. */
uint16_t orc_double_to_bf16(double v)
{
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    double a = fabs(v);
    if (a == 0.0) return sign;
    if (isnan(v)) return 0x7FC0u;
    if (isinf(v)) return (uint16_t)(sign | 0x7F80u);
    int e;
    (void)frexp(a, &e); /* a = f * 2^e, f in [0.5,1) -> a in [2^(e-1), 2^e) */
    int ex = e - 1;     /* unbiased exponent of the leading bit */
    if (ex < -126) ex = -126; /* subnormal range shares the spacing of the lowest binade */
    /* spacing of bf16 numbers in this binade: 2^(ex-7) */
    double q = rint(ldexp(a, 7 - ex)); /* integer significand, 128..256 for normals */
    if (q >= 256.0) { q = 128.0; ex += 1; }
    if (ex > 127) return (uint16_t)(sign | 0x7F80u);
    uint16_t bits;
    if (q < 128.0) bits = (uint16_t)q;                         /* subnormal */
    else bits = (uint16_t)(((ex + 127) << 7) | ((int)q - 128)); /* normal */
    return (uint16_t)(sign | bits);
}

/* Value of a code, closed form: (-1)^s 2^(e-bias) (1 + m/2^mbits) for e > 0,
 * (-1)^s 2^(1-bias) (m/2^mbits) for e = 0. */
static double orc_decode(const orc_minifloat_t *f, unsigned code)
{
    unsigned mmask = (1u << f->mbits) - 1u;
    unsigned emask = (1u << f->ebits) - 1u;
    unsigned m = code & mmask;
    unsigned e = (code >> f->mbits) & emask;
    unsigned s = (code >> (f->mbits + f->ebits)) & 1u;
    double frac = (double)m / (double)(1u << f->mbits);
    double mag = (e == 0) ? ldexp(frac, 1 - f->bias) : ldexp(1.0 + frac, (int)e - f->bias);
    return s ? -mag : mag;
}

double orc_decode_e4m3(uint8_t code) { return orc_decode(&ORC_E4M3, code); }
double orc_decode_e2m1(uint8_t code) { return orc_decode(&ORC_E2M1, code & 0xFu); }

double orc_decode_code(int fmt, uint8_t code)
{
    const orc_minifloat_t *f = orc_format(fmt);
    return f ? orc_decode(f, code) : 0.0;
}

/* Round a binary32 value to the format: nearest, ties to even, saturate to +-max_value.
 * The significand is rounded with rint() in the default (ties-to-even) rounding mode; all the
 * scalings by powers of two are exact in binary64. */
static unsigned orc_encode(const orc_minifloat_t *f, float t)
{
    unsigned sign = signbit(t) ? (1u << (f->ebits + f->mbits)) : 0u;
    double a = fabs((double)t);
    int emin = 1 - f->bias; /* exponent of the lowest normal binade */
    unsigned mag;
    if (a >= f->max_value) {
        /* saturate to the largest finite magnitude */
        int e;
        double frac = frexp(f->max_value, &e); /* max = frac * 2^e */
        int ex = e - 1;
        unsigned m = (unsigned)rint((frac * 2.0 - 1.0) * (double)(1u << f->mbits));
        mag = ((unsigned)(ex + f->bias) << f->mbits) | m;
    } else if (a == 0.0) {
        mag = 0u;
    } else {
        int e;
        (void)frexp(a, &e);
        int ex = e - 1;
        if (ex < emin) ex = emin; /* subnormals use the spacing of the lowest normal binade */
        /* a / 2^(ex - mbits) is the significand counted in units of the last place */
        double q = rint(ldexp(a, f->mbits - ex));
        double one = (double)(1u << f->mbits);
        if (q >= 2.0 * one) { q = one; ex += 1; } /* rounded up into the next binade */
        if (q < one) mag = (unsigned)q;            /* subnormal (or zero) */
        else mag = ((unsigned)(ex + f->bias) << f->mbits) | (unsigned)(q - one);
        /* rounding up cannot pass max_value: a < max_value and max_value is representable */
    }
    return sign | mag;
}

uint8_t orc_encode_e4m3(float t) { return (uint8_t)orc_encode(&ORC_E4M3, t); }
uint8_t orc_encode_e2m1(float t) { return (uint8_t)orc_encode(&ORC_E2M1, t); }

/* Scale of one tile: Sec. 2.3, scale = FPX_MAX / max(abs(x)), evaluated in binary32. */
float orc_tile_scale(int fmt, float amax)
{
    float fmax = (float)orc_fpx_max(fmt);
    if (amax == 0.0f) return 1.0f;
    volatile float s = fmax / amax; /* volatile: force a genuine binary32 quotient */
    float r = s;
    if (isinf(r)) r = FLT_MAX;
    return r;
}

/* Power-of-two variant of the scale ("new quantization methods can be added as further options",
 * Sec. 3.2; block scales that are powers of two are what the MX formats cited in Sec. 2.3 use):
 * the largest S = 2^e with amax * S <= FPX_MAX, so that the hardware can apply 1/S as an 8-bit
 * exponent.  e is clamped to [-126, 127]; S = 1 for an all-zero tile.  Worked out on the exponents
 * and significands, no division: amax = m_a 2^ea, FPX_MAX = m_f 2^ef with m in [1,2), then
 * e = ef - ea if m_a <= m_f, else ef - ea - 1. */
float orc_tile_scale_pow2(int fmt, float amax)
{
    if (amax == 0.0f) return 1.0f;
    int xa, xf;
    double ma = 2.0 * frexp((double)amax, &xa);            /* amax = ma * 2^(xa-1) */
    double mf = 2.0 * frexp(orc_fpx_max(fmt), &xf);
    int e = (xf - 1) - (xa - 1) - (ma > mf ? 1 : 0);
    if (e > 127) e = 127;
    if (e < -126) e = -126;
    return (float)ldexp(1.0, e);
}

/* ---------------------------------------------------------------------------------------- */
/* Quantizer                                                                                 */
/* ---------------------------------------------------------------------------------------- */

/* ---- stochastic rounding (Sec. 6.1: FP4 output gradients are rounded probabilistically to one of
 * the two nearest representable values) ------------------------------------------------------
 *
 * The paper names the method and cites it; the concrete rule used here (a reading): with
 * a = min(|t|, FPX_MAX) and lo <= a < hi the neighbouring representable magnitudes (subnormals
 * included; a == FPX_MAX stays), round to hi iff (a - lo) / (hi - lo) > (u + 1/2) / 2^16, where u
 * is a 16-bit uniform integer owned by the element; the sign bit is copied from t.  A representable
 * a has fraction 0 and never moves.  P(round up) equals the fraction to within 2^-17.
 *
 * The uniforms come from the counter-based generator Philox4x32 with 10 rounds (Salmon, Moraes,
 * Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", 2011): counter = (idx / 8 as two
 * 32-bit words, 0, 0), key = the two words of the seed; its four output words hold the eight
 * uniforms of elements 8*(idx/8) .. +7, element j in bits [16*(j%2), 16*(j%2)+16) of word j/2.
 */
static void orc_mulhilo32(uint32_t a, uint32_t b, uint32_t *hi, uint32_t *lo)
{
    uint64_t p = (uint64_t)a * (uint64_t)b;
    *hi = (uint32_t)(p >> 32);
    *lo = (uint32_t)p;
}

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint32_t hi0, lo0, hi1, lo1;
        orc_mulhilo32(0xD2511F53u, c0, &hi0, &lo0);
        orc_mulhilo32(0xCD9E8D57u, c2, &hi1, &lo1);
        uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; /* key schedule: golden-ratio and sqrt(3)-1 increments */
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

uint32_t orc_sr_uniform16(uint64_t seed, uint64_t idx)
{
    uint64_t blk = idx / 8;
    uint32_t ctr[4] = {(uint32_t)blk, (uint32_t)(blk >> 32), 0u, 0u};
    uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    uint32_t w[4];
    orc_philox4x32_10(ctr, key, w);
    unsigned j = (unsigned)(idx % 8);
    return (w[j / 2] >> (16 * (j % 2))) & 0xFFFFu;
}

/* Stochastically rounded code of the binary32 value t given the element's 16-bit uniform u.  The
 * neighbours are found by scanning the table of representable magnitudes (obviously correct, slow). */
static unsigned orc_encode_sr_fmt(const orc_minifloat_t *f, float t, uint32_t u)
{
    unsigned sign = signbit(t) ? 1u : 0u;
    double a = fabs((double)t);
    unsigned nmag = 1u << (f->ebits + f->mbits);      /* magnitude codes 0 .. nmag-1 */
    unsigned top = 0;                                  /* largest magnitude code in use (E4M3: 0x7E, 0x7F is NaN) */
    for (unsigned m = 0; m < nmag; ++m)
        if (orc_decode(f, m) <= f->max_value) top = m;
    double vmax = orc_decode(f, top);
    if (a >= vmax) return (sign << (f->ebits + f->mbits)) | top;
    unsigned lo = 0;
    for (unsigned m = 0; m <= top; ++m)
        if (orc_decode(f, m) <= a) lo = m;             /* magnitudes ascend with the code */
    double vlo = orc_decode(f, lo), vhi = orc_decode(f, lo + 1);
    double frac = (a - vlo) / (vhi - vlo);
    double thr = ((double)u + 0.5) / 65536.0;
    unsigned mag = frac > thr ? lo + 1 : lo;
    return (sign << (f->ebits + f->mbits)) | mag;
}

uint8_t orc_encode_sr(int fmt, float t, uint32_t u16)
{
    const orc_minifloat_t *f = orc_format(fmt);
    return f ? (uint8_t)orc_encode_sr_fmt(f, t, u16 & 0xFFFFu) : 0;
}

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* Shape of the scale tensor for a rows x cols input (Sec. 2.3 granularity):
 *   ROW: [ceil(cols/128)][rows]    one scale per 1x128 tile, tile index outermost
 *   COL: [ceil(rows/128)][cols]    one scale per 128x1 tile
 *   BLK: [ceil(rows/128)][ceil(cols/128)]
 *   ROW32: [ceil(cols/32)][rows]   one scale per 1x32 tile;   COL32: [ceil(rows/32)][cols]   one per 32x1 tile
 */
void orc_scale_shape(int64_t rows, int64_t cols, int block, int64_t *d0, int64_t *d1)
{
    if (block == ORC_BLOCK_ROW) { *d0 = ceil_div(cols, ORC_TILE); *d1 = rows; }
    else if (block == ORC_BLOCK_COL) { *d0 = ceil_div(rows, ORC_TILE); *d1 = cols; }
    else if (block == ORC_BLOCK_ROW32) { *d0 = ceil_div(cols, ORC_SUBTILE); *d1 = rows; }
    else if (block == ORC_BLOCK_COL32) { *d0 = ceil_div(rows, ORC_SUBTILE); *d1 = cols; }
    else { *d0 = ceil_div(rows, ORC_TILE); *d1 = ceil_div(cols, ORC_TILE); }
}

/* Index of the scale that governs element (r, c). */
static int64_t orc_scale_index(int64_t rows, int64_t cols, int block, int64_t r, int64_t c)
{
    if (block == ORC_BLOCK_ROW) return (c / ORC_TILE) * rows + r;
    if (block == ORC_BLOCK_COL) return (r / ORC_TILE) * cols + c;
    if (block == ORC_BLOCK_ROW32) return (c / ORC_SUBTILE) * rows + r;
    if (block == ORC_BLOCK_COL32) return (r / ORC_SUBTILE) * cols + c;
    return (r / ORC_TILE) * ceil_div(cols, ORC_TILE) + (c / ORC_TILE);
}

/*
 * Quantize a row-major rows x cols bf16 matrix.
 *   codes      [rows*cols] one code per byte (FP4 codes in the low nibble), may be NULL
 *   scales     scale tensor in the shape above, may be NULL
 *   xhat       [rows*cols] dequantized values in binary64, may be NULL
 *   sumsq      [2] = { sum x^2, sum (x - xhat)^2 }, may be NULL
 *   row_sumsq  [2*rows] = per-row {sum x^2, sum err^2} pairs, may be NULL
 * fmt = BF16 is the identity: no scales, xhat = x, zero error.
 * Returns 0, or -1 on a bad argument.
 */
int orc_quantize_rule(const uint16_t *x, int64_t rows, int64_t cols, int fmt, int block, int pow2_scale,
                      uint8_t *codes, float *scales, double *xhat, double *sumsq, double *row_sumsq);

int orc_quantize(const uint16_t *x, int64_t rows, int64_t cols, int fmt, int block,
                 uint8_t *codes, float *scales, double *xhat, double *sumsq,
                 double *row_sumsq)
{
    return orc_quantize_rule(x, rows, cols, fmt, block, 0, codes, scales, xhat, sumsq, row_sumsq);
}

static int orc_quantize_impl(const uint16_t *x, int64_t rows, int64_t cols, int fmt, int block, int pow2_scale,
                             int stochastic, uint64_t seed,
                             uint8_t *codes, float *scales, double *xhat, double *sumsq, double *row_sumsq);

/* Same with the scale rule selectable: pow2_scale = 0 is the paper's quotient FPX_MAX / amax,
 * pow2_scale = 1 the power-of-two option above.  Everything else is identical. */
int orc_quantize_rule(const uint16_t *x, int64_t rows, int64_t cols, int fmt, int block, int pow2_scale,
                      uint8_t *codes, float *scales, double *xhat, double *sumsq, double *row_sumsq)
{
    return orc_quantize_impl(x, rows, cols, fmt, block, pow2_scale, 0, 0, codes, scales, xhat, sumsq, row_sumsq);
}

/* Same with stochastic rounding of the codes (Sec. 6.1: used for FP4 output gradients): element
 * (r, c) draws the 16-bit uniform orc_sr_uniform16(seed, r * cols + c) and is rounded by
 * orc_encode_sr.  Scales are unchanged (they depend on amax only). */
int orc_quantize_sr(const uint16_t *x, int64_t rows, int64_t cols, int fmt, int block, int pow2_scale, uint64_t seed,
                    uint8_t *codes, float *scales, double *xhat, double *sumsq, double *row_sumsq)
{
    if (!orc_format(fmt)) return -1;
    return orc_quantize_impl(x, rows, cols, fmt, block, pow2_scale, 1, seed, codes, scales, xhat, sumsq, row_sumsq);
}

static int orc_quantize_impl(const uint16_t *x, int64_t rows, int64_t cols, int fmt, int block, int pow2_scale,
                             int stochastic, uint64_t seed,
                             uint8_t *codes, float *scales, double *xhat, double *sumsq, double *row_sumsq)
{
    if (!x || rows < 0 || cols < 0) return -1;
    if (fmt != ORC_FMT_BF16 && !orc_format(fmt)) return -1;
    if (block < ORC_BLOCK_ROW || block > ORC_BLOCK_COL32) return -1;
    const orc_minifloat_t *f = orc_format(fmt);

    int64_t sd0 = 0, sd1 = 0;
    orc_scale_shape(rows, cols, block, &sd0, &sd1);
    int64_t nscales = sd0 * sd1;
    float *S = NULL;

    if (f) {
        /* pass 1: amax per tile, then the scale */
        S = (float *)malloc(sizeof(float) * (size_t)(nscales > 0 ? nscales : 1));
        if (!S) return -1;
        for (int64_t i = 0; i < nscales; ++i) S[i] = 0.0f; /* holds amax first */
        /* groups of 128 rows never share a tile, so they can run in parallel */
        int64_t ngroups = ceil_div(rows, ORC_TILE);
#pragma omp parallel for schedule(static)
        for (int64_t g = 0; g < ngroups; ++g) {
            int64_t r1 = (g + 1) * ORC_TILE < rows ? (g + 1) * ORC_TILE : rows;
            for (int64_t r = g * ORC_TILE; r < r1; ++r)
                for (int64_t c = 0; c < cols; ++c) {
                    float a = fabsf(orc_bf16_to_float(x[r * cols + c]));
                    int64_t si = orc_scale_index(rows, cols, block, r, c);
                    if (a > S[si]) S[si] = a;
                }
        }
        for (int64_t i = 0; i < nscales; ++i) S[i] = pow2_scale ? orc_tile_scale_pow2(fmt, S[i]) : orc_tile_scale(fmt, S[i]);
        if (scales) memcpy(scales, S, sizeof(float) * (size_t)nscales);
    }

    /* pass 2: encode, dequantize, per-row statistics (rows are independent) */
    double *rs = (double *)malloc(sizeof(double) * 2 * (size_t)(rows > 0 ? rows : 1));
    if (!rs) { free(S); return -1; }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double rx = 0.0, re = 0.0;
        for (int64_t c = 0; c < cols; ++c) {
            float xf = orc_bf16_to_float(x[r * cols + c]);
            double xd = (double)xf;
            double xh;
            if (f) {
                float s = S[orc_scale_index(rows, cols, block, r, c)];
                volatile float t = xf * s; /* one binary32 rounding, never fused */
                unsigned code = stochastic ? orc_encode_sr_fmt(f, t, orc_sr_uniform16(seed, (uint64_t)(r * cols + c)))
                                           : orc_encode(f, t);
                if (codes) codes[r * cols + c] = (uint8_t)code;
                xh = orc_decode(f, code) / (double)s;
            } else {
                xh = xd;
            }
            if (xhat) xhat[r * cols + c] = xh;
            double d = xd - xh;
            rx += xd * xd;
            re += d * d;
        }
        rs[2 * r] = rx;
        rs[2 * r + 1] = re;
    }
    /* totals: rows added in ascending order, so the result does not depend on threading */
    double tot_x = 0.0, tot_e = 0.0;
    for (int64_t r = 0; r < rows; ++r) { tot_x += rs[2 * r]; tot_e += rs[2 * r + 1]; }
    if (row_sumsq) memcpy(row_sumsq, rs, sizeof(double) * 2 * (size_t)rows);
    free(rs);
    if (sumsq) { sumsq[0] = tot_x; sumsq[1] = tot_e; }
    free(S);
    return 0;
}

/*
 * Two-level block scaling in the style of NVFP4 (added option; the paper lets further quantization methods plug in
 * as options, Sec. 3.2): E2M1 codes in tiles of 16 along the contraction, one E4M3 scale byte per tile (used
 * unsigned), one binary32 factor per tensor.  The paper gives no rule for it; this one is fixed here:
 *   enc   = binary32 quotient 2688 / tensor_amax   (2688 = 448 * 6; enc = 1 if tensor_amax == 0)
 *   d     = binary32 product of the binary32 quotient amax_tile / 6 with enc
 *   sf    = d rounded to E4M3 (nearest, ties to even, saturating at 448): a code 0x00 .. 0x7E
 *   E     = binary32 quotient enc / value(sf)         (a tile with value(sf) == 0 gets all-zero codes)
 *   t     = binary32 product x * E;  code = t rounded to E2M1 (nearest even, saturating at 6)
 *   xhat  = value(code) * value(sf) / enc  in binary64  (what the block-scaled tensor core followed by one
 *           division by enc computes)
 * col_tiles = 0: 1x16 tiles along the columns, sf[ceil(cols/16)][rows]; 1: 16x1 tiles along the rows,
 * sf[ceil(rows/16)][cols].  tensor_amax is an input (any positive bound of max|x| works; the exact maximum uses the
 * scale bytes' range best).  codes / sf / xhat / sumsq may be NULL.  Returns 0, or -1 on a bad argument.
 */
int orc_quantize_nvfp4_sr(const uint16_t *x, int64_t rows, int64_t cols, int col_tiles, float tensor_amax, int stochastic, uint64_t seed,
                          uint8_t *codes, uint8_t *sf, float *enc_out, double *xhat, double *sumsq);

int orc_quantize_nvfp4(const uint16_t *x, int64_t rows, int64_t cols, int col_tiles, float tensor_amax,
                       uint8_t *codes, uint8_t *sf, float *enc_out, double *xhat, double *sumsq)
{
    return orc_quantize_nvfp4_sr(x, rows, cols, col_tiles, tensor_amax, 0, 0, codes, sf, enc_out, xhat, sumsq);
}

/* The same with the codes rounded stochastically (Sec. 6.1: FP4 output gradients), by the rule and generator of
 * orc_quantize_sr applied to the product t; the scale bytes do not change. */
int orc_quantize_nvfp4_sr(const uint16_t *x, int64_t rows, int64_t cols, int col_tiles, float tensor_amax, int stochastic, uint64_t seed,
                          uint8_t *codes, uint8_t *sf, float *enc_out, double *xhat, double *sumsq)
{
    if (!x || rows < 0 || cols < 0 || !(tensor_amax >= 0.0f)) return -1;
    const int64_t tl = 16;
    const int64_t nt = col_tiles ? ceil_div(rows, tl) : ceil_div(cols, tl);   /* tiles per line */
    const int64_t lines = col_tiles ? cols : rows;
    volatile float enc = tensor_amax == 0.0f ? 1.0f : 2688.0f / tensor_amax;
    if (isinf(enc)) enc = FLT_MAX;
    if (enc_out) *enc_out = enc;
    uint8_t *sfl = (uint8_t *)malloc((size_t)(nt * lines > 0 ? nt * lines : 1));
    float *am = (float *)calloc((size_t)(nt * lines > 0 ? nt * lines : 1), sizeof(float));
    if (!sfl || !am) { free(sfl); free(am); return -1; }
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float a = fabsf(orc_bf16_to_float(x[r * cols + c]));
            int64_t si = col_tiles ? (r / tl) * cols + c : (c / tl) * rows + r;
            if (a > am[si]) am[si] = a;
        }
    for (int64_t i = 0; i < nt * lines; ++i) {
        volatile float q = am[i] / 6.0f;
        volatile float d = q * enc;
        sfl[i] = (uint8_t)orc_encode(&ORC_E4M3, d);
    }
    double *rs = (double *)malloc(sizeof(double) * 2 * (size_t)(rows > 0 ? rows : 1));
    if (!rs) { free(sfl); free(am); return -1; }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) {
        double tx = 0.0, te = 0.0;
        for (int64_t c = 0; c < cols; ++c) {
            float xf = orc_bf16_to_float(x[r * cols + c]);
            int64_t si = col_tiles ? (r / tl) * cols + c : (c / tl) * rows + r;
            double sv = orc_decode(&ORC_E4M3, sfl[si]);
            unsigned code = 0;
            if (sv != 0.0) {
                volatile float E = enc / (float)sv;
                volatile float t = xf * E;
                code = stochastic ? orc_encode_sr_fmt(&ORC_E2M1, t, orc_sr_uniform16(seed, (uint64_t)(r * cols + c))) : orc_encode(&ORC_E2M1, t);
            } else if (signbit(xf)) {
                code = 0x8;   /* the sign survives, as it does for an underflowing product */
            }
            double xh = orc_decode(&ORC_E2M1, code) * sv / (double)enc;
            if (codes) codes[r * cols + c] = (uint8_t)code;
            if (xhat) xhat[r * cols + c] = xh;
            double xd = (double)xf, dd = xd - xh;
            tx += xd * xd;
            te += dd * dd;
        }
        rs[2 * r] = tx;
        rs[2 * r + 1] = te;
    }
    double tot_x = 0.0, tot_e = 0.0;   /* rows added in ascending order: independent of threading */
    for (int64_t r = 0; r < rows; ++r) { tot_x += rs[2 * r]; tot_e += rs[2 * r + 1]; }
    free(rs);
    if (sf) memcpy(sf, sfl, (size_t)(nt * lines));
    if (sumsq) { sumsq[0] = tot_x; sumsq[1] = tot_e; }
    free(sfl);
    free(am);
    return 0;
}

/* Dequantize codes + scales to binary64: xhat = value(code) / S (Sec. 2.3: the scale is removed
 * after the operator by dividing by it). */
int orc_dequantize(const uint8_t *codes, const float *scales, int64_t rows, int64_t cols,
                   int fmt, int block, double *xhat)
{
    const orc_minifloat_t *f = orc_format(fmt);
    if (!f || !codes || !scales || !xhat) return -1;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float s = scales[orc_scale_index(rows, cols, block, r, c)];
            xhat[r * cols + c] = orc_decode(f, codes[r * cols + c]) / (double)s;
        }
    return 0;
}

/*
 * Storage layout of the codes as the library defines it.
 *   transposed = 0: element (r,c) at linear index r*cols + c
 *   transposed = 1: element (r,c) at linear index c*rows + r   (the matrix is stored as its
 *                   transpose, so that the other dimension becomes contiguous)
 * FP8: one byte per element at that index.  FP4: two per byte; the element with the even
 * linear index sits in bits [3:0], the odd one in bits [7:4].  BF16: not packed here.
 * `out` has rows*cols bytes (FP8) or rows*cols/2 bytes (FP4; the contiguous dimension must be
 * even).
 */
int orc_pack_codes(const uint8_t *codes, int64_t rows, int64_t cols, int fmt, int transposed,
                   uint8_t *out)
{
    if (!codes || !out) return -1;
    if (fmt != ORC_FMT_FP8_E4M3 && fmt != ORC_FMT_FP4_E2M1) return -1;
    int64_t inner = transposed ? rows : cols;
    if (fmt == ORC_FMT_FP4_E2M1 && (inner & 1)) return -1;
    if (fmt == ORC_FMT_FP4_E2M1) memset(out, 0, (size_t)(rows * cols / 2));
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            int64_t lin = transposed ? c * rows + r : r * cols + c;
            uint8_t code = codes[r * cols + c];
            if (fmt == ORC_FMT_FP8_E4M3) out[lin] = code;
            else if (lin & 1) out[lin >> 1] |= (uint8_t)((code & 0xFu) << 4);
            else out[lin >> 1] |= (uint8_t)(code & 0xFu);
        }
    return 0;
}

/* ---------------------------------------------------------------------------------------- */
/* GEMMs: the plain definitions in binary64 (Fig. 5; shapes from Sec. 4.2 / 4.3)            */
/* ---------------------------------------------------------------------------------------- */

/* Y[M,N] = X[M,K] . W[N,K]^T */
void orc_gemm_fwd(const double *X, const double *W, double *Y, int64_t M, int64_t N, int64_t K)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int64_t k = 0; k < K; ++k) s += X[m * K + k] * W[n * K + k];
            Y[m * N + n] = s;
        }
}

/* dX[M,K] = dY[M,N] . W[N,K] */
void orc_gemm_dgrad(const double *dY, const double *W, double *dX, int64_t M, int64_t N,
                    int64_t K)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int64_t k = 0; k < K; ++k) dX[m * K + k] = 0.0;
        for (int64_t n = 0; n < N; ++n) {
            double g = dY[m * N + n];
            for (int64_t k = 0; k < K; ++k) dX[m * K + k] += g * W[n * K + k];
        }
    }
}

/* dW[N,K] = dY[M,N]^T . X[M,K] */
void orc_gemm_wgrad(const double *dY, const double *X, double *dW, int64_t M, int64_t N,
                    int64_t K)
{
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t k = 0; k < K; ++k) dW[n * K + k] = 0.0;
        for (int64_t m = 0; m < M; ++m) {
            double g = dY[m * N + n];
            for (int64_t k = 0; k < K; ++k) dW[n * K + k] += g * X[m * K + k];
        }
    }
}

/* Round a binary64 array to bf16 bit patterns (the GEMM output stays in BF16, Sec. 2.2). */
void orc_round_to_bf16(const double *v, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_double_to_bf16(v[i]);
}

/* Sum of squares of a bf16 tensor in binary64 (plain Frobenius norm squared, Sec. 3.1). */
double orc_sumsq_bf16(const uint16_t *x, int64_t n)
{
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double v = (double)orc_bf16_to_float(x[i]);
        s += v * v;
    }
    return s;
}

/* ---- AdamW sensitivity term (Sec. 4.3: weight divergence) --------------------------------------
 *
 * Step 1 also collects the Frobenius norm of the elementwise term
 *     T = (1 - beta1) / (sqrt(v) + eps)  -  (1 - beta2) m g / ( sqrt(v) (sqrt(v) + eps)^2 ),
 * the derivative of the AdamW direction m / (sqrt(v) + eps) with respect to the gradient g (m, v are
 * the moments after they absorbed g).  Returns sum T^2 in binary64.  m, v, g: binary64 copies of the
 * inputs.  Reading: where v == 0 (then g == 0 and m == 0 in AdamW) the second term is taken as 0. */
double orc_adamw_sensitivity_sumsq(const double *m, const double *v, const double *g, int64_t n, double beta1, double beta2, double eps)
{
    double acc = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        double s = sqrt(v[i]);
        double d = s + eps;
        double first = (1.0 - beta1) / d;
        double second = v[i] == 0.0 ? 0.0 : (1.0 - beta2) * m[i] * g[i] / (s * d * d);
        double t = first - second;
        acc += t * t;
    }
    return acc;
}

/* Number of threads the parallel loops use from now on (timing aid: the benchmark also reports a
 * one-core figure).  No effect without OpenMP. */
void orc_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
