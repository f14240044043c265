/*
 * CPU oracle for the 8-bit passes of the precision ladder (Table 1: the GEMMs that are not
 * switched to MXFP4 stay in FP8).
 *
 * TEST INFRASTRUCTURE ONLY, like mxfp4_oracle.c: shares nothing with the CUDA library.
 *
 * The paper names the 8-bit format only as "FP8".  Reading taken here (listed in the design
 * notes): the micro-scaled 8-bit format of the same family as MXFP4 -- Eq. (1) of Appendix A.1
 * with E4M3 elements instead of E2M1: blocks of 32 along the reduction axis, one E8M0 scale
 *   2^(floor(log2 amax) - 8)            (8 = largest exponent of an E4M3 value, 448 = 1.75 * 2^8)
 * stored as clamp(biased_exponent(amax) - 8, 0, 254), elements rounded to the nearest E4M3
 * value, ties to the even code, saturating at 448, sign kept on zero.  No rotation and no
 * stochastic rounding: the paper applies its stabilisers to the MXFP4 GEMMs only.
 *
 * E4M3 ("fn" flavour: no infinities): code = s eeee mmm,
 *   e > 0 : (-1)^s * 2^(e - 7) * (1 + m / 8)       largest finite: e = 15, m = 6 -> 448
 *   e = 0 : (-1)^s * 2^(-6) * (m / 8)              (sub-normals, step 2^-9)
 *   0x7F / 0xFF are NaN and never produced.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MX_BLOCK 32

static float bf16_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

static uint32_t bits_of(float f)
{
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    return u;
}

/* Value of an E4M3 code (finite codes only), exact in double. */
double oracle_e4m3_decode(uint8_t code)
{
    int s = code >> 7, e = (code >> 3) & 0xF, m = code & 7;
    double mag = e ? ldexp(1.0 + m / 8.0, e - 7) : ldexp(m / 8.0, -6);
    return s ? -mag : mag;
}

/* Magnitude code (7 bits) of the E4M3 value nearest to a >= 0, ties to the even code,
 * everything from 448 upward -> 448.  Works on the definition: pick the exponent, round the
 * significand to 3 fractional bits (rint = ties-to-even in the default rounding mode; the
 * significand's even/odd is the code's even/odd), carry into the exponent if it reaches 2. */
static int e4m3_rne_magnitude(double a)
{
    if (a >= 448.0) return 0x7E;
    if (a < ldexp(1.0, -6)) {                       /* sub-normal range: multiples of 2^-9 */
        int q = (int)rint(ldexp(a, 9));             /* 0..8 */
        return q;                                   /* q == 8 is code 0x08 = 2^-6: e = 1, m = 0 */
    }
    int ex;
    double fr = frexp(a, &ex);                      /* a = fr * 2^ex, fr in [0.5, 1) */
    int e = ex - 1;                                 /* a = (2 fr) * 2^e, 2 fr in [1, 2) */
    int m = (int)rint((2.0 * fr - 1.0) * 8.0);      /* 0..8 */
    if (m == 8) {
        m = 0;
        e += 1;
    }
    int code = ((e + 7) << 3) | m;
    return code > 0x7E ? 0x7E : code;
}

uint8_t oracle_e4m3_encode(float s)
{
    int sign = (int)(bits_of(s) >> 31);
    return (uint8_t)((sign << 7) | e4m3_rne_magnitude(fabs((double)s)));
}

/*
 * oracle_quantize_mxfp8: operand view, block orientation and scale array exactly as
 * oracle_quantize of the 4-bit oracle (axis = 1: V[o][k] = src[o][k]; axis = 0: V[o][k] = src[k][o]).
 * codes  : [outer x K] bytes, one E4M3 code per element
 * scales : [outer x K/32] bytes, canonical row-major
 */
int oracle_quantize_mxfp8(const uint16_t* src, int64_t rows, int64_t cols, int64_t ld, int axis,
                          uint8_t* codes, uint8_t* scales)
{
    if (!src || !codes || !scales) return -1;
    if (axis != 0 && axis != 1) return -1;
    int64_t outer = axis ? rows : cols;
    int64_t K = axis ? cols : rows;
    if (outer <= 0 || K <= 0 || K % MX_BLOCK != 0 || ld < cols) return -1;
    const int64_t nt = K / MX_BLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < outer; ++o) {
        for (int64_t t = 0; t < nt; ++t) {
            float v[MX_BLOCK];
            float amax = 0.0f;
            for (int j = 0; j < MX_BLOCK; ++j) {
                int64_t k = t * MX_BLOCK + j;
                v[j] = bf16_to_float(axis ? src[o * ld + k] : src[k * ld + o]);
                if (fabsf(v[j]) > amax) amax = fabsf(v[j]);
            }
            int byte = (int)((bits_of(amax) >> 23) & 0xFFu) - 8;
            if (byte < 0) byte = 0;
            if (byte > 254) byte = 254;
            scales[o * nt + t] = (uint8_t)byte;
            float mult = ldexpf(1.0f, 127 - byte);          /* exact power of two */
            for (int j = 0; j < MX_BLOCK; ++j)
                codes[o * K + t * MX_BLOCK + j] = oracle_e4m3_encode(v[j] * mult);
        }
    }
    return 0;
}

/*
 * oracle_gemm_rows_mxfp8: plain definition of the block-scaled product on E4M3 codes,
 *   ref[i][n] = alpha * sum_k deq(A)[rows[i]][k] * deq(B)[n][k]      (fp64)
 *   S[i][n]   = |alpha| * sum_k |...|                                (tolerance base)
 * with deq(code, scale) = e4m3(code) * 2^(scale - 127).  rows == NULL means all M rows.
 */
int oracle_gemm_rows_mxfp8(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                           const uint8_t* b_scales, int64_t M, int64_t N, int64_t K, double alpha,
                           const int64_t* rows, int64_t nrows, double* ref, double* S)
{
    if (!a_codes || !a_scales || !b_codes || !b_scales || !ref) return -1;
    if (M <= 0 || N <= 0 || K <= 0 || K % MX_BLOCK != 0 || nrows <= 0) return -1;
    if (!rows && nrows != M) return -1;
    const int64_t nt = K / MX_BLOCK;
    double* Bd = (double*)malloc((size_t)N * (size_t)K * sizeof(double));
    double* Ad = (double*)malloc((size_t)nrows * (size_t)K * sizeof(double));
    if (!Bd || !Ad) {
        free(Bd);
        free(Ad);
        return -2;
    }
    for (int64_t n = 0; n < N; ++n)
        for (int64_t k = 0; k < K; ++k)
            Bd[n * K + k] = ldexp(oracle_e4m3_decode(b_codes[n * K + k]), (int)b_scales[n * nt + k / MX_BLOCK] - 127);
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t m = rows ? rows[i] : i;
        if (m < 0 || m >= M) {
            free(Bd);
            free(Ad);
            return -1;
        }
        for (int64_t k = 0; k < K; ++k)
            Ad[i * K + k] = ldexp(oracle_e4m3_decode(a_codes[m * K + k]), (int)a_scales[m * nt + k / MX_BLOCK] - 127);
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < nrows; ++i) {
        const double* a = Ad + i * K;
        for (int64_t n = 0; n < N; ++n) {
            const double* b = Bd + n * K;
            double acc = 0.0, sabs = 0.0;
            for (int64_t k = 0; k < K; ++k) {
                double p = a[k] * b[k];
                acc += p;
                sabs += fabs(p);
            }
            ref[i * N + n] = alpha * acc;
            if (S) S[i * N + n] = fabs(alpha) * sabs;
        }
    }
    free(Bd);
    free(Ad);
    return 0;
}
