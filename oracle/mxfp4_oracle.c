/*
 * CPU oracle for the MXFP4 quantize + block-scaled GEMM path.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes.  It shares no code, header, table or constant generator with
 * the CUDA library; only tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  The product path never does.
 *
 * What it follows:
 *   - MX micro-scaling, Appendix A.1, Eq. (1): one shared power-of-two scale per
 *     block of 32 elements, elements rounded to the nearest 4-bit float.
 *   - Hadamard rotation before the quantizer, Appendix A.2 (tiled: one transform
 *     per MX block along the reduction axis; deterministic or with random sign
 *     flips).
 *   - Which axis each GEMM operand is rotated/quantized along: Appendix C
 *     (Fprop, Dgrad, Wgrad cancellation identities).
 *   - Row-wise (1x32) and column-wise (32x1) block orientation: Appendix D.
 *
 * Readings fixed where the paper is silent (each also listed in the design notes):
 *   - scale = 2^(floor(log2 amax) - 2)  (the E2M1 format's emax is 2), stored as an
 *     E8M0 byte clamp(biased_exponent(amax) - 2, 0, 254); values above 6*scale clip.
 *   - nearest = round-to-nearest, ties to the even code; the sign bit is kept
 *     even when the magnitude rounds to zero.
 *   - H is the unnormalised +-1 Sylvester matrix, applied with a fixed five-stage
 *     fp32 butterfly (h = 1,2,4,8,16); the 1/32 is an exact factor on the GEMM.
 *   - random sign flips: one 32-bit mask per seed, shared by every tile and by
 *     both operands (so D*D = I cancels in the product).
 *   - the 16-point variant (the paper's final choice, Appendix A.2) rotates each half of an
 *     MX block with its own 16-point transform (stages h = 1,2,4,8); its randomized form
 *     uses the low 16 bits of the same mask for both halves; the exact factor is 1/16.
 *   - stochastic rounding: 8 random bits per element from Philox4x32-10 keyed by
 *     the seed and counted by the element index in the operand view.
 *     PARITY UNPINNED against the paper for the stochastic-rounding bit pattern:
 *     the paper names the technique but defines neither generator nor bit width.
 *     The rule as fixed here is pinned by the generator's published known answers, by
 *     hand-derived worked tiles (keying and indexing; the strictness of the u < frac
 *     comparison at equality) and by statistical invariants.
 *
 * Build: gcc -O2 -std=c11 -fPIC -shared -fopenmp -ffp-contract=off (no fast-math).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MX_BLOCK 32

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (counter-based generator; the round function is the published */
/* one: two 32x32->64 multiplies, xor with the neighbouring counter words and   */
/* the key, key bumped by the Weyl constants between rounds).                   */
/* ------------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit sign mask of the randomized rotation: bit j set => element j of
 * every 32-tile is negated before the transform (Appendix A.2, "random sign
 * flips").  Drawn from a Philox stream separate from the rounding stream. */
uint32_t oracle_sign_mask(uint64_t seed)
{
    uint32_t ctr[4] = {0u, 0u, 0u, 1u};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t out[4];
    oracle_philox4x32_10(ctr, key, out);
    return out[0];
}

/* ------------------------------------------------------------------------- */
/* 32-point unnormalised Walsh-Hadamard transform, Sylvester order              */
/* (Appendix A.2: H has entries +-1).  Every add/sub is one fp32 operation.     */
/* ------------------------------------------------------------------------- */
void oracle_fwht32(float v[MX_BLOCK])
{
    for (int h = 1; h < MX_BLOCK; h *= 2) {
        for (int i = 0; i < MX_BLOCK; i += 2 * h) {
            for (int j = i; j < i + h; ++j) {
                float a = v[j];
                float b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
        }
    }
}

/* Two independent 16-point transforms, one per half of the 32-tile (Appendix A.2: H16 in a
 * tiled layout): the first four stages of the 32-point butterfly. */
void oracle_fwht16x2(float v[MX_BLOCK])
{
    for (int h = 1; h < 16; h *= 2) {
        for (int i = 0; i < MX_BLOCK; i += 2 * h) {
            for (int j = i; j < i + h; ++j) {
                float a = v[j];
                float b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
        }
    }
}

static inline float bf16_bits_to_float(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static inline uint32_t float_bits(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    return u;
}

/* E2M1 magnitudes by code 0..7; bit 3 of a code is the sign. */
static const double E2M1_GRID[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

/* Round-to-nearest, ties to the even code, saturating at 6 (Eq. (1): Q_FP4). */
static int e2m1_rne(float a)
{
    if (a <= 0.25f) return 0;
    if (a < 0.75f) return 1;
    if (a <= 1.25f) return 2;
    if (a < 1.75f) return 3;
    if (a <= 2.5f) return 4;
    if (a < 3.5f) return 5;
    if (a <= 5.0f) return 6;
    return 7;
}

/* Stochastic rounding between the two neighbouring grid points using an 8-bit
 * uniform u = (u8 + 0.5)/256: round up iff u < frac.  Clipping above 6 stays
 * deterministic; frac == 0 never moves. */
static int e2m1_sr(float a, uint32_t u8)
{
    if (a >= 6.0f) return 7;
    int c = 0;
    while (c < 6 && !(a < (float)E2M1_GRID[c + 1])) ++c;
    float lo = (float)E2M1_GRID[c];
    float hi = (float)E2M1_GRID[c + 1];
    float frac = (a - lo) / (hi - lo); /* exact: Sterbenz difference, power-of-two step */
    float lhs = (float)(2u * u8 + 1u);
    float rhs = 512.0f * frac;
    return (lhs < rhs) ? c + 1 : c;
}

/* The 8 random bits of element e in the operand view (seed, operand tag). */
static uint32_t sr_bits(uint64_t e, uint64_t seed, uint32_t tag)
{
    uint64_t g = e >> 4;
    uint32_t ctr[4] = {(uint32_t)(g & 0xFFFFFFFFu), (uint32_t)(g >> 32), tag, 0u};
    uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t w[4];
    oracle_philox4x32_10(ctr, key, w);
    uint32_t word = w[(e & 15u) >> 2];
    return (word >> (8u * (uint32_t)(e & 3u))) & 0xFFu;
}

/* Largest magnitude of one 32-tile that is already in fp32 (after the optional rotation). */
static float tile_amax(const float v[MX_BLOCK])
{
    float amax = 0.0f;
    for (int j = 0; j < MX_BLOCK; ++j) {
        float a = fabsf(v[j]);
        if (a > amax) amax = a;
    }
    return amax;
}

/* E8M0 byte of Eq. (1) for a block whose largest magnitude is amax:
 * 2^(floor(log2 amax) - 2), i.e. the fp32 biased exponent minus 2, clamped to [0, 254]. */
static uint8_t scale_byte_from_amax(float amax)
{
    int E = (int)((float_bits(amax) >> 23) & 0xFFu);
    int byte = E - 2;
    if (byte < 0) byte = 0;
    if (byte > 254) byte = 254;
    return (uint8_t)byte;
}

/* Round the 32 values of a tile to E2M1 codes (one per byte, unpacked) under a given scale. */
static void round_tile(const float v[MX_BLOCK], uint8_t byte, int rounding, uint64_t e0, uint64_t seed,
                       uint32_t tag, uint8_t code[MX_BLOCK])
{
    float mult = ldexpf(1.0f, 127 - (int)byte);
    for (int j = 0; j < MX_BLOCK; ++j) {
        float s = v[j] * mult;
        float a = fabsf(s);
        int mag = (rounding == 0) ? e2m1_rne(a) : e2m1_sr(a, sr_bits(e0 + (uint64_t)j, seed, tag));
        int sign = (int)(float_bits(v[j]) >> 31);
        code[j] = (uint8_t)((sign << 3) | mag);
    }
}

/* Quantize one 32-tile (1D block: the tile is its own scale group).
 * Writes 32 codes and returns the E8M0 scale byte. */
static uint8_t quantize_tile(const float v[MX_BLOCK], int rounding, uint64_t e0, uint64_t seed,
                             uint32_t tag, uint8_t code[MX_BLOCK])
{
    uint8_t byte = scale_byte_from_amax(tile_amax(v));
    round_tile(v, byte, rounding, e0, seed, tag, code);
    return byte;
}

/* One 32-tile of the operand view, widened to fp32, sign-flipped and rotated as the mode asks. */
static void load_rotated_tile(const uint16_t* src, int64_t ld, int axis, int64_t o, int64_t t,
                              int hadamard_mode, uint32_t mask, float v[MX_BLOCK])
{
    for (int j = 0; j < MX_BLOCK; ++j) {
        int64_t k = t * MX_BLOCK + j;
        uint16_t b = axis ? src[o * ld + k] : src[k * ld + o];
        v[j] = bf16_bits_to_float(b);
    }
    if (hadamard_mode == 2 || hadamard_mode == 4) {
        for (int j = 0; j < MX_BLOCK; ++j)
            if ((mask >> j) & 1u) v[j] = -v[j];
    }
    if (hadamard_mode == 1 || hadamard_mode == 2) oracle_fwht32(v);
    if (hadamard_mode == 3 || hadamard_mode == 4) oracle_fwht16x2(v);
}

static uint32_t mode_sign_mask(int hadamard_mode, uint64_t seed)
{
    if (hadamard_mode == 2) return oracle_sign_mask(seed);
    if (hadamard_mode == 4) {
        uint32_t m16 = oracle_sign_mask(seed) & 0xFFFFu;   /* same 16 signs for both halves */
        return m16 | (m16 << 16);
    }
    return 0u;
}

/*
 * oracle_quantize: src is a row-major [rows x cols] bf16 matrix (raw 16-bit
 * patterns) with leading dimension ld (elements).  The operand view is
 *   axis = 1: V[o][k] = src[o][k], outer = rows, K = cols   (row-wise 1x32 blocks)
 *   axis = 0: V[o][k] = src[k][o], outer = cols, K = rows   (column-wise 32x1 blocks;
 *             the output is the transposed operand, Appendix C Dgrad/Wgrad)
 * codes  : [outer x K/2] bytes, element k even in bits 3:0, odd in bits 7:4
 * scales : [outer x K/32] bytes, canonical row-major
 * hadamard_mode: 0 none, 1 deterministic H32, 2 randomized H32 (sign mask from seed),
 *                3 deterministic H16 (per half-block), 4 randomized H16
 * rounding     : 0 round-to-nearest-even, 1 stochastic
 * Returns 0, or -1 on a bad argument.
 */
int oracle_quantize(const uint16_t* src, int64_t rows, int64_t cols, int64_t ld, int axis,
                    int hadamard_mode, int rounding, uint64_t seed, uint32_t tag, uint8_t* codes,
                    uint8_t* scales)
{
    if (!src || !codes || !scales) return -1;
    if (axis != 0 && axis != 1) return -1;
    if (hadamard_mode < 0 || hadamard_mode > 4 || rounding < 0 || rounding > 1) return -1;
    int64_t outer = axis ? rows : cols;
    int64_t K = axis ? cols : rows;
    if (outer <= 0 || K <= 0 || K % MX_BLOCK != 0 || ld < cols) return -1;
    const uint32_t mask = mode_sign_mask(hadamard_mode, seed);
    const int64_t nt = K / MX_BLOCK;

#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < outer; ++o) {
        for (int64_t t = 0; t < nt; ++t) {
            float v[MX_BLOCK];
            uint8_t code[MX_BLOCK];
            load_rotated_tile(src, ld, axis, o, t, hadamard_mode, mask, v);
            uint64_t e0 = (uint64_t)o * (uint64_t)K + (uint64_t)(t * MX_BLOCK);
            uint8_t byte = quantize_tile(v, rounding, e0, seed, tag, code);
            scales[o * nt + t] = byte;
            uint8_t* dst = codes + o * (K / 2) + t * (MX_BLOCK / 2);
            for (int j = 0; j < MX_BLOCK; j += 2) dst[j / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
        }
    }
    return 0;
}

/*
 * oracle_quantize_2d: the 32 x 32 block strategy of Appendix D.  Same operand view, rotation,
 * rounding, code packing and canonical scale array as oracle_quantize, but ONE E8M0 scale is
 * shared by a region of 32 consecutive operand rows x one 32-element block along K (regions are
 * aligned to multiples of 32 in both directions; when outer is not a multiple of 32 the last
 * region has fewer rows).  The scale comes from the largest magnitude over the whole region --
 * of the rotated values when a rotation is on -- and is written to scales[o][t] for every row o
 * of the region, so a consumer of 1D scales reads it unchanged.
 */
int oracle_quantize_2d(const uint16_t* src, int64_t rows, int64_t cols, int64_t ld, int axis,
                       int hadamard_mode, int rounding, uint64_t seed, uint32_t tag, uint8_t* codes,
                       uint8_t* scales)
{
    if (!src || !codes || !scales) return -1;
    if (axis != 0 && axis != 1) return -1;
    if (hadamard_mode < 0 || hadamard_mode > 4 || rounding < 0 || rounding > 1) return -1;
    int64_t outer = axis ? rows : cols;
    int64_t K = axis ? cols : rows;
    if (outer <= 0 || K <= 0 || K % MX_BLOCK != 0 || ld < cols) return -1;
    const uint32_t mask = mode_sign_mask(hadamard_mode, seed);
    const int64_t nt = K / MX_BLOCK;
    const int64_t groups = (outer + MX_BLOCK - 1) / MX_BLOCK;

#pragma omp parallel for schedule(static)
    for (int64_t g = 0; g < groups; ++g) {
        const int64_t o_begin = g * MX_BLOCK;
        const int64_t o_end = o_begin + MX_BLOCK < outer ? o_begin + MX_BLOCK : outer;
        for (int64_t t = 0; t < nt; ++t) {
            float v[MX_BLOCK][MX_BLOCK];
            float amax = 0.0f;
            for (int64_t o = o_begin; o < o_end; ++o) {
                load_rotated_tile(src, ld, axis, o, t, hadamard_mode, mask, v[o - o_begin]);
                float a = tile_amax(v[o - o_begin]);
                if (a > amax) amax = a;
            }
            const uint8_t byte = scale_byte_from_amax(amax);
            for (int64_t o = o_begin; o < o_end; ++o) {
                uint8_t code[MX_BLOCK];
                uint64_t e0 = (uint64_t)o * (uint64_t)K + (uint64_t)(t * MX_BLOCK);
                round_tile(v[o - o_begin], byte, rounding, e0, seed, tag, code);
                scales[o * nt + t] = byte;
                uint8_t* dst = codes + o * (K / 2) + t * (MX_BLOCK / 2);
                for (int j = 0; j < MX_BLOCK; j += 2) dst[j / 2] = (uint8_t)(code[j] | (code[j + 1] << 4));
            }
        }
    }
    return 0;
}

/* Byte offset of scale (o, t) in the 128-row x 4-block tiled layout the GEMM
 * consumes; nt = number of 32-blocks along K.  A pure permutation of the
 * canonical layout (padding rows / blocks are extra bytes). */
int64_t oracle_scale_offset_tiled(int64_t o, int64_t t, int64_t nt)
{
    int64_t tiles_k = (nt + 3) / 4;
    int64_t tile = (o / 128) * tiles_k + (t / 4);
    return tile * 512 + (o % 32) * 16 + ((o % 128) / 32) * 4 + (t % 4);
}

/* Eq. (1) read right-to-left: value = grid[code] * 2^(scale - 127), in fp64 (exact). */
int oracle_dequantize(const uint8_t* codes, const uint8_t* scales, int64_t outer, int64_t K,
                      double* out)
{
    if (!codes || !scales || !out || outer <= 0 || K <= 0 || K % MX_BLOCK != 0) return -1;
    const int64_t nt = K / MX_BLOCK;
#pragma omp parallel for schedule(static)
    for (int64_t o = 0; o < outer; ++o) {
        for (int64_t k = 0; k < K; ++k) {
            uint8_t byte = codes[o * (K / 2) + k / 2];
            int c = (k & 1) ? (byte >> 4) : (byte & 0xF);
            double mag = E2M1_GRID[c & 7];
            double val = (c & 8) ? -mag : mag;
            out[o * K + k] = ldexp(val, (int)scales[o * nt + k / MX_BLOCK] - 127);
        }
    }
    return 0;
}

/*
 * oracle_gemm_rows: the plain definition of the block-scaled product.
 *   ref[i][n] = alpha * sum_k deq(A)[rows[i]][k] * deq(B)[n][k]      (fp64)
 *   S[i][n]   = |alpha| * sum_k |deq(A)[rows[i]][k] * deq(B)[n][k]|  (tolerance base)
 * A is [M x K], B is [N x K], both K-contiguous with canonical scales.
 * rows == NULL means all M rows (nrows must then equal M).
 */
int oracle_gemm_rows(const uint8_t* a_codes, const uint8_t* a_scales, const uint8_t* b_codes,
                     const uint8_t* b_scales, int64_t M, int64_t N, int64_t K, double alpha,
                     const int64_t* rows, int64_t nrows, double* ref, double* S)
{
    if (!a_codes || !a_scales || !b_codes || !b_scales || !ref) return -1;
    if (M <= 0 || N <= 0 || K <= 0 || K % MX_BLOCK != 0 || nrows <= 0) return -1;
    if (!rows && nrows != M) return -1;
    double* Bd = (double*)malloc((size_t)N * (size_t)K * sizeof(double));
    double* Ad = (double*)malloc((size_t)nrows * (size_t)K * sizeof(double));
    if (!Bd || !Ad) {
        free(Bd);
        free(Ad);
        return -2;
    }
    oracle_dequantize(b_codes, b_scales, N, K, Bd);
    const int64_t nt = K / MX_BLOCK;
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t m = rows ? rows[i] : i;
        if (m < 0 || m >= M) {
            free(Bd);
            free(Ad);
            return -1;
        }
        oracle_dequantize(a_codes + m * (K / 2), a_scales + m * nt, 1, K, Ad + i * K);
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

/* Threads the outer loops will use (reported beside CPU-baseline timings). */
int oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}
