/*
 * fp4q oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, step-by-step CPU statement of what the hot path computes:
 * transposition-invariant 2D-block FP4 quantization (Section 3, Section 3.1,
 * appendix "2D Block Scaling and Transposition Consistency", appendix
 * "Rounding and Gradient Propagation"), the MXFP8 operand format of the
 * Q/K projections (Section 3.2) and the three linear-layer GEMMs (Section 3,
 * "Application to linear layers") on dequantized values.
 *
 * Everything is written from the definitions, in double precision and plain
 * integers, with no blocking, fusion or bit tricks, so that it can be checked
 * against the paper by eye.  Only tests, the smoke check and the CPU-baseline
 * leg of the benchmark may call it; the CUDA library shares no code with it.
 * OpenMP, where present, parallelises independent tiles/rows only.
 *
 * Pins (tests marked "not gpu"): exhaustive code tables, exhaustive scale rule
 * against exact rational arithmetic, exhaustive nearest/stochastic rounding
 * decisions against exact rational arithmetic, Philox against two library
 * implementations, brute force on tiny tiles, transposition invariance,
 * no-clipping, unbiasedness.  Parity unpinned: none of the functions below;
 * the paper's model-quality claims are out of scope.
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#define ORC_BLOCK 32            /* 2D block size b (Section 3: 32x32 blocks)            */
#define ORC_MODE_NEAREST 0      /* forward rounding (appendix "Rounding ...")           */
#define ORC_MODE_STOCHASTIC 1   /* backward rounding of gradient tensors (Section 3.1)  */
#define ORC_FLAG_INDEX_TRANSPOSED 1u

/* ------------------------------------------------------------------ formats */

/* BF16 bit pattern -> value.  BF16 is the upper half of an IEEE binary32. */
double orc_bf16_to_double(uint16_t bits)
{
    uint32_t w = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* E2M1 (Section 2: the 4-bit element format of MXFP4): 1 sign, 2 exponent,
 * 1 mantissa bit, exponent bias 1, subnormal at exponent 0, no Inf/NaN.
 * Written from the format definition, not from a table. */
double orc_e2m1_value(int code)
{
    int s = (code >> 3) & 1, e = (code >> 1) & 3, m = code & 1;
    double mag = (e == 0) ? 0.5 * m : ldexp(1.0 + 0.5 * m, e - 1);
    return s ? -mag : mag;
}

/* Q_p and Q_n of Section 3.1 for E2M1: the largest and smallest code values. */
static double orc_qp(void) { return orc_e2m1_value(0x7); }
static double orc_qn(void) { return orc_e2m1_value(0xF); }

/* E4M3 (MXFP8 element format): 1 sign, 4 exponent, 3 mantissa bits, bias 7,
 * subnormals at exponent 0, 0x7F/0xFF are NaN, no Inf; largest finite 448. */
double orc_e4m3_value(int code)
{
    int s = (code >> 7) & 1, e = (code >> 3) & 15, m = code & 7;
    double mag;
    if (e == 15 && m == 7) return NAN;
    mag = (e == 0) ? ldexp((double)m / 8.0, -6) : ldexp(1.0 + (double)m / 8.0, e - 7);
    return s ? -mag : mag;
}

/* --------------------------------------------------------------- scale rule */

/* Truncation-free scale (Section 3.1; appendix "2D Block Scaling ..."):
 *   S = 2^ceil(log2(2M / (Q_p - Q_n))).
 * With Q_p - Q_n = 2*Q_max this is the smallest power of two with
 * Q_max * S >= M, which is evaluated here exactly with ldexp (no floating
 * log2).  The exponent is clamped to what one UE8M0 byte can hold
 * (e in [-127,127], code = e + 127); M = 0 takes the lowest exponent.
 * Raising S (the lower clamp) can never cause clipping. */
static int orc_pow2_exponent_for(double M, double qmax)
{
    int e = -127;
    while (e < 127 && ldexp(qmax, e) < M) e++;
    return e;
}

int orc_scale_exponent(double M)
{
    double qmax = (orc_qp() - orc_qn()) / 2.0;
    return orc_pow2_exponent_for(M, qmax);
}

int orc_mxfp8_scale_exponent(double M)
{
    return orc_pow2_exponent_for(M, 448.0);
}

/* ------------------------------------------------------------------- Philox */

/* Philox4x32-10 counter-based generator (Salmon et al., SC'11): ten rounds of
 * two 32x32->64 multiplies with the key bumped by Weyl constants each round. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    int round;
    for (round = 0; round < 10; round++) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The random byte of one element: stream keyed on (seed, tensor id, element
 * index).  One Philox block covers 16 consecutive element indices. */
unsigned orc_random_byte(uint64_t seed, uint32_t tensor_id, uint64_t idx)
{
    uint64_t blk = idx >> 4;
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), tensor_id, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return (out[(idx >> 2) & 3] >> (8 * (idx & 3))) & 0xFFu;
}

/* ----------------------------------------------------------------- rounding */

/* Round-to-nearest onto the E2M1 magnitudes (appendix "Rounding ...": forward
 * pass).  v = |x|/S in [0, Q_p].  Brute force over the eight magnitudes; a tie
 * goes to the even code (IEEE default). */
int orc_round_nearest(double v)
{
    int best = 0, c;
    double bestd = fabs(v - orc_e2m1_value(0));
    for (c = 1; c < 8; c++) {
        double d = fabs(v - orc_e2m1_value(c));
        if (d < bestd || (d == bestd && (c & 1) == 0 && (best & 1) == 1)) {
            best = c;
            bestd = d;
        }
    }
    return best;
}

/* Stochastic rounding (Section 3.1, E[roundS(x)] = x): v lies between the
 * adjacent magnitudes lo <= v < hi; it goes up with probability
 * floor(256 p)/256, p = (v - lo)/(hi - lo), decided by the element's random
 * byte r8: up iff floor(256 p) + r8 >= 256.  Exactly expectation-preserving
 * whenever 256 p is an integer; otherwise biased toward zero by less than
 * (hi - lo)/256. */
int orc_round_stochastic(double v, unsigned r8)
{
    int lo = 0, c;
    double vlo, vhi, p;
    for (c = 0; c < 8; c++)
        if (orc_e2m1_value(c) <= v) lo = c;
    if (lo == 7) return 7;
    vlo = orc_e2m1_value(lo);
    vhi = orc_e2m1_value(lo + 1);
    p = (v - vlo) / (vhi - vlo);
    return ((unsigned)floor(256.0 * p) + r8 >= 256u) ? lo + 1 : lo;
}

/* ---------------------------------------------------------------- quantizer */

static void orc_put_nibble(uint8_t *row, int64_t k, int code)
{
    if (k & 1) row[k >> 1] = (uint8_t)((row[k >> 1] & 0x0F) | (code << 4));
    else       row[k >> 1] = (uint8_t)((row[k >> 1] & 0xF0) | code);
}

static int orc_get_nibble(const uint8_t *row, int64_t k)
{
    return (k & 1) ? (row[k >> 1] >> 4) : (row[k >> 1] & 0x0F);
}

/*
 * quantize2d: X[rows, cols] BF16 (leading dimension ld_x elements) ->
 *   scale[ceil(rows/32), ld_s]  UE8M0 byte per 32x32 block  (code = e + 127)
 *   q_rm [rows, ld_rm] bytes    element (i,j) = nibble j&1 of q_rm[i*ld_rm + j/2]
 *   q_t  [cols, ld_t ] bytes    element (i,j) = nibble i&1 of q_t [j*ld_t  + i/2]
 * (low nibble = even index; bytes between the logical extent and ld are 0;
 *  q_t may be NULL).  Steps, in the paper's order: block partition B_ij,
 * block maximum M_ij over the valid entries only (boundary blocks),
 * truncation-free scale S_ij, rounding of B_ij/S_ij to E2M1.  The code is
 * written once into both layouts: they share one scale matrix.
 * Non-finite inputs are outside the method; they are given a defined result
 * so that nothing is undefined: M is taken over finite entries, +-Inf takes
 * the largest magnitude with its sign, NaN becomes code 0.
 *
 * The window form processes block rows [I0, I1) and block columns [J0, J1) of
 * the full tensor only and indexes its outputs from the window's origin
 * (output row i - 32*I0, output column j - 32*J0), so that a sample of a large
 * tensor can be produced without the whole; the stochastic-rounding stream is
 * still keyed on the element's index in the full tensor.
 * Returns 0, or -1 on a bad argument.
 */
int orc_quantize2d_window(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld_x,
                          int mode, uint64_t seed, uint32_t tensor_id, uint32_t flags,
                          int64_t I0, int64_t I1, int64_t J0, int64_t J1,
                          uint8_t *q_rm, int64_t ld_rm, uint8_t *q_t, int64_t ld_t,
                          uint8_t *scale, int64_t ld_s)
{
    int64_t rt = (rows + ORC_BLOCK - 1) / ORC_BLOCK, ct = (cols + ORC_BLOCK - 1) / ORC_BLOCK;
    int64_t wr0 = I0 * ORC_BLOCK, wc0 = J0 * ORC_BLOCK, wrows, wcols, I;
    if (rows < 0 || cols < 0 || (mode != ORC_MODE_NEAREST && mode != ORC_MODE_STOCHASTIC)) return -1;
    if (I0 < 0 || J0 < 0 || I1 > rt || J1 > ct) return -1;
    if (rows == 0 || cols == 0 || I0 >= I1 || J0 >= J1) return 0;
    wrows = (I1 * ORC_BLOCK < rows ? I1 * ORC_BLOCK : rows) - wr0;
    wcols = (J1 * ORC_BLOCK < cols ? J1 * ORC_BLOCK : cols) - wc0;
    if (!x || !q_rm || !scale || ld_x < cols || ld_rm < (wcols + 1) / 2 || ld_s < J1 - J0) return -1;
    if (q_t && ld_t < (wrows + 1) / 2) return -1;

    for (I = 0; I < wrows; I++) memset(q_rm + I * ld_rm, 0, (size_t)ld_rm);
    if (q_t) for (I = 0; I < wcols; I++) memset(q_t + I * ld_t, 0, (size_t)ld_t);

    /* blocks of one block-row write disjoint bytes of q_rm and scale; a q_t byte
     * is shared by two adjacent rows, which always lie in the same block-row */
#pragma omp parallel for schedule(static)
    for (I = I0; I < I1; I++) {
        int64_t J;
        for (J = J0; J < J1; J++) {
            int64_t i0 = I * ORC_BLOCK, j0 = J * ORC_BLOCK;
            int64_t i1 = i0 + ORC_BLOCK < rows ? i0 + ORC_BLOCK : rows;
            int64_t j1 = j0 + ORC_BLOCK < cols ? j0 + ORC_BLOCK : cols;
            int64_t i, j;
            double M = 0.0, S;
            int e;
            for (i = i0; i < i1; i++)
                for (j = j0; j < j1; j++) {
                    double a = fabs(orc_bf16_to_double(x[i * ld_x + j]));
                    if (isfinite(a) && a > M) M = a;
                }
            e = orc_scale_exponent(M);
            S = ldexp(1.0, e);
            scale[(I - I0) * ld_s + (J - J0)] = (uint8_t)(e + 127);
            for (i = i0; i < i1; i++)
                for (j = j0; j < j1; j++) {
                    uint16_t bits = x[i * ld_x + j];
                    double a = orc_bf16_to_double(bits);
                    int sign = (bits >> 15) & 1, mag, code;
                    if (isnan(a)) {
                        code = 0;
                    } else {
                        if (isinf(a)) {
                            mag = 7;
                        } else {
                            double v = fabs(a) / S;          /* exact: S is a power of two */
                            if (mode == ORC_MODE_NEAREST) {
                                mag = orc_round_nearest(v);
                            } else {
                                uint64_t idx = (flags & ORC_FLAG_INDEX_TRANSPOSED)
                                                   ? (uint64_t)j * (uint64_t)rows + (uint64_t)i
                                                   : (uint64_t)i * (uint64_t)cols + (uint64_t)j;
                                mag = orc_round_stochastic(v, orc_random_byte(seed, tensor_id, idx));
                            }
                        }
                        code = (sign << 3) | mag;
                    }
                    orc_put_nibble(q_rm + (i - wr0) * ld_rm, j - wc0, code);
                    if (q_t) orc_put_nibble(q_t + (j - wc0) * ld_t, i - wr0, code);
                }
        }
    }
    return 0;
}

int orc_quantize2d(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld_x,
                   int mode, uint64_t seed, uint32_t tensor_id, uint32_t flags,
                   uint8_t *q_rm, int64_t ld_rm, uint8_t *q_t, int64_t ld_t,
                   uint8_t *scale, int64_t ld_s)
{
    return orc_quantize2d_window(x, rows, cols, ld_x, mode, seed, tensor_id, flags,
                                 0, (rows + ORC_BLOCK - 1) / ORC_BLOCK, 0, (cols + ORC_BLOCK - 1) / ORC_BLOCK,
                                 q_rm, ld_rm, q_t, ld_t, scale, ld_s);
}

/* Dequantized values  x^ = S * code value  (appendix "2D Block Scaling ...",
 * the quantized block), exact in double.  transposed = 0 reads q_rm/[rows,cols];
 * the row-major payload is the only one the GEMM oracle reads. */
void orc_dequantize2d(const uint8_t *q_rm, int64_t ld_rm, const uint8_t *scale, int64_t ld_s,
                      int64_t rows, int64_t cols, double *out, int64_t ld_out)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; i++) {
        int64_t j;
        for (j = 0; j < cols; j++) {
            int e = (int)scale[(i / ORC_BLOCK) * ld_s + j / ORC_BLOCK] - 127;
            out[i * ld_out + j] = ldexp(orc_e2m1_value(orc_get_nibble(q_rm + i * ld_rm, j)), e);
        }
    }
}

/* ------------------------------------------------------- block-size variants (b x b, b free) */

/*
 * The 2D scheme with another block size (the block-size study, Table 4: 8 / 16 / 32 / 64): the matrix is cut into
 * b x b blocks, each with one truncation-free power-of-two scale; everything else as orc_quantize2d (E2M1 codes,
 * nearest-even or stochastic rounding with the random byte of the element's index, +-Inf -> +-6, NaN -> +0, block
 * maximum over finite entries, out-of-range entries excluded).  scale[ceil(rows/b), ld_s >= ceil(cols/b)].
 * q_rm[rows, ld_rm >= ceil(cols/2)], q_t[cols, ld_t >= ceil(rows/2)] or NULL; payload rows are cleared first.
 */
int orc_quantize2d_block(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld_x, int block, int mode, uint64_t seed,
                         uint32_t tensor_id, uint32_t flags, uint8_t *q_rm, int64_t ld_rm, uint8_t *q_t, int64_t ld_t,
                         uint8_t *scale, int64_t ld_s)
{
    int64_t rt, ct, I, i;
    if (block < 1 || rows < 0 || cols < 0 || (mode != ORC_MODE_NEAREST && mode != ORC_MODE_STOCHASTIC)) return -1;
    if (rows == 0 || cols == 0) return 0;
    rt = (rows + block - 1) / block;
    ct = (cols + block - 1) / block;
    if (!x || !q_rm || !scale || ld_x < cols || ld_rm < (cols + 1) / 2 || ld_s < ct) return -1;
    if (q_t && ld_t < (rows + 1) / 2) return -1;
    for (i = 0; i < rows; i++) memset(q_rm + i * ld_rm, 0, (size_t)ld_rm);
    if (q_t)
        for (i = 0; i < cols; i++) memset(q_t + i * ld_t, 0, (size_t)ld_t);
    for (I = 0; I < rt; I++) {
        int64_t J;
        for (J = 0; J < ct; J++) {
            int64_t i0 = I * block, j0 = J * block, j;
            int64_t i1 = i0 + block < rows ? i0 + block : rows, j1 = j0 + block < cols ? j0 + block : cols;
            double M = 0.0, S;
            int e;
            for (i = i0; i < i1; i++)
                for (j = j0; j < j1; j++) {
                    double a = fabs(orc_bf16_to_double(x[i * ld_x + j]));
                    if (isfinite(a) && a > M) M = a;
                }
            e = orc_scale_exponent(M);
            S = ldexp(1.0, e);
            scale[I * ld_s + J] = (uint8_t)(e + 127);
            for (i = i0; i < i1; i++)
                for (j = j0; j < j1; j++) {
                    uint16_t bits = x[i * ld_x + j];
                    double a = orc_bf16_to_double(bits);
                    int sign = (bits >> 15) & 1, mag, code;
                    if (isnan(a)) {
                        code = 0;
                    } else {
                        if (isinf(a)) {
                            mag = 7;
                        } else if (mode == ORC_MODE_NEAREST) {
                            mag = orc_round_nearest(fabs(a) / S);
                        } else {
                            uint64_t idx = (flags & ORC_FLAG_INDEX_TRANSPOSED) ? (uint64_t)j * (uint64_t)rows + (uint64_t)i
                                                                               : (uint64_t)i * (uint64_t)cols + (uint64_t)j;
                            mag = orc_round_stochastic(fabs(a) / S, orc_random_byte(seed, tensor_id, idx));
                        }
                        code = (sign << 3) | mag;
                    }
                    orc_put_nibble(q_rm + i * ld_rm, j, code);
                    if (q_t) orc_put_nibble(q_t + j * ld_t, i, code);
                }
        }
    }
    return 0;
}

/* Dequantized values of a b x b block tensor (row-major payload), exact in double. */
void orc_dequantize2d_block(const uint8_t *q_rm, int64_t ld_rm, const uint8_t *scale, int64_t ld_s, int block,
                            int64_t rows, int64_t cols, double *out, int64_t ld_out)
{
    int64_t i, j;
    for (i = 0; i < rows; i++)
        for (j = 0; j < cols; j++) {
            int e = (int)scale[(i / block) * ld_s + j / block] - 127;
            out[i * ld_out + j] = ldexp(orc_e2m1_value(orc_get_nibble(q_rm + i * ld_rm, j)), e);
        }
}

/* ------------------------------------------------------- 1D (1 x 32) FP4 blocks */

/*
 * The activation layout the paper keeps (Section 3, "Application to linear layers": activations stay in 1D
 * blocks; appendix "Quantization Placement", paragraph Activations): one scale per 32 consecutive elements of a row, everything
 * else as in the 2D scheme - truncation-free power-of-two scale, E2M1 codes, nearest-even or stochastic rounding
 * with the random byte of the element's row-major index i*cols + j (j*rows + i with the transposed-index flag).
 * q[rows, ld_q] packed two codes per byte (low nibble = even column), scale[rows, ld_s], ld_s >= ceil(cols/32).
 * +-Inf -> +-6, NaN -> +0, block maximum over finite entries.  Payload bytes up to ld_q are written as 0.
 */
int orc_quantize1d(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld_x, int mode, uint64_t seed,
                   uint32_t tensor_id, uint32_t flags, uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s)
{
    int64_t nb = (cols + ORC_BLOCK - 1) / ORC_BLOCK, i;
    if (rows < 0 || cols < 0 || (mode != ORC_MODE_NEAREST && mode != ORC_MODE_STOCHASTIC)) return -1;
    if (rows == 0 || cols == 0) return 0;
    if (!x || !q || !scale || ld_x < cols || ld_q < (cols + 1) / 2 || ld_s < nb) return -1;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; i++) {
        int64_t b;
        memset(q + i * ld_q, 0, (size_t)ld_q);
        for (b = 0; b < nb; b++) {
            int64_t j0 = b * ORC_BLOCK, j1 = j0 + ORC_BLOCK < cols ? j0 + ORC_BLOCK : cols, j;
            double M = 0.0, S;
            int e;
            for (j = j0; j < j1; j++) {
                double a = fabs(orc_bf16_to_double(x[i * ld_x + j]));
                if (isfinite(a) && a > M) M = a;
            }
            e = orc_scale_exponent(M);
            S = ldexp(1.0, e);
            scale[i * ld_s + b] = (uint8_t)(e + 127);
            for (j = j0; j < j1; j++) {
                uint16_t bits = x[i * ld_x + j];
                double a = orc_bf16_to_double(bits);
                int sign = (bits >> 15) & 1, mag, code;
                if (isnan(a)) {
                    code = 0;
                } else {
                    if (isinf(a)) {
                        mag = 7;
                    } else if (mode == ORC_MODE_NEAREST) {
                        mag = orc_round_nearest(fabs(a) / S);
                    } else {
                        uint64_t idx = (flags & ORC_FLAG_INDEX_TRANSPOSED) ? (uint64_t)j * (uint64_t)rows + (uint64_t)i
                                                                           : (uint64_t)i * (uint64_t)cols + (uint64_t)j;
                        mag = orc_round_stochastic(fabs(a) / S, orc_random_byte(seed, tensor_id, idx));
                    }
                    code = (sign << 3) | mag;
                }
                orc_put_nibble(q + i * ld_q, j, code);
            }
        }
    }
    return 0;
}

/* Dequantized values of a 1D-block tensor, exact in double. */
void orc_dequantize1d(const uint8_t *q, int64_t ld_q, const uint8_t *scale, int64_t ld_s, int64_t rows, int64_t cols,
                      double *out, int64_t ld_out)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; i++) {
        int64_t j;
        for (j = 0; j < cols; j++) {
            int e = (int)scale[i * ld_s + j / ORC_BLOCK] - 127;
            out[i * ld_out + j] = ldexp(orc_e2m1_value(orc_get_nibble(q + i * ld_q, j)), e);
        }
    }
}

/* -------------------------------------------------------------------- MXFP8 */

/* Nearest E4M3 magnitude code (0x00..0x7E) for v in [0, 448], ties to the even
 * code, by brute force over every finite magnitude. */
int orc_round_nearest_e4m3(double v)
{
    int best = 0, c;
    double bestd = fabs(v - orc_e4m3_value(0));
    for (c = 1; c <= 0x7E; c++) {
        double d = fabs(v - orc_e4m3_value(c));
        if (d < bestd || (d == bestd && (c & 1) == 0 && (best & 1) == 1)) {
            best = c;
            bestd = d;
        }
    }
    return best;
}

/*
 * MXFP8 operand (Section 3.2: Q and K projections): X[rows, cols] BF16 ->
 * E4M3 payload q[rows, ld_q] and one UE8M0 scale per 32 consecutive elements
 * of a row, scale[rows, ld_s] with ld_s >= ceil(cols/32).  The block scale
 * follows the same truncation-free rule with the E4M3 bound 448; rounding is
 * to nearest, ties to even.  Payload bytes between cols and ld_q are 0.
 * +-Inf -> +-448, NaN -> 0, block maximum over finite entries.
 */
int orc_mxfp8_quantize1d(const uint16_t *x, int64_t rows, int64_t cols, int64_t ld_x,
                         uint8_t *q, int64_t ld_q, uint8_t *scale, int64_t ld_s)
{
    int64_t nb = (cols + ORC_BLOCK - 1) / ORC_BLOCK, i;
    if (rows < 0 || cols < 0) return -1;
    if (rows == 0 || cols == 0) return 0;
    if (!x || !q || !scale || ld_x < cols || ld_q < cols || ld_s < nb) return -1;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; i++) {
        int64_t b, j;
        memset(q + i * ld_q, 0, (size_t)ld_q);
        for (b = 0; b < nb; b++) {
            int64_t j0 = b * ORC_BLOCK, j1 = j0 + ORC_BLOCK < cols ? j0 + ORC_BLOCK : cols;
            double M = 0.0, S;
            int e;
            for (j = j0; j < j1; j++) {
                double a = fabs(orc_bf16_to_double(x[i * ld_x + j]));
                if (isfinite(a) && a > M) M = a;
            }
            e = orc_mxfp8_scale_exponent(M);
            S = ldexp(1.0, e);
            scale[i * ld_s + b] = (uint8_t)(e + 127);
            for (j = j0; j < j1; j++) {
                uint16_t bits = x[i * ld_x + j];
                double a = orc_bf16_to_double(bits);
                int sign = (bits >> 15) & 1, code;
                if (isnan(a)) code = 0;
                else if (isinf(a)) code = (sign << 7) | 0x7E;
                else code = (sign << 7) | orc_round_nearest_e4m3(fabs(a) / S);
                q[i * ld_q + j] = (uint8_t)code;
            }
        }
    }
    return 0;
}

void orc_mxfp8_dequantize(const uint8_t *q, int64_t ld_q, const uint8_t *scale, int64_t ld_s,
                          int64_t rows, int64_t cols, double *out, int64_t ld_out)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < rows; i++) {
        int64_t j;
        for (j = 0; j < cols; j++) {
            int e = (int)scale[i * ld_s + j / ORC_BLOCK] - 127;
            out[i * ld_out + j] = ldexp(orc_e4m3_value(q[i * ld_q + j]), e);
        }
    }
}

/* --------------------------------------------------------------------- GEMM */

/* C[m, n] = sum_k A[m, k] * B[n, k]  in double: the textbook definition that
 * all three linear-layer products reduce to once the operands are laid out as
 * (output row) x (contraction):
 *   forward  Y  = X^  W^^T          A = X^ [T,K],     B = W^ [N,K]
 *   dgrad    dX = dY^ W^            A = dY^[T,N],     B = W^^T [K,N]
 *   wgrad    dW = dY^^T X^          A = dY^^T [N,T],  B = X^^T [K,T]
 * (Section 3, "Application to linear layers").  Callers form the transposes
 * explicitly. */
void orc_gemm_nt(const double *A, const double *B, double *C, int64_t M, int64_t N, int64_t K)
{
    int64_t m;
#pragma omp parallel for schedule(static)
    for (m = 0; m < M; m++) {
        int64_t n, k;
        for (n = 0; n < N; n++) {
            double acc = 0.0;
            for (k = 0; k < K; k++) acc += A[m * K + k] * B[n * K + k];
            C[m * N + n] = acc;
        }
    }
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
