/*
 * CPU oracle for the stochastically-rounded quantized linear layer.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what
 * the method computes; it exists so that the CUDA library can be checked
 * against it element by element.  It shares no code, header, table or
 * constant generator with the CUDA path, and the product never calls it.
 *
 * Every function follows one passage of the paper ("Training with Fewer
 * Bits: Unlocking Edge LLMs Training with Stochastic Rounding"):
 *   - Def. 1  threshold quantizer  Q_D(x, eps)
 *   - Def. 2  round-to-nearest     eps = 1/2, ties toward +infinity
 *   - Def. 3  stochastic rounding  eps ~ U[0,1], independent per element
 *   - Sec. 2.2.2  mixed-precision matmul = exact product of the two
 *                 quantized matrices (low-precision multiply, wide accumulate)
 *   - Alg. 1  forward   A_out = Q(A_in) Q(W)
 *   - Alg. 2  backward  dA_in = Q(dA_out) Q(W)^T,  dW = Q(A_in)^T Q(dA_out)
 *
 * Storage convention (the usual deep-learning one, transposed with respect
 * to the paper's W[in,out]):  A[T,K], W[N,K], dY[T,N];  Y[T,N] = A W^T,
 * dA[T,K] = dY W,  dW[N,K] = dY^T A.
 *
 * Floating point: the rounding decision is taken in IEEE binary32 with
 * round-to-nearest and no fused multiply-add (compile with
 * -ffp-contract=off), because the decision yields an integer code and both
 * sides of a parity test must take it in the same precision.  bfloat16
 * inputs are widened to binary32 (exactly) by the caller.
 *
 * The step size D of a group g of elements is not fixed by the paper (D is
 * a free "precision level" in Def. 1); it is the symmetric absmax rule
 * D_g = max_g|x| / qmax,  qmax = 2^(bits-1) - 1,  codes in [-qmax, qmax].
 *
 * Pins for every function here live in tests/test_oracle_*.py.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_PER_TENSOR 0
#define ORC_PER_ROW 1
#define ORC_SR 0
#define ORC_RTN 1
#define ORC_SR8 2   /* stochastic rounding with 8 random bits per element */

/* ---------------------------------------------------------------------- */
/* Thresholds eps (Def. 3): counter-based Philox4x32-10                     */
/* (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as       */
/* 1, 2, 3", SC'11).  A 128-bit counter and a 64-bit key give four 32-bit  */
/* words after ten rounds; the key is bumped by the Weyl constants between */
/* rounds.                                                                 */
/* ---------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
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

/*
 * The 24-bit threshold of the element with flat index i (row-major index of
 * the SOURCE tensor plus index_offset): Philox block j = i >> 2 with counter
 * {lo(j), hi(j), lo(tensor_id), hi(tensor_id)} and key {lo(seed), hi(seed)};
 * the element takes word i & 3, and its top 24 bits u24 stand for
 * eps = u24 * 2^-24 in [0, 1).
 */
uint32_t orc_threshold_u24(uint64_t seed, uint64_t tensor_id, uint64_t i)
{
    uint64_t j = i >> 2;
    uint32_t ctr[4] = { (uint32_t)j, (uint32_t)(j >> 32),
                        (uint32_t)tensor_id, (uint32_t)(tensor_id >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return out[i & 3] >> 8;
}

/*
 * Thresholds with 8 random bits per element.  The paper's hardware section
 * argues that a rounding unit needs only a few pseudo-random bits (its FPGA
 * estimate uses a 6-bit LFSR); this variant takes eps = (b + 1/2) / 256 with b
 * one byte of the Philox stream, so that one 128-bit block serves 16 elements:
 * block j = i >> 4, word (i >> 2) & 3 of it, byte i & 3 of that word (least
 * significant byte first).  Returned on the 2^-24 lattice of orc_threshold_u24,
 * (2 b + 1) 2^15, so that the same comparison rule applies.  The half offset
 * centres the 256 thresholds: P(round up) is then the fraction rounded to the
 * nearest multiple of 1/256 (ties down), within 2^-9 of it and without a
 * systematic sign.
 */
uint32_t orc_threshold_sr8(uint64_t seed, uint64_t tensor_id, uint64_t i)
{
    uint64_t j = i >> 4;
    uint32_t ctr[4] = { (uint32_t)j, (uint32_t)(j >> 32),
                        (uint32_t)tensor_id, (uint32_t)(tensor_id >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    uint32_t b = (out[(i >> 2) & 3] >> (8 * (i & 3))) & 0xFFu;
    return (2u * b + 1u) << 15;
}

/* Threshold of element i on the 2^-24 lattice for the given rounding mode (0 for RTN). */
static uint32_t orc_threshold(int round_mode, uint64_t seed, uint64_t tensor_id, uint64_t i)
{
    if (round_mode == ORC_SR) return orc_threshold_u24(seed, tensor_id, i);
    if (round_mode == ORC_SR8) return orc_threshold_sr8(seed, tensor_id, i);
    return 0u;
}

/* ---------------------------------------------------------------------- */
/* Step size (absmax rule)                                                  */
/* ---------------------------------------------------------------------- */
static int orc_qmax(int bits) { return (1 << (bits - 1)) - 1; }

/*
 * D = m / qmax (one binary32 division, round to nearest) and the reciprocal
 * actually multiplied in, inv = qmax / m ROUNDED TOWARD ZERO: the largest
 * binary32 number not above qmax / m.  Def. 1 has no saturation: with
 * D = m / qmax every |x / D| of the group is at most qmax.  Rounding the
 * reciprocal toward zero keeps that property for the computed quotient
 * (|x| <= m gives |x * inv| <= m * inv <= qmax in real numbers, and rounding
 * the product to binary32 cannot pass the representable number qmax), so no
 * code ever leaves [-qmax, qmax].  A reciprocal rounded to nearest would let
 * the extreme element overshoot qmax by an ulp and force a clamp that the
 * definition does not have.
 * m = 0 is Def. 1's D = 0 case (Q_0 is the identity, and the group is all
 * zeros, so codes 0 with scale 0 reproduce it).  A group whose absmax is so
 * small that qmax / m overflows binary32 (m below about 4e-37) is treated
 * the same way.
 */
void orc_scale_from_absmax(float m, int bits, float *delta, float *inv)
{
    float qmax = (float)orc_qmax(bits);
    float r = (m == 0.0f) ? 0.0f : qmax / m;
    if (isinf(r) || r != r) r = 0.0f;
    /* the product of two binary32 numbers is exact in binary64 */
    if (r != 0.0f && (double)r * (double)m > (double)qmax) r = nextafterf(r, 0.0f);
    *inv = r;
    *delta = (r == 0.0f) ? 0.0f : m / qmax;
}

/* ---------------------------------------------------------------------- */
/* Def. 1-3: one element                                                    */
/* ---------------------------------------------------------------------- */
/*
 * Code q such that Q_D(x, eps) = q * D, with x/D evaluated as t = x * inv
 * (one binary32 multiply).  With f = floor(t) and the fractional part
 * p = t - f:
 *   SR : round up  iff  eps < p   (strict, so grid-exact x never moves;
 *        Def. 1 rounds down when p < eps, up otherwise; with eps on a
 *        2^-24 lattice the strict form keeps P(up) within 2^-24 of p)
 *   RTN: round up  iff  p >= 1/2  (Def. 1 with eps = 1/2; a tie goes up,
 *        i.e. toward +infinity, Def. 2)
 * Def. 1 states these comparisons on real numbers, so they are evaluated
 * without rounding p: multiplied through by 2^24, eps < t - f becomes
 * u24 + f 2^24 < t 2^24, and every term of that is exact in binary64
 * (t has 24 significant bits, f is an integer of magnitude <= 2^8).
 *   q = f + up.  With inv from orc_scale_from_absmax and |x| <= absmax the
 *   result is always inside [-qmax, qmax]; the clamp below only matters for
 *   callers that pass some other inv.
 */
int orc_quantize_scalar(float x, float inv, int bits, int round_mode, uint32_t u24)
{
    int qmax = orc_qmax(bits);
    float t = x * inv;
    double td = (double)t;
    double f = floor(td);
    int up;
    if (round_mode == ORC_SR || round_mode == ORC_SR8)
        up = ((double)u24 + f * 0x1p24) < td * 0x1p24;
    else
        up = (f * 0x1p24 + 0x1p23) <= td * 0x1p24;
    int q = (int)f + up;
    if (q > qmax) q = qmax;
    if (q < -qmax) q = -qmax;
    return q;
}

/*
 * Sum of the SR codes of x over all 2^24 possible thresholds.  With eps
 * uniform on the lattice (Def. 3), E[q] = sum / 2^24 exactly; the tests use
 * it to check P(round up) without sampling.
 */
int64_t orc_sum_sr_codes_over_all_thresholds(float x, float inv, int bits)
{
    int64_t sum = 0;
    for (uint32_t u = 0; u < (1u << 24); ++u)
        sum += orc_quantize_scalar(x, inv, bits, ORC_SR, u);
    return sum;
}

/* ---------------------------------------------------------------------- */
/* absmax over the three kinds of group                                     */
/* ---------------------------------------------------------------------- */
void orc_absmax_tensor(const float *x, int64_t rows, int64_t cols, int64_t ld, float *m)
{
    float best = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float a = fabsf(x[r * ld + c]);
            if (a > best) best = a;
        }
    m[0] = best;
}

void orc_absmax_rows(const float *x, int64_t rows, int64_t cols, int64_t ld, float *m)
{
    for (int64_t r = 0; r < rows; ++r) {
        float best = 0.0f;
        for (int64_t c = 0; c < cols; ++c) {
            float a = fabsf(x[r * ld + c]);
            if (a > best) best = a;
        }
        m[r] = best;
    }
}

void orc_absmax_cols(const float *x, int64_t rows, int64_t cols, int64_t ld, float *m)
{
    for (int64_t c = 0; c < cols; ++c) m[c] = 0.0f;
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c) {
            float a = fabsf(x[r * ld + c]);
            if (a > m[c]) m[c] = a;
        }
}

/* ---------------------------------------------------------------------- */
/* Matrix quantizer (Def. 3, "matrix stochastic rounding is element-wise") */
/* ---------------------------------------------------------------------- */
/*
 * x[rows, cols] (row pitch ld) -> int8 codes in either or both layouts.
 *
 *   codes_rm[rows, cols] with scale_rm: [1] (per tensor) or [rows] (one step
 *       size per row);
 *   codes_tr[cols, rows] (the transpose) with scale_tr: [1] or [cols] (one
 *       step size per COLUMN of x, i.e. per row of the transposed view).
 *
 * A step size can be pulled out of a matrix product only if it is constant
 * along the contracted axis, which is the contiguous axis of each layout;
 * hence "per row" always means per row of the layout being written.  Per
 * tensor, both layouts hold the same codes.  Either way the element x[r,c]
 * uses ONE threshold, that of flat index index_offset + r*cols + c, for both
 * layouts (one eps per element per quantization point, Alg. 2).
 *
 * Any output pointer pair may be NULL.  Returns 0, or 1 if bits is outside
 * 2..8.
 */
int orc_sr_quantize(const float *x, int64_t rows, int64_t cols, int64_t ld,
                    int bits, int scale_mode, int round_mode,
                    uint64_t seed, uint64_t tensor_id, uint64_t index_offset,
                    int8_t *codes_rm, float *scale_rm,
                    int8_t *codes_tr, float *scale_tr)
{
    if (bits < 2 || bits > 8) return 1;
    float m_tensor = 0.0f;
    if (scale_mode == ORC_PER_TENSOR) orc_absmax_tensor(x, rows, cols, ld, &m_tensor);

    if (codes_rm) {
        if (scale_mode == ORC_PER_TENSOR) {
            float delta, inv;
            orc_scale_from_absmax(m_tensor, bits, &delta, &inv);
            scale_rm[0] = delta;
        } else {
            orc_absmax_rows(x, rows, cols, ld, scale_rm); /* holds absmax for now */
        }
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < rows; ++r) {
            float delta, inv;
            if (scale_mode == ORC_PER_TENSOR) {
                orc_scale_from_absmax(m_tensor, bits, &delta, &inv);
            } else {
                orc_scale_from_absmax(scale_rm[r], bits, &delta, &inv);
                scale_rm[r] = delta;
            }
            for (int64_t c = 0; c < cols; ++c) {
                uint64_t i = index_offset + (uint64_t)r * (uint64_t)cols + (uint64_t)c;
                uint32_t u24 = orc_threshold(round_mode, seed, tensor_id, i);
                codes_rm[r * cols + c] =
                    (int8_t)orc_quantize_scalar(x[r * ld + c], inv, bits, round_mode, u24);
            }
        }
    }

    if (codes_tr) {
        if (scale_mode == ORC_PER_TENSOR) {
            float delta, inv;
            orc_scale_from_absmax(m_tensor, bits, &delta, &inv);
            scale_tr[0] = delta;
        } else {
            orc_absmax_cols(x, rows, cols, ld, scale_tr);
        }
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < cols; ++c) {
            float delta, inv;
            if (scale_mode == ORC_PER_TENSOR) {
                orc_scale_from_absmax(m_tensor, bits, &delta, &inv);
            } else {
                orc_scale_from_absmax(scale_tr[c], bits, &delta, &inv);
                scale_tr[c] = delta;
            }
            for (int64_t r = 0; r < rows; ++r) {
                uint64_t i = index_offset + (uint64_t)r * (uint64_t)cols + (uint64_t)c;
                uint32_t u24 = orc_threshold(round_mode, seed, tensor_id, i);
                codes_tr[c * rows + r] =
                    (int8_t)orc_quantize_scalar(x[r * ld + c], inv, bits, round_mode, u24);
            }
        }
    }
    return 0;
}

/* ---------------------------------------------------------------------- */
/* Sec. 2.2.2: product of two code matrices, both stored with the           */
/* contracted axis contiguous:  acc[i,j] = sum_k a[i,k] * b[j,k].           */
/* The sum is formed in 64 bits; the return value counts entries that do    */
/* not fit in 32 bits (a caller precondition, 0 in every valid use).        */
/* ---------------------------------------------------------------------- */
int64_t orc_gemm_i8_nt(const int8_t *a, const int8_t *b, int64_t M, int64_t N, int64_t Kc,
                       int32_t *acc)
{
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            int64_t s = 0;
            for (int64_t k = 0; k < Kc; ++k)
                s += (int64_t)a[i * Kc + k] * (int64_t)b[j * Kc + k];
            if (s > INT32_MAX || s < INT32_MIN) overflow += 1;
            acc[i * N + j] = (int32_t)s;
        }
    return overflow;
}

/*
 * Value of the product of the two quantized matrices: the integer sum times
 * the two step sizes,  out[i,j] = float(acc[i,j]) * (s_row[i] * s_col[j]),
 * each operation one binary32 rounding, the scale product formed first.
 * row_stride / col_stride are 0 for a per-tensor scale and 1 for per-row.
 */
void orc_dequant(const int32_t *acc, int64_t M, int64_t N,
                 const float *s_row, int row_stride, const float *s_col, int col_stride,
                 float *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            float s = s_row[i * row_stride] * s_col[j * col_stride];
            out[i * N + j] = (float)acc[i * N + j] * s;
        }
}

/* ---------------------------------------------------------------------- */
/* One quantization point = (bits, scale mode, rounding mode, seed, id,    */
/* index offset): the paper's (Delta, eps) for one operand.                 */
/* ---------------------------------------------------------------------- */
typedef struct {
    int32_t bits;
    int32_t scale_mode;
    int32_t round_mode;
    int32_t reserved;
    uint64_t seed;
    uint64_t tensor_id;
    uint64_t index_offset;
} orc_qspec;

/*
 * Alg. 1:  Y[T,N] = Q(A) Q(W)^T.  Caller provides scratch for the codes,
 * scales (T and N floats, of which one is used per tensor) and accumulators,
 * which are outputs too.  Returns the overflow count of the product.
 */
int64_t orc_qlinear_fwd(const float *A, const float *W, int64_t T, int64_t N, int64_t K,
                        const orc_qspec *qa, const orc_qspec *qw,
                        int8_t *codes_a /*[T,K]*/, float *scale_a,
                        int8_t *codes_w /*[N,K]*/, float *scale_w,
                        int32_t *acc /*[T,N]*/, float *Y /*[T,N]*/)
{
    orc_sr_quantize(A, T, K, K, qa->bits, qa->scale_mode, qa->round_mode, qa->seed, qa->tensor_id,
                    qa->index_offset, codes_a, scale_a, NULL, NULL);
    orc_sr_quantize(W, N, K, K, qw->bits, qw->scale_mode, qw->round_mode, qw->seed, qw->tensor_id,
                    qw->index_offset, codes_w, scale_w, NULL, NULL);
    int64_t ov = orc_gemm_i8_nt(codes_a, codes_w, T, N, K, acc);
    orc_dequant(acc, T, N, scale_a, qa->scale_mode == ORC_PER_ROW, scale_w,
                qw->scale_mode == ORC_PER_ROW, Y);
    return ov;
}

/*
 * Alg. 2, input gradient:  dA[T,K] = Q(dY) Q(W).  The contraction runs over
 * N, so W is taken in its transposed layout W^T[K,N] (per-row scale = one
 * per input feature k).
 */
int64_t orc_qlinear_bwd_input(const float *dY, const float *W, int64_t T, int64_t N, int64_t K,
                              const orc_qspec *qdy, const orc_qspec *qw,
                              int8_t *codes_dy /*[T,N]*/, float *scale_dy,
                              int8_t *codes_wt /*[K,N]*/, float *scale_wt,
                              int32_t *acc /*[T,K]*/, float *dA /*[T,K]*/)
{
    orc_sr_quantize(dY, T, N, N, qdy->bits, qdy->scale_mode, qdy->round_mode, qdy->seed,
                    qdy->tensor_id, qdy->index_offset, codes_dy, scale_dy, NULL, NULL);
    orc_sr_quantize(W, N, K, K, qw->bits, qw->scale_mode, qw->round_mode, qw->seed, qw->tensor_id,
                    qw->index_offset, NULL, NULL, codes_wt, scale_wt);
    int64_t ov = orc_gemm_i8_nt(codes_dy, codes_wt, T, K, N, acc);
    orc_dequant(acc, T, K, scale_dy, qdy->scale_mode == ORC_PER_ROW, scale_wt,
                qw->scale_mode == ORC_PER_ROW, dA);
    return ov;
}

/*
 * Alg. 2, weight gradient:  dW[N,K] = Q(dY)^T Q(A).  The contraction runs
 * over the T samples (the axis along which the SR noise averages out), so
 * both operands are taken in their transposed layouts dY^T[N,T], A^T[K,T].
 */
int64_t orc_qlinear_bwd_weight(const float *dY, const float *A, int64_t T, int64_t N, int64_t K,
                               const orc_qspec *qdy, const orc_qspec *qa,
                               int8_t *codes_dyt /*[N,T]*/, float *scale_dyt,
                               int8_t *codes_at /*[K,T]*/, float *scale_at,
                               int32_t *acc /*[N,K]*/, float *dW /*[N,K]*/)
{
    orc_sr_quantize(dY, T, N, N, qdy->bits, qdy->scale_mode, qdy->round_mode, qdy->seed,
                    qdy->tensor_id, qdy->index_offset, NULL, NULL, codes_dyt, scale_dyt);
    orc_sr_quantize(A, T, K, K, qa->bits, qa->scale_mode, qa->round_mode, qa->seed, qa->tensor_id,
                    qa->index_offset, NULL, NULL, codes_at, scale_at);
    int64_t ov = orc_gemm_i8_nt(codes_dyt, codes_at, N, K, T, acc);
    orc_dequant(acc, N, K, scale_dyt, qdy->scale_mode == ORC_PER_ROW, scale_at,
                qa->scale_mode == ORC_PER_ROW, dW);
    return ov;
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ====================================================================== */
/* E4M3 grid (the 8-bit floating-point formats of the paper's experiments  */
/* section are E4M0 / E4M1 / E4M2; E4M3 is the member of that family the    */
/* tensor cores multiply natively).  Format: 1 sign bit, 4 exponent bits    */
/* with bias 7, 3 mantissa bits, subnormals at exponent field 0, no         */
/* infinities, largest finite value 448 (exponent field 15, mantissa 6).    */
/* ====================================================================== */

/* Value of an E4M3 code byte, written out from the format's definition.
 * The two NaN codes (0x7f, 0xff) return NaN. */
double orc_e4m3_decode(uint8_t code)
{
    int sign = code >> 7, ex = (code >> 3) & 15, man = code & 7;
    double v;
    if (ex == 15 && man == 7) return NAN;
    if (ex == 0) v = ldexp((double)man, -9);            /* subnormal: man/8 * 2^-6 */
    else v = ldexp(1.0 + man / 8.0, ex - 7);
    return sign ? -v : v;
}

/* Code byte of a value that lies on the E4M3 grid (|v| <= 448); zero is +0. */
static uint8_t orc_e4m3_encode_on_grid(double v)
{
    if (v == 0.0) return 0;
    uint8_t sign = v < 0 ? 0x80 : 0;
    double a = fabs(v);
    int ex2;
    double m = frexp(a, &ex2);          /* a = m 2^ex2, m in [0.5, 1) */
    int e = ex2 - 1;                    /* a in [2^e, 2^(e+1)) */
    if (e < -6) return (uint8_t)(sign | (int)ldexp(a, 9));            /* subnormal: a / 2^-9 */
    int man = (int)ldexp(m, 4) - 8;                                   /* (a / 2^e - 1) * 8 */
    return (uint8_t)(sign | ((e + 7) << 3) | man);
}

/*
 * The narrower members E4M2, E4M1, E4M0 (the formats of the paper's experiments section, which
 * names them without defining them).  Reading used here: E4Mk keeps the sign, the four exponent
 * bits and the bias of E4M3 and has k mantissa bits, i.e. its values are the E4M3 values whose
 * low 3 - k mantissa bits are zero: inside binade e the spacing is 2^(e-k), the subnormal
 * spacing (below 2^-6) is 2^(-6-k), and the largest finite value is the largest such E4M3
 * value: 448 for k = 3 and 2 (1.75 2^8), 384 for k = 1 (1.5 2^8), 256 for k = 0 (2^8).
 * Codes are stored as E4M3 bytes, so that one product routine serves all four.
 */
double orc_e4m_max(int mant)
{
    return mant >= 2 ? 448.0 : (mant == 1 ? 384.0 : 256.0);
}

/*
 * Def. 1 on the E4Mk grid.  The grid is uniform inside each binade, so the
 * precision level of Def. 1 is taken locally: for t = x * inv with
 * 2^e <= |t| < 2^(e+1) (e clamped to [-6, 8]; below 2^-6 the subnormal spacing
 * continues) the step is D = 2^(e-k), and Q_D(t, eps) is exactly the rule of
 * orc_quantize_scalar applied to u = t / D: round up (toward +infinity) iff
 * eps < frac(u) for SR, iff frac(u) >= 1/2 for RTN.  Both neighbours D floor(u)
 * and D (floor(u) + 1) are grid values (a binade's upper end is the next
 * binade's first value).  Scaling by D is exact, and the comparison is
 * evaluated in binary64 where every term is exact.  Returns the E4M3 code byte.
 */
uint8_t orc_quantize_e4m_scalar(float x, float inv, int mant, int round_mode, uint32_t u24)
{
    float t = x * inv;
    double td = (double)t, a = fabs(td);
    if (a == 0.0) return 0;
    int ex2;
    (void)frexp(a, &ex2);
    int e = ex2 - 1;
    if (e < -6) e = -6;
    if (e > 8) e = 8;
    double u = ldexp(td, mant - e);              /* t / D, exact */
    double f = floor(u);
    int up;
    if (round_mode == ORC_SR || round_mode == ORC_SR8)
        up = ((double)u24 + f * 0x1p24) < u * 0x1p24;
    else
        up = (f * 0x1p24 + 0x1p23) <= u * 0x1p24;
    double v = ldexp(f + up, e - mant);
    double top = orc_e4m_max(mant);
    if (v > top) v = top;                        /* unreachable with inv from orc_scale_e4m */
    if (v < -top) v = -top;
    return orc_e4m3_encode_on_grid(v);
}

uint8_t orc_quantize_e4m3_scalar(float x, float inv, int round_mode, uint32_t u24)
{
    return orc_quantize_e4m_scalar(x, inv, 3, round_mode, u24);
}

/* Step size D = m / top (round to nearest), top the largest value of the grid, and the reciprocal
 * multiplied in, top / m rounded toward zero, so that |x * inv| <= top for the whole group
 * (same reasoning as orc_scale_from_absmax). */
void orc_scale_e4m(float m, int mant, float *delta, float *inv)
{
    float top = (float)orc_e4m_max(mant);
    float r = (m == 0.0f) ? 0.0f : top / m;
    if (isinf(r) || r != r) r = 0.0f;
    if (r != 0.0f && (double)r * (double)m > (double)top) r = nextafterf(r, 0.0f);
    *inv = r;
    *delta = (r == 0.0f) ? 0.0f : m / top;
}

void orc_scale_e4m3(float m, float *delta, float *inv)
{
    orc_scale_e4m(m, 3, delta, inv);
}

/*
 * Matrix form, same conventions as orc_sr_quantize (two layouts, per-tensor
 * or per-row step sizes, one threshold per element by flat source index);
 * codes are E4M3 bytes.
 */
int orc_sr_quantize_e4m(const float *x, int64_t rows, int64_t cols, int64_t ld,
                        int mant, int scale_mode, int round_mode,
                        uint64_t seed, uint64_t tensor_id, uint64_t index_offset,
                        uint8_t *codes_rm, float *scale_rm,
                        uint8_t *codes_tr, float *scale_tr)
{
    float m_tensor = 0.0f;
    if (scale_mode == ORC_PER_TENSOR) orc_absmax_tensor(x, rows, cols, ld, &m_tensor);
    if (codes_rm) {
        if (scale_mode == ORC_PER_ROW) orc_absmax_rows(x, rows, cols, ld, scale_rm);
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < rows; ++r) {
            float delta, inv;
            orc_scale_e4m(scale_mode == ORC_PER_TENSOR ? m_tensor : scale_rm[r], mant, &delta, &inv);
            if (scale_mode == ORC_PER_ROW) scale_rm[r] = delta;
            else if (r == 0) scale_rm[0] = delta;
            for (int64_t c = 0; c < cols; ++c) {
                uint64_t i = index_offset + (uint64_t)r * (uint64_t)cols + (uint64_t)c;
                uint32_t u24 = orc_threshold(round_mode, seed, tensor_id, i);
                codes_rm[r * cols + c] = orc_quantize_e4m_scalar(x[r * ld + c], inv, mant, round_mode, u24);
            }
        }
        if (scale_mode == ORC_PER_TENSOR && rows == 0) { float d, iv; orc_scale_e4m(m_tensor, mant, &d, &iv); scale_rm[0] = d; }
    }
    if (codes_tr) {
        if (scale_mode == ORC_PER_ROW) orc_absmax_cols(x, rows, cols, ld, scale_tr);
#pragma omp parallel for schedule(static)
        for (int64_t c = 0; c < cols; ++c) {
            float delta, inv;
            orc_scale_e4m(scale_mode == ORC_PER_TENSOR ? m_tensor : scale_tr[c], mant, &delta, &inv);
            if (scale_mode == ORC_PER_ROW) scale_tr[c] = delta;
            else if (c == 0) scale_tr[0] = delta;
            for (int64_t r = 0; r < rows; ++r) {
                uint64_t i = index_offset + (uint64_t)r * (uint64_t)cols + (uint64_t)c;
                uint32_t u24 = orc_threshold(round_mode, seed, tensor_id, i);
                codes_tr[c * rows + r] = orc_quantize_e4m_scalar(x[r * ld + c], inv, mant, round_mode, u24);
            }
        }
    }
    return 0;
}

int orc_sr_quantize_e4m3(const float *x, int64_t rows, int64_t cols, int64_t ld,
                         int scale_mode, int round_mode,
                         uint64_t seed, uint64_t tensor_id, uint64_t index_offset,
                         uint8_t *codes_rm, float *scale_rm,
                         uint8_t *codes_tr, float *scale_tr)
{
    return orc_sr_quantize_e4m(x, rows, cols, ld, 3, scale_mode, round_mode, seed, tensor_id, index_offset,
                               codes_rm, scale_rm, codes_tr, scale_tr);
}

/*
 * Sec. 2.2.2 for E4M3 codes: acc[i,j] = sum_k val(a[i,k]) val(b[j,k]) with the
 * sum formed in binary64.  Every product of two E4M3 values is exact in
 * binary64 (8 significant bits), and the partial sums of the lengths used here
 * stay exact as well (all terms are multiples of 2^-18 below 2^18 each), so
 * this is the exact product of the two quantized matrices.
 * out[i,j] = acc[i,j] * (s_row[i] * s_col[j]), the scale product one binary32
 * multiply, the rest binary64.
 */
void orc_gemm_e4m3_nt(const uint8_t *a, const uint8_t *b, int64_t M, int64_t N, int64_t Kc,
                      const float *s_row, int row_stride, const float *s_col, int col_stride,
                      double *acc, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            double s = 0.0;
            for (int64_t k = 0; k < Kc; ++k)
                s += orc_e4m3_decode(a[i * Kc + k]) * orc_e4m3_decode(b[j * Kc + k]);
            acc[i * N + j] = s;
            float sc = s_row[i * row_stride] * s_col[j * col_stride];
            out[i * N + j] = s * (double)sc;
        }
}

/* ====================================================================== */
/* Output options of a product                                              */
/* ====================================================================== */
/*
 * Quantization of a product's output for the layer that consumes it (the
 * next layer's Q(A_in), Alg. 1; or the previous layer's Q(dA_out), Alg. 2)
 * with a step size D that the caller supplies, because the absmax of the
 * output is not known before the product has finished.  1/D is one binary32
 * division; t = out * (1/D) is SATURATED to [-qmax, qmax] (a step size taken
 * from an earlier tensor does not bound this one), then rounded by the rule of
 * orc_quantize_scalar with the threshold of flat index
 * index_offset + i * N + j.  D = 0 (or a reciprocal that overflows) gives
 * codes 0.  Also returns max |out| through absmax.
 */
void orc_requantize(const float *out, int64_t M, int64_t N, float step, int bits, int round_mode,
                    uint64_t seed, uint64_t tensor_id, uint64_t index_offset,
                    int8_t *codes, float *absmax)
{
    float qmax = (float)orc_qmax(bits);
    float inv = (step == 0.0f) ? 0.0f : 1.0f / step;
    if (isinf(inv) || inv != inv) inv = 0.0f;
    float best = 0.0f;
    for (int64_t i = 0; i < M; ++i)
        for (int64_t j = 0; j < N; ++j) {
            float o = out[i * N + j];
            if (fabsf(o) > best) best = fabsf(o);
            float t = o * inv;
            if (t > qmax) t = qmax;
            if (t < -qmax) t = -qmax;
            uint64_t idx = index_offset + (uint64_t)i * (uint64_t)N + (uint64_t)j;
            uint32_t u24 = (round_mode == ORC_SR) ? orc_threshold_u24(seed, tensor_id, idx) : 0u;
            codes[i * N + j] = (int8_t)orc_quantize_scalar(t, 1.0f, bits, round_mode, u24);
        }
    if (absmax) *absmax = best;
}

/* Gradient accumulation over micro-batches: dst += src, one binary32 addition per element. */
void orc_accumulate(float *dst, const float *src, int64_t n)
{
    for (int64_t i = 0; i < n; ++i) dst[i] = dst[i] + src[i];
}

/*
 * A product stored as bfloat16 (the optional narrow output of the dequantizing step): the
 * bfloat16 number nearest to the binary32 value, ties to the one whose last kept bit is even.
 * bfloat16 is the upper half of the binary32 pattern, so the two neighbours are the pattern with
 * its low 16 bits cleared and that plus one unit of the 17th bit; the discarded half decides.
 * Finite inputs only (a value beyond the largest bfloat16 goes to infinity, as the format says).
 */
void orc_to_bf16(const float *x, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) {
        uint32_t b;
        memcpy(&b, &x[i], 4);
        uint32_t keep = b >> 16, rest = b & 0xFFFFu;
        if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep += 1u;
        out[i] = (uint16_t)keep;
    }
}
