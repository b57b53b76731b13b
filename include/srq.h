/*
 * srq — stochastically-rounded quantized linear layer for NVIDIA B200 (sm_100a).
 *
 * C ABI of libsrq.so.  The operations are those of the paper "Training with
 * Fewer Bits: Unlocking Edge LLMs Training with Stochastic Rounding":
 * the threshold quantizer Q_D(x, eps) (Def. 1) in its round-to-nearest
 * (Def. 2) and stochastic-rounding (Def. 3) forms, the mixed-precision
 * forward pass (Alg. 1) and the mixed-precision backward pass (Alg. 2).
 *
 * Conventions for every entry point
 *   - Storage: activations A[T,K], weights W[N,K], output gradients dY[T,N],
 *     all row-major; Y[T,N] = Q(A) Q(W)^T, dA[T,K] = Q(dY) Q(W),
 *     dW[N,K] = Q(dY)^T Q(A).  (The paper writes W as [in,out]; this is the
 *     same mathematics with W stored [out,in].)
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, the
 *     workspace included.  qspec pointers and the debug struct are HOST
 *     pointers, read before the call returns.  The library allocates no
 *     device memory.  Between calls it keeps only what it has learned about the
 *     devices (SM count, how many CTAs of a kernel fit, the address of the array
 *     sr_quantize_static uses; each found once, thread-safely) and the launch
 *     counter of srq_launch_count; nothing of it changes a result.
 *     (sr_quantize_static is the one exception to "no device memory": see there.)
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*, NULL
 *     for the default stream) and the call returns without waiting.
 *   - Errors the host can see (null pointer, bits outside the grid's range, a pitch or
 *     pointer that breaks the alignment rules below, workspace too small,
 *     a contraction long enough to overflow int32) return a status at once
 *     and enqueue nothing.  Conditions only the device can see (an input
 *     that is not finite, a bounded wait inside a kernel that ran out) are
 *     recorded in a status word at the start of the workspace; read it with
 *     srq_poll_status (sr_quantize_static, which has no workspace, reports
 *     through a word the caller passes).  After such a condition the outputs are
 *     unspecified.
 *   - Outputs are overwritten, unless a srq_output_t (the *_ex entry points) asks for accumulation.
 *   - Both operands of a layer pass use the same grid (srq_qspec_t.format).  With the
 *     floating-point grid (E4M3, or E4M2 / E4M1 / E4M0 by `bits`) the codes are E4M3 bytes,
 *     D_g = absmax_g / (largest value of the grid: 448, 448, 384, 256), the products run in
 *     kind::f8f6f4 with binary32 accumulation, and the `acc` member of the debug struct receives
 *     binary32 sums (same size as int32).
 *   - Alignment: input base pointers 16-byte aligned; input pitch `ld` in
 *     elements; fp32 outputs 16-byte aligned; the workspace 256-byte aligned.
 *     Inputs whose pitch or extent is not a multiple of 4 elements take a
 *     slower element-wise path with identical results.
 *
 * Step size.  The paper leaves the precision level D of Def. 1 free.  Here
 * D_g = absmax_g / qmax with qmax = 2^(bits-1) - 1 and codes in
 * [-qmax, qmax]; x / D is evaluated as x * inv_g, one binary32 multiply,
 * with inv_g = qmax / absmax_g rounded toward zero, so that the quotient of
 * every element of the group stays within [-qmax, qmax] as in Def. 1.  The group g is the whole tensor (SRQ_PER_TENSOR) or one row of
 * the code layout being written (SRQ_PER_ROW), i.e. one index of the
 * dimension that is NOT contracted in the product that consumes the codes.
 *
 * Thresholds.  eps of Def. 3 is never stored: element x[r,c] uses
 * eps = u24 * 2^-24, where u24 is the top 24 bits of word (i & 3) of
 * Philox4x32-10 with counter {lo(i>>2), hi(i>>2), lo(tensor_id),
 * hi(tensor_id)} and key {lo(seed), hi(seed)}, i = index_offset + r*cols + c.
 * SR rounds up iff eps < frac(x/D); RTN rounds up iff frac(x/D) >= 1/2.
 * The same (seed, tensor_id, index_offset, bits, scale, round) reproduces the
 * same codes, which is how one quantized W serves forward and backward.
 */
#ifndef SRQ_H
#define SRQ_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SRQ_OK = 0,
    SRQ_ERR_INVALID_ARG = 1,   /* null pointer, bad enum, bad extent, misaligned pointer/pitch */
    SRQ_ERR_UNSUPPORTED = 2,   /* bits outside 2..8 (5..8 on the floating-point grid); options that do not combine */
    SRQ_ERR_WORKSPACE = 3,     /* workspace smaller than srq_*_workspace_bytes says */
    SRQ_ERR_ACC_OVERFLOW = 4,  /* contraction length * qmax_a * qmax_b >= 2^31 */
    SRQ_ERR_CUDA = 5,          /* a CUDA call failed (launch, tensor-map encode, copy) */
    SRQ_ERR_NONFINITE = 6,     /* device: an input group has a NaN or infinite absmax */
    SRQ_ERR_TIMEOUT = 7        /* device: a bounded wait in a kernel ran out */
} srq_status_t;

typedef enum { SRQ_F32 = 0, SRQ_BF16 = 1 } srq_dtype_t;
typedef enum { SRQ_PER_TENSOR = 0, SRQ_PER_ROW = 1 } srq_scale_t;
/* SRQ_SR8: stochastic rounding with 8 random bits per element instead of 24 (the paper's hardware
 * section argues that a few pseudo-random bits per rounding suffice): eps = (b + 1/2) / 256 with b
 * byte (i & 3) of word ((i >> 2) & 3) of Philox block i >> 4, so that one block serves 16 elements.
 * P(round up) is the fraction rounded to the nearest 1/256.  Integer grid only. */
typedef enum { SRQ_SR = 0, SRQ_RTN = 1, SRQ_SR8 = 2 } srq_round_t;
/* Grid of a quantization point: integers times the step size (bits 2..8), or 8-bit floating-point
 * values times the step size.  SRQ_GRID_E4M3 with bits = 8 is E4M3 (1 sign, 4 exponent, 3 mantissa
 * bits, bias 7, no infinities, largest value 448); bits = 7, 6, 5 select E4M2, E4M1, E4M0, the
 * formats of the paper's experiments section, taken as the E4M3 values with 2, 1, 0 mantissa bits
 * (largest values 448, 384, 256; Def. 1 with the binade's own step).  Their codes are E4M3 bytes
 * with the low mantissa bits clear, so one product (kind::f8f6f4) serves all four. */
typedef enum { SRQ_GRID_INT = 0, SRQ_GRID_E4M3 = 1, SRQ_GRID_NONE = 2 /* operand left unquantized */ } srq_grid_t;

/* One quantization point: the paper's (D, eps) pair for one operand of one pass
 * (five per layer: A and W forward; A, W and dY backward). */
typedef struct {
    int32_t bits;          /* integer grid: 2..8 (codes are stored one per int8 whatever the width);
                              floating-point grid: 8, 7, 6, 5 = E4M3, E4M2, E4M1, E4M0 */
    int32_t scale;         /* srq_scale_t */
    int32_t round;         /* srq_round_t */
    int32_t format;        /* srq_grid_t; 0 = integer grid */
    uint64_t seed;         /* Philox key; one per training step */
    uint64_t tensor_id;    /* Philox counter words 2-3; one per (layer, operand, pass) */
    uint64_t index_offset; /* added to the flat index; first_row*cols for a row shard */
    const float *absmax;   /* optional, DEVICE pointer.  SRQ_PER_TENSOR: one float, max |x| of the operand
                            * when the caller already knows it (srq_absmax, or an all-reduced maximum
                            * over token shards); the absmax pass over the operand is then skipped.
                            * SRQ_PER_ROW: [cols] floats, max |x[:, c]| of every column of the source
                            * matrix (srq_absmax_cols, max-reduced over token shards), used for the
                            * step sizes of the TRANSPOSED layout, whose groups run over the rows,
                            * i.e. over tokens other shards may hold; the row-major layout's row
                            * maxima are always computed here.  Values must not be smaller than the
                            * true maxima (codes are unspecified otherwise).  NULL: compute them. */
} srq_qspec_t;

/* Optional copies of what a layer pass fed to its product: dense code matrices in the layout
 * the product consumed (contracted axis contiguous), their step sizes, and the int32 sums.
 * Any member may be NULL.  All are device pointers. */
typedef struct {
    int8_t *codes_a;   /* first operand  [M, Kc] */
    float *scale_a;    /* [1] or [M] */
    int8_t *codes_b;   /* second operand [Nn, Kc] */
    float *scale_b;    /* [1] or [Nn] */
    int32_t *acc;      /* [M, Nn] */
} srq_debug_out_t;

/* Bytes of workspace sr_quantize needs for a [rows, cols] input. */
size_t srq_quantize_workspace_bytes(int64_t rows, int64_t cols);

/* Bytes of workspace srq_gemm_i8 needs for an [M, N] output (partial sums of a split contraction). */
size_t srq_gemm_workspace_bytes(int64_t M, int64_t N);

/* Bytes of workspace that suffices for any one of the qlinear_* calls on a layer with
 * T tokens, N output and K input features. */
size_t srq_workspace_bytes(int64_t T, int64_t N, int64_t K);

/*
 * Def. 1-3 applied element-wise to x[rows, cols] (row pitch ld elements, type dt).
 * Writes int8 codes in the row-major layout codes_rm[rows, ld_rm] with scale_rm ([1] per
 * tensor, [rows] per row) and/or the transposed layout codes_tr[cols, ld_tr] with scale_tr
 * ([1] per tensor, [cols] per row of that layout, i.e. per column of x).  A NULL code
 * pointer skips that layout (its scale pointer is then ignored).  Per tensor both layouts
 * hold the same codes; per row they differ in step size but share each element's threshold.
 * ld_rm >= cols, ld_tr >= rows; padding bytes are left untouched.
 */
srq_status_t sr_quantize(const void *x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                         const srq_qspec_t *q,
                         int8_t *codes_rm, int64_t ld_rm, float *scale_rm,
                         int8_t *codes_tr, int64_t ld_tr, float *scale_tr,
                         void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * sr_quantize for callers that cannot allocate device memory.  (The paper has no counterpart
 * of this entry point; it exists for deployment reasons only.)  Same operation, arguments and
 * results as sr_quantize, but without a workspace: the scratch words come from a 1 MiB array
 * built into the library, which every device that loads the library holds until the process
 * exits.  Meant for code that runs where cudaMalloc is unavailable or unwelcome: inside a
 * framework whose memory pool is already fully assigned, in a plug-in that is handed only its
 * input and output tensors, or in a latency-critical loop that must not hit the allocator's
 * implicit synchronisation.  The call itself allocates nothing, on the host or the device.
 *   - Limit: 512 + 2 * (pad64(rows) + pad64(cols)) * 4 bytes must fit in 1 MiB, pad64 rounding
 *     up to a multiple of 64 (about rows + cols <= 131000); larger inputs return
 *     SRQ_ERR_WORKSPACE and enqueue nothing.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - device_status: optional caller-owned device word (4-byte aligned) that is cleared and
 *     then receives SRQ_ERR_NONFINITE if an input group is not finite; pass NULL to ignore.
 *   - All calls on a device share the array, and it keeps the previous call's contents; each
 *     call clears what it needs.  Calls whose kernels may overlap on the same device (streams
 *     with no ordering between them) race with each other: order them, or use sr_quantize.
 */
srq_status_t sr_quantize_static(const void *x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                                const srq_qspec_t *q,
                                int8_t *codes_rm, int64_t ld_rm, float *scale_rm,
                                int8_t *codes_tr, int64_t ld_tr, float *scale_tr,
                                uint32_t *device_status, void *cuda_stream);

/* max |x| over x[rows, cols] (row pitch ld elements) into *absmax (device, one float), e.g. to
 * share it between the forward and the backward quantization point of the same tensor, or to
 * all-reduce it over token shards, through srq_qspec_t.absmax.  Needs no workspace. */
srq_status_t srq_absmax(const void *x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                        float *absmax, void *cuda_stream);

/* max |x[:, c]| of every column into absmax_cols (device, [cols] floats, overwritten): what a token
 * shard contributes to the per-row step sizes of the transposed layout (the operands of the
 * weight-gradient product); max-reduce it over the shards and pass it through srq_qspec_t.absmax. */
srq_status_t srq_absmax_cols(const void *x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                             float *absmax_cols, void *cuda_stream);

/*
 * The product of two quantized matrices (mixed-precision matmul subsection): int8 codes
 * a[M, Kc] (pitch lda) and b[N, Kc] (pitch ldb), both with the contracted axis contiguous,
 * multiplied on the tensor cores with exact int32 accumulation, then
 *     out[i, j] = float(acc[i, j]) * (s_row[i * row_stride] * s_col[j * col_stride])
 * (each operation one binary32 rounding).  row_stride / col_stride are 0 for a per-tensor
 * step size and 1 for per-row.  acc_out, if not NULL, also receives the raw sums [M, N]
 * (pitch N).  lda and ldb must be multiples of 16 and a, b 16-byte aligned (TMA rule).
 * Requires Kc * 127 * 127 < 2^31 unless the caller passes smaller code ranges through the
 * qlinear_* entry points, which check the bound for their own bit widths.
 */
srq_status_t srq_gemm_i8(const int8_t *a, int64_t lda, const int8_t *b, int64_t ldb,
                         int64_t M, int64_t N, int64_t Kc,
                         const float *s_row, int32_t row_stride,
                         const float *s_col, int32_t col_stride,
                         float *out, int64_t ldo, int32_t *acc_out,
                         void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The same product for E4M3 codes (the 8-bit floating-point grid; the paper's experiments use
 * the E4M0 / E4M1 / E4M2 members of this family): a[M, Kc], b[N, Kc] are E4M3 bytes, multiplied
 * on the tensor cores (kind::f8f6f4) with binary32 accumulation, whose summation order is the
 * hardware's, so results agree with the exact product to about 1e-5 * |row| * |col| rather than
 * bit for bit.  out[i, j] = acc[i, j] * (s_row[i] * s_col[j]); acc_out, if not NULL, receives
 * the raw binary32 sums [M, N].  Alignment rules as for srq_gemm_i8; the contraction is never
 * split, so the workspace only needs its 256-byte header.
 */
srq_status_t srq_gemm_e4m3(const uint8_t *a, int64_t lda, const uint8_t *b, int64_t ldb,
                           int64_t M, int64_t N, int64_t Kc,
                           const float *s_row, int32_t row_stride,
                           const float *s_col, int32_t col_stride,
                           float *out, int64_t ldo, float *acc_out,
                           void *ws, size_t ws_bytes, void *cuda_stream);

/* Alg. 1: Y[T,N] = Q(A) Q(W)^T.  qA, qW are the forward quantization points of A and W.
 * Per row: A per token, W per output feature.
 * qA->format == SRQ_GRID_NONE gives the forward pass of the paper's mixed-precision SGD for the
 * quantization-aware objective, which leaves the forward activations unquantized (D_A^fwd = 0):
 * Y = A Q(W)^T with A used as the bfloat16 numbers it holds (dt must be SRQ_BF16, K a multiple
 * of 8, W on the integer grid).  The product then runs in bfloat16 with binary32 accumulation,
 * so Y agrees with the exact product to about 1e-5 * |row| * |col| rather than bit for bit; dbg
 * is ignored. */
srq_status_t qlinear_fwd(const void *A, const void *W, srq_dtype_t dt,
                         int64_t T, int64_t N, int64_t K,
                         const srq_qspec_t *qA, const srq_qspec_t *qW,
                         float *Y, const srq_debug_out_t *dbg,
                         void *ws, size_t ws_bytes, void *cuda_stream);

/* Alg. 2, input gradient: dA[T,K] = Q(dY) Q(W).  The contraction runs over N, so Q(W) is
 * written in its transposed layout [K,N].  Per row: dY per token, W per input feature. */
srq_status_t qlinear_bwd_input(const void *dY, const void *W, srq_dtype_t dt,
                               int64_t T, int64_t N, int64_t K,
                               const srq_qspec_t *qdY, const srq_qspec_t *qW,
                               float *dA, const srq_debug_out_t *dbg,
                               void *ws, size_t ws_bytes, void *cuda_stream);

/* Alg. 2, weight gradient: dW[N,K] = Q(dY)^T Q(A).  The contraction runs over the T tokens;
 * both operands are written in their transposed layouts [N,T] and [K,T].  Per row: dY per
 * output feature, A per input feature. */
srq_status_t qlinear_bwd_weight(const void *dY, const void *A, srq_dtype_t dt,
                                int64_t T, int64_t N, int64_t K,
                                const srq_qspec_t *qdY, const srq_qspec_t *qA,
                                float *dW, const srq_debug_out_t *dbg,
                                void *ws, size_t ws_bytes, void *cuda_stream);

/* Alg. 2 as a whole: dA[T,K] = Q(dY) Q(W) and dW[N,K] = Q(dY)^T Q(A) in one call.  Alg. 2
 * quantizes dY once and uses it in both products; here dY is read once and its codes are written
 * in both layouts ([T,N] for dA, [N,T] for dW) by the same pass, which saves one absmax and one
 * quantization pass over dY compared with qlinear_bwd_input followed by qlinear_bwd_weight.  The
 * results are bit for bit those of the two separate calls with the same quantization points.
 * dbg_input / dbg_weight receive the operands and sums of the dA and dW products. */
srq_status_t qlinear_bwd(const void *dY, const void *A, const void *W, srq_dtype_t dt,
                         int64_t T, int64_t N, int64_t K,
                         const srq_qspec_t *qdY, const srq_qspec_t *qA, const srq_qspec_t *qW,
                         float *dA, float *dW,
                         const srq_debug_out_t *dbg_input, const srq_debug_out_t *dbg_weight,
                         void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * What else a product does with its results; every member is optional (zero / NULL).
 *   accumulate  1: out += result (one binary32 addition per element) instead of out = result.
 *               The paper emulates large batches by accumulating gradients over micro-batches
 *               (hardware-considerations section); this is that accumulation for dW.
 *               2: the int32 sums are accumulated instead: acc_out += sums (the call's acc_out /
 *               dbg->acc matrix is required and holds the running sums; zero it before the first
 *               micro-batch) and out = float(acc_out) * (s_row * s_col) is written from the total.
 *               Exact - the result equals one product over the concatenated contraction - as
 *               long as every micro-batch uses the same step sizes (srq_qspec_t.absmax) and the
 *               totals fit int32; a wrap is reported as SRQ_ERR_ACC_OVERFLOW by srq_poll_status.
 *               Integer grid only.
 *   q, step, codes, ld_codes
 *               also write Q(result) as int8 codes [M, ld_codes] for the layer that consumes the
 *               result (the next layer's Q(A_in) of Alg. 1, the previous layer's Q(dA_out) of
 *               Alg. 2), fused into the product's epilogue so that the result is not read again.
 *               The absmax of a result is not known until the product has finished, so the step
 *               size comes from the caller: *step (device, [1]); x / D is out * (1 / D) with one
 *               binary32 division, SATURATED to [-qmax, qmax], then rounded by q->round with the
 *               thresholds of (q->seed, q->tensor_id, q->index_offset + i * N + j).  q must be on
 *               the integer grid; q->scale is ignored (one step for the whole result).  With
 *               codes given, the fp32 output pointer of the call may be NULL.
 *   absmax      device [1], holding a non-negative number (usually 0) on entry: raised to
 *               max |result|, from which the caller derives the step size of its next step.
 *   out_bf16    1: the output pointer of the call addresses bfloat16 numbers (pass it cast to
 *               float *; its pitch counts bfloat16 elements): each binary32 result is rounded to
 *               the nearest bfloat16, ties to even, as it is stored, which halves the bytes the
 *               product writes.  Codes and absmax still come from the binary32 result.  Not with
 *               accumulate = 1 (SRQ_ERR_UNSUPPORTED): running binary32 sums stay in binary32.
 *   raw_sums    1: the output pointer of the call addresses int32 numbers (pass it cast to float *;
 *               its pitch counts int32 elements) and receives the exact sums themselves; nothing
 *               is scaled.  For token shards on several devices (the batch axis of the variance
 *               lemma): the shards' sums are added with an integer all-reduce, which is exact in
 *               any order, and srq_dequant_i32 then scales the total once, so that the weight
 *               gradient is bit for bit the one a single device computes on the whole batch
 *               (given shared step sizes, srq_qspec_t.absmax).  Integer grid only; not combined
 *               with any other member (SRQ_ERR_UNSUPPORTED).
 * Products with q or absmax set are never split along the contraction.
 */
typedef struct {
    int32_t accumulate;
    int32_t out_bf16;
    const srq_qspec_t *q;
    const float *step;
    int8_t *codes;
    int64_t ld_codes;
    float *absmax;
    int32_t raw_sums;
} srq_output_t;

/* srq_gemm_i8, qlinear_fwd and qlinear_bwd with output options (NULL = none, i.e. the plain call).
 * In qlinear_bwd_ex, output_dA applies to dA[T,K] and output_dW to dW[N,K]. */
srq_status_t srq_gemm_i8_ex(const int8_t *a, int64_t lda, const int8_t *b, int64_t ldb,
                            int64_t M, int64_t N, int64_t Kc,
                            const float *s_row, int32_t row_stride,
                            const float *s_col, int32_t col_stride,
                            float *out, int64_t ldo, int32_t *acc_out, const srq_output_t *output,
                            void *ws, size_t ws_bytes, void *cuda_stream);
srq_status_t qlinear_fwd_ex(const void *A, const void *W, srq_dtype_t dt,
                            int64_t T, int64_t N, int64_t K,
                            const srq_qspec_t *qA, const srq_qspec_t *qW, float *Y,
                            const srq_output_t *output, const srq_debug_out_t *dbg,
                            void *ws, size_t ws_bytes, void *cuda_stream);
srq_status_t qlinear_bwd_ex(const void *dY, const void *A, const void *W, srq_dtype_t dt,
                            int64_t T, int64_t N, int64_t K,
                            const srq_qspec_t *qdY, const srq_qspec_t *qA, const srq_qspec_t *qW,
                            float *dA, float *dW,
                            const srq_output_t *output_dA, const srq_output_t *output_dW,
                            const srq_debug_out_t *dbg_input, const srq_debug_out_t *dbg_weight,
                            void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The finishing step of a product on its own (the last line of Alg. 1 / Alg. 2 once the integer
 * sums exist): out[i, j] = float(acc[i, j]) * (s_row[i * row_stride] * s_col[j * col_stride]) over a
 * caller's int32 matrix acc[M, N] (pitch ld_acc), with the same three roundings in the same order as
 * the products' own epilogue, so that sums collected with raw_sums and scaled here give the very
 * bits the one-call product gives.  out is binary32 [M, ldo], or bfloat16 when out_bf16 = 1 (round
 * to nearest even).  All pointers are device pointers, 4-byte aligned (16-byte alignment and
 * pitches that are multiples of 4 allow vector accesses).  Needs no workspace.
 */
srq_status_t srq_dequant_i32(const int32_t *acc, int64_t ld_acc, int64_t M, int64_t N,
                             const float *s_row, int32_t row_stride,
                             const float *s_col, int32_t col_stride,
                             void *out, int64_t ldo, int32_t out_bf16, void *cuda_stream);

/* Waits for the stream, then returns the device status word of the workspace: SRQ_OK, or the
 * first device-side condition recorded by the calls that used this workspace since its header
 * was last cleared (every entry point clears it when it starts). */
srq_status_t srq_poll_status(void *ws, void *cuda_stream);

/* Host-side planning rule of the product kernel, exposed so that it can be checked without a device:
 * with `tiles` output tiles, `k_blocks` 128-byte blocks along the contraction and `groups` tiles
 * running at a time, tiles [0, *full_tiles) are computed whole and each remaining tile in *splits
 * parts (*splits == 1: nothing is split).  Invalid arguments give 0, 0. */
void srq_plan_splits(int64_t tiles, int32_t k_blocks, int32_t groups, int32_t *full_tiles, int32_t *splits);

/* Self-test of the failure path of the product kernel: enqueues a one-thread kernel that waits, for
 * at most limit_us microseconds (1 .. 1000000), on a barrier that nothing signals.  The wait gives
 * up in the same way the bounded waits of the product kernel do: the status word of ws receives
 * SRQ_ERR_TIMEOUT (read it with srq_poll_status), the kernel returns and the context stays usable. */
srq_status_t srq_selftest_bounded_wait(void *ws, size_t ws_bytes, uint32_t limit_us, void *cuda_stream);

/* Measurement aid, not part of the layer: device-side timing of the product kernel inside whatever
 * sequence of calls the caller runs (a whole layer step), which stream events around a call cannot
 * give because a call enqueues several kernels.  slots is a caller-owned DEVICE array of 2 * n
 * 64-bit words that the caller has initialised to (all ones, zero) pairs: the i-th product launch
 * after this call lowers slots[2 i] to the nanosecond time (%globaltimer) at which its first CTA
 * starts work, after the kernel before it has finished, and raises slots[2 i + 1] to the time its
 * last CTA ends; launches beyond n are not timed.  Two atomics per CTA, nothing else changes.
 * srq_set_product_timer(NULL, 0) switches it off.  The setting is process-wide (all streams and
 * devices): time one stream at a time. */
srq_status_t srq_set_product_timer(uint64_t *slots, int64_t n);

/* Measurement aid, not part of the layer: the issue rate of the tensor pipe for the instruction the
 * products use (tcgen05.mma.cta_group::2.kind::i8, M256 N256 K32).  Every CTA pair of the device
 * multiplies operand blocks that already sit in its shared memory, k_blocks (1 .. 2^22) blocks of 128
 * bytes of contraction, into TMEM; nothing moves through global memory.  *ops (host, optional)
 * receives the integer operations of the launch (2 * 256 * 256 * 128 per pair and block); time the
 * launch on the stream and divide.  This is the ceiling the main loop of the products is compared
 * with: the kind::i8 pipe at the clock the power limit allows, with no data movement at all.  The
 * status word of ws reports a wait that ran out (SRQ_ERR_TIMEOUT), as in the product kernel. */
srq_status_t srq_selftest_mma_rate(void *ws, size_t ws_bytes, int32_t k_blocks, int64_t *ops, void *cuda_stream);

/* Static, human-readable name of a status. */
const char *srq_status_string(srq_status_t s);

/* Number of kernels the library has launched in this process (for launch accounting). */
uint64_t srq_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SRQ_H */
