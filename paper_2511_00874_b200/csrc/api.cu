// C-ABI entry points of libsrq: argument checks, workspace carving and launch sequencing.
// All arithmetic is in quantize.cu and gemm_i8.cu.
#include "common.cuh"

using namespace srq;

// Host-side validation of one quantization point, shared by every entry point that takes one.
srq_status_t srq::check_qspec(const srq_qspec_t* q) {
    if (!q) return SRQ_ERR_INVALID_ARG;
    if (q->format != SRQ_GRID_INT && q->format != SRQ_GRID_E4M3) return SRQ_ERR_INVALID_ARG;
    if (q->format == SRQ_GRID_INT && (q->bits < 2 || q->bits > 8)) return SRQ_ERR_UNSUPPORTED;
    if (q->format == SRQ_GRID_E4M3 && (q->bits < 5 || q->bits > 8)) return SRQ_ERR_UNSUPPORTED;   // E4M0 .. E4M3
    if (q->scale != SRQ_PER_TENSOR && q->scale != SRQ_PER_ROW) return SRQ_ERR_INVALID_ARG;
    if (q->round != SRQ_SR && q->round != SRQ_RTN && q->round != SRQ_SR8) return SRQ_ERR_INVALID_ARG;
    if (q->round == SRQ_SR8 && q->format != SRQ_GRID_INT) return SRQ_ERR_UNSUPPORTED;
    if (q->absmax && ((uintptr_t)q->absmax % 4) != 0) return SRQ_ERR_INVALID_ARG;
    return SRQ_OK;
}

namespace {

inline int qmax_of(int bits) { return (1 << (bits - 1)) - 1; }

// Host-side checks of the output options of a product with an [M, N] result, and their device form.
srq_status_t make_out_options(const srq_output_t* o, int64_t N, bool have_out, OutOptions* r) {
    *r = OutOptions();
    if (!o) return have_out ? SRQ_OK : SRQ_ERR_INVALID_ARG;
    if (o->accumulate < 0 || o->accumulate > 2) return SRQ_ERR_INVALID_ARG;
    if (o->accumulate && !have_out) return SRQ_ERR_INVALID_ARG;
    if (o->out_bf16 != 0 && o->out_bf16 != 1) return SRQ_ERR_INVALID_ARG;
    if (o->out_bf16 && o->accumulate == 1) return SRQ_ERR_UNSUPPORTED;   // running binary32 sums stay in binary32
    if (o->raw_sums != 0 && o->raw_sums != 1) return SRQ_ERR_INVALID_ARG;
    if (o->raw_sums && (!have_out || o->accumulate || o->out_bf16 || o->q || o->absmax)) return SRQ_ERR_UNSUPPORTED;
    r->accumulate = o->accumulate;
    r->out_bf16 = o->out_bf16;
    r->raw_sums = o->raw_sums;
    if (o->q) {
        srq_status_t s = check_qspec(o->q);
        if (s != SRQ_OK) return s;
        if (o->q->format != SRQ_GRID_INT || o->q->round == SRQ_SR8) return SRQ_ERR_UNSUPPORTED;
        if (!o->step || !o->codes || o->ld_codes < N || ((uintptr_t)o->step % 4) != 0) return SRQ_ERR_INVALID_ARG;
        r->requant = 1;
        r->rq_sr = o->q->round == SRQ_SR;
        r->rq_lim = (float)(((1 << (o->q->bits - 1)) - 1)) * 16777216.0f;
        r->rq_step = o->step; r->rq_codes = o->codes; r->rq_ld = o->ld_codes;
        r->rq_offset = o->q->index_offset;
        r->rq_keys = make_philox_keys(o->q->seed, o->q->tensor_id);
    } else if (!have_out) {
        return SRQ_ERR_INVALID_ARG;                       // nothing would be produced
    }
    if (o->absmax) {
        if (((uintptr_t)o->absmax % 4) != 0) return SRQ_ERR_INVALID_ARG;
        r->absmax_bits = (uint32_t*)o->absmax;
    }
    return SRQ_OK;
}

inline bool aligned_to(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }
inline int64_t pitch16(int64_t n) { return (n + 15) / 16 * 16; }
inline size_t f32_block(int64_t n) { return align_up((size_t)n * 4); }

cudaError_t clear_header(void* ws, cudaStream_t st) { return cudaMemsetAsync(ws, 0, sizeof(WsHeader), st); }

// One operand of a layer pass: source matrix, which code layout the product needs, its spec.
struct Operand {
    const void* x; int64_t rows, cols;   // source extents (pitch = cols)
    bool transposed;                     // false: codes [rows, cols]; true: codes [cols, rows]
    const srq_qspec_t* q;
    int64_t out_rows() const { return transposed ? cols : rows; }
    int64_t out_cols() const { return transposed ? rows : cols; }   // contraction length
};

// Carving of a qlinear workspace.
struct LayerPlan {
    size_t off_scratch[2], off_scale[2], off_codes[2], off_split, total;
    int64_t pitch;
};

LayerPlan plan_layer(const Operand& a, const Operand& b) {
    LayerPlan p;
    size_t o = sizeof(WsHeader);
    const Operand* ops[2] = {&a, &b};
    for (int i = 0; i < 2; ++i) { p.off_scratch[i] = o; o += quant_scratch_bytes(ops[i]->rows, ops[i]->cols); }
    for (int i = 0; i < 2; ++i) { p.off_scale[i] = o; o += f32_block(ops[i]->out_rows()); }
    p.pitch = pitch16(a.out_cols());
    for (int i = 0; i < 2; ++i) { p.off_codes[i] = o; o += align_up((size_t)ops[i]->out_rows() * p.pitch); }
    p.off_split = o;
    o += gemm_splitk_bytes(a.out_rows(), b.out_rows());
    p.total = o;
    return p;
}

srq_status_t run_layer(const Operand& a, const Operand& b, srq_dtype_t dt, float* out, const srq_output_t* oopt,
                       const srq_debug_out_t* dbg, void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!a.x || !b.x || !ws) return SRQ_ERR_INVALID_ARG;
    OutOptions opt;
    {
        const srq_status_t so = make_out_options(oopt, b.out_rows(), out != nullptr, &opt);
        if (so != SRQ_OK) return so;
    }
    if (dt != SRQ_F32 && dt != SRQ_BF16) return SRQ_ERR_INVALID_ARG;
    if (a.rows < 0 || a.cols < 0 || b.rows < 0 || b.cols < 0) return SRQ_ERR_INVALID_ARG;
    srq_status_t s;
    if ((s = check_qspec(a.q)) != SRQ_OK) return s;
    if ((s = check_qspec(b.q)) != SRQ_OK) return s;
    if (!aligned_to(a.x, 16) || !aligned_to(b.x, 16) || !aligned_to(out, 16) || !aligned_to(ws, 256)) return SRQ_ERR_INVALID_ARG;
    if ((opt.requant || opt.raw_sums) && a.q->format != SRQ_GRID_INT) return SRQ_ERR_UNSUPPORTED;
    const int64_t M = a.out_rows(), Nn = b.out_rows(), Kc = a.out_cols();
    if (Kc != b.out_cols()) return SRQ_ERR_INVALID_ARG;
    if (a.q->format != b.q->format) return SRQ_ERR_INVALID_ARG;          // one product, one kind of code
    if (a.q->format == SRQ_GRID_INT && (double)Kc * qmax_of(a.q->bits) * qmax_of(b.q->bits) >= 2147483648.0) return SRQ_ERR_ACC_OVERFLOW;
    const LayerPlan p = plan_layer(a, b);
    if (ws_bytes < p.total) return SRQ_ERR_WORKSPACE;
    if (M == 0 || Nn == 0) return SRQ_OK;

    char* base = (char*)ws;
    uint32_t* status = &((WsHeader*)ws)->status;
    // one clear for the status word and the scratch of both operands
    if (cudaMemsetAsync(ws, 0, p.off_scale[0], st) != cudaSuccess) return SRQ_ERR_CUDA;

    const Operand* ops[2] = {&a, &b};
    int8_t* codes[2];
    float* scales[2];
    QuantArgs qargs[2];
    QuantScratch qscr[2];
    for (int i = 0; i < 2; ++i) {
        const Operand& o = *ops[i];
        codes[i] = (int8_t*)(base + p.off_codes[i]);
        scales[i] = (float*)(base + p.off_scale[i]);
        QuantArgs& qa = qargs[i];
        qa.x = o.x; qa.dt = dt; qa.rows = o.rows; qa.cols = o.cols; qa.ld = o.cols; qa.q = *o.q;
        qa.codes_rm = o.transposed ? nullptr : codes[i]; qa.ld_rm = p.pitch; qa.scale_rm = o.transposed ? nullptr : scales[i];
        qa.codes_tr = o.transposed ? codes[i] : nullptr; qa.ld_tr = p.pitch; qa.scale_tr = o.transposed ? scales[i] : nullptr;
        qscr[i] = carve_quant_scratch(base + p.off_scratch[i], o.rows, o.cols);
    }
    // both operands: one pair of launches when the problem is small, else operand by operand
    if (Kc > 0 && launch_quantize_batch(qargs, qscr, 2, status, st, true) != cudaSuccess) return SRQ_ERR_CUDA;
    if (Kc == 0) {   // empty contraction: the product is zero
        if (!out || opt.accumulate) return SRQ_OK;
        const size_t eb = opt.out_bf16 ? 2 : 4;
        return cudaMemset2DAsync(out, (size_t)Nn * eb, 0, (size_t)Nn * eb, (size_t)M, st) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
    }

    GemmArgs g;
    g.a = codes[0]; g.lda = p.pitch; g.b = codes[1]; g.ldb = p.pitch;
    g.M = M; g.N = Nn; g.Kc = Kc; g.kind = a.q->format == SRQ_GRID_E4M3;
    g.s_row = scales[0]; g.row_stride = a.q->scale == SRQ_PER_ROW;
    g.s_col = scales[1]; g.col_stride = b.q->scale == SRQ_PER_ROW;
    g.out = out; g.ldo = Nn; g.acc_out = dbg ? dbg->acc : nullptr; g.opt = opt;
    g.splitk_ws = base + p.off_split; g.splitk_ws_bytes = p.total - p.off_split;
    if ((s = launch_gemm_i8(g, status, st)) != SRQ_OK) return s;

    if (dbg) {
        const int64_t rows[2] = {M, Nn};
        int8_t* dcodes[2] = {dbg->codes_a, dbg->codes_b};
        float* dscale[2] = {dbg->scale_a, dbg->scale_b};
        for (int i = 0; i < 2; ++i) {
            if (dcodes[i] && cudaMemcpy2DAsync(dcodes[i], (size_t)Kc, codes[i], (size_t)p.pitch, (size_t)Kc, (size_t)rows[i],
                                               cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return SRQ_ERR_CUDA;
            const size_t n = ops[i]->q->scale == SRQ_PER_ROW ? (size_t)rows[i] : 1;
            if (dscale[i] && cudaMemcpyAsync(dscale[i], scales[i], n * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
                return SRQ_ERR_CUDA;
        }
    }
    return SRQ_OK;
}

// Forward pass with unquantized activations (the paper's SR-MP-SGD for the QAT objective keeps
// D_A^fwd = 0): Y = A Q(W)^T with A taken as the bfloat16 numbers it holds.  Q(W) is quantized as
// usual, its integer codes are widened to bfloat16 (exact) and the product runs in kind::f16 with
// binary32 accumulation; Y[t, n] = acc[t, n] * D_W[n].
struct FpActPlan { size_t off_scratch, off_scale, off_one, off_codes8, off_codes16, total; int64_t pitch8, pitch16; };

FpActPlan plan_fp_act(int64_t N, int64_t K) {
    FpActPlan p;
    size_t o = sizeof(WsHeader);
    p.off_scratch = o; o += quant_scratch_bytes(N, K);
    p.off_scale = o; o += f32_block(N);
    p.off_one = o; o += f32_block(1);
    p.pitch8 = pitch16(K); p.pitch16 = pitch16(2 * K) / 2;       // elements; rows start on 16-byte boundaries
    p.off_codes8 = o; o += align_up((size_t)N * p.pitch8);
    p.off_codes16 = o; o += align_up((size_t)N * p.pitch16 * 2);
    p.total = o;
    return p;
}

srq_status_t run_fwd_fp_act(const void* A, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                            const srq_qspec_t* qW, float* Y, void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!A || !W || !Y || !ws || T < 0 || N < 0 || K < 0) return SRQ_ERR_INVALID_ARG;
    if (dt != SRQ_BF16) return SRQ_ERR_UNSUPPORTED;                  // the activations feed the tensor cores as they are
    srq_status_t s = check_qspec(qW);
    if (s != SRQ_OK) return s;
    if (qW->format != SRQ_GRID_INT) return SRQ_ERR_UNSUPPORTED;
    if (K % 8 != 0) return SRQ_ERR_INVALID_ARG;                      // rows of A must start on 16-byte boundaries (TMA)
    if (!aligned_to(A, 16) || !aligned_to(W, 16) || !aligned_to(Y, 16) || !aligned_to(ws, 256)) return SRQ_ERR_INVALID_ARG;
    const FpActPlan p = plan_fp_act(N, K);
    if (ws_bytes < p.total) return SRQ_ERR_WORKSPACE;
    if (T == 0 || N == 0) return SRQ_OK;
    if (K == 0) return cudaMemset2DAsync(Y, (size_t)N * 4, 0, (size_t)N * 4, (size_t)T, st) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
    char* base = (char*)ws;
    uint32_t* status = &((WsHeader*)ws)->status;
    if (cudaMemsetAsync(ws, 0, p.off_scale, st) != cudaSuccess) return SRQ_ERR_CUDA;      // status word and scratch
    int8_t* c8 = (int8_t*)(base + p.off_codes8);
    float* scale = (float*)(base + p.off_scale);
    float* one = (float*)(base + p.off_one);
    QuantArgs q; q.x = W; q.dt = dt; q.rows = N; q.cols = K; q.ld = K; q.q = *qW;
    q.codes_rm = c8; q.ld_rm = p.pitch8; q.scale_rm = scale; q.codes_tr = nullptr; q.ld_tr = 0; q.scale_tr = nullptr;
    if (launch_quantize(q, carve_quant_scratch(base + p.off_scratch, N, K), status, st, true) != cudaSuccess) return SRQ_ERR_CUDA;
    if (launch_widen_codes(c8, N, K, p.pitch8, base + p.off_codes16, p.pitch16, one, st) != cudaSuccess) return SRQ_ERR_CUDA;
    GemmArgs g;
    g.a = (const int8_t*)A; g.lda = 2 * K; g.b = (const int8_t*)(base + p.off_codes16); g.ldb = 2 * p.pitch16;
    g.M = T; g.N = N; g.Kc = 2 * K; g.kind = 2;
    g.s_row = one; g.row_stride = 0; g.s_col = scale; g.col_stride = qW->scale == SRQ_PER_ROW;
    g.out = Y; g.ldo = N; g.acc_out = nullptr; g.splitk_ws = nullptr; g.splitk_ws_bytes = 0;
    return launch_gemm_i8(g, status, st);
}

// Alg. 2 as one call: dY is read once and written in both code layouts, then both products run.
struct BwdPlan {
    size_t off_scratch[3], off_scale[4], off_codes[4], off_split[2], total;
    int64_t pitch_n, pitch_t;
};

BwdPlan plan_bwd(int64_t T, int64_t N, int64_t K) {
    BwdPlan p;
    size_t o = sizeof(WsHeader);
    const int64_t src[3][2] = {{T, N}, {N, K}, {T, K}};                 // dY, W, A
    for (int i = 0; i < 3; ++i) { p.off_scratch[i] = o; o += quant_scratch_bytes(src[i][0], src[i][1]); }
    const int64_t nscale[4] = {T, N, K, K};                             // dY [T,N], dY^T [N,T], W^T [K,N], A^T [K,T]
    for (int i = 0; i < 4; ++i) { p.off_scale[i] = o; o += f32_block(nscale[i]); }
    p.pitch_n = pitch16(N); p.pitch_t = pitch16(T);
    const int64_t rows[4] = {T, N, K, K};
    const int64_t pitch[4] = {p.pitch_n, p.pitch_t, p.pitch_n, p.pitch_t};
    for (int i = 0; i < 4; ++i) { p.off_codes[i] = o; o += align_up((size_t)rows[i] * pitch[i]); }
    p.off_split[0] = o; o += gemm_splitk_bytes(T, K);
    p.off_split[1] = o; o += gemm_splitk_bytes(N, K);
    p.total = o;
    return p;
}

srq_status_t copy_debug(const srq_debug_out_t* dbg, const int8_t* ca, const float* sa, int64_t rows_a, bool per_row_a,
                        const int8_t* cb, const float* sb, int64_t rows_b, bool per_row_b, int64_t Kc, int64_t pitch,
                        cudaStream_t st) {
    if (!dbg) return SRQ_OK;
    if (dbg->codes_a && cudaMemcpy2DAsync(dbg->codes_a, (size_t)Kc, ca, (size_t)pitch, (size_t)Kc, (size_t)rows_a, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SRQ_ERR_CUDA;
    if (dbg->codes_b && cudaMemcpy2DAsync(dbg->codes_b, (size_t)Kc, cb, (size_t)pitch, (size_t)Kc, (size_t)rows_b, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SRQ_ERR_CUDA;
    if (dbg->scale_a && cudaMemcpyAsync(dbg->scale_a, sa, (per_row_a ? (size_t)rows_a : 1) * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SRQ_ERR_CUDA;
    if (dbg->scale_b && cudaMemcpyAsync(dbg->scale_b, sb, (per_row_b ? (size_t)rows_b : 1) * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return SRQ_ERR_CUDA;
    return SRQ_OK;
}

srq_status_t run_bwd(const void* dY, const void* A, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                     const srq_qspec_t* qdY, const srq_qspec_t* qA, const srq_qspec_t* qW, float* dA, float* dW,
                     const srq_output_t* o_in, const srq_output_t* o_w,
                     const srq_debug_out_t* dbg_in, const srq_debug_out_t* dbg_w, void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!dY || !A || !W || !ws) return SRQ_ERR_INVALID_ARG;
    OutOptions opt_in, opt_w;
    {
        srq_status_t so = make_out_options(o_in, K, dA != nullptr, &opt_in);
        if (so == SRQ_OK) so = make_out_options(o_w, K, dW != nullptr, &opt_w);
        if (so != SRQ_OK) return so;
    }
    if (dt != SRQ_F32 && dt != SRQ_BF16) return SRQ_ERR_INVALID_ARG;
    if (T < 0 || N < 0 || K < 0) return SRQ_ERR_INVALID_ARG;
    srq_status_t s;
    if ((s = check_qspec(qdY)) != SRQ_OK) return s;
    if ((s = check_qspec(qA)) != SRQ_OK) return s;
    if ((s = check_qspec(qW)) != SRQ_OK) return s;
    if (!aligned_to(dY, 16) || !aligned_to(A, 16) || !aligned_to(W, 16) || !aligned_to(dA, 16) || !aligned_to(dW, 16) || !aligned_to(ws, 256))
        return SRQ_ERR_INVALID_ARG;
    if (qdY->format != qW->format || qdY->format != qA->format) return SRQ_ERR_INVALID_ARG;
    const int kind = qdY->format == SRQ_GRID_E4M3;
    if (kind && (opt_in.raw_sums || opt_w.raw_sums)) return SRQ_ERR_UNSUPPORTED;       // int32 sums exist on the integer grid only
    if (!kind && (double)N * qmax_of(qdY->bits) * qmax_of(qW->bits) >= 2147483648.0) return SRQ_ERR_ACC_OVERFLOW;
    if (!kind && (double)T * qmax_of(qdY->bits) * qmax_of(qA->bits) >= 2147483648.0) return SRQ_ERR_ACC_OVERFLOW;
    const BwdPlan p = plan_bwd(T, N, K);
    if (ws_bytes < p.total) return SRQ_ERR_WORKSPACE;

    char* base = (char*)ws;
    uint32_t* status = &((WsHeader*)ws)->status;
    if (cudaMemsetAsync(ws, 0, p.off_scale[0], st) != cudaSuccess) return SRQ_ERR_CUDA;   // status word and all scratch
    float* sc[4]; int8_t* cd[4];
    for (int i = 0; i < 4; ++i) { sc[i] = (float*)(base + p.off_scale[i]); cd[i] = (int8_t*)(base + p.off_codes[i]); }

    QuantArgs qargs[3];
    QuantScratch qscr[3];
    int nq = 0;
    if (T > 0 && N > 0) {      // dY -> [T,N] codes for dA and [N,T] codes for dW, one read of dY
        QuantArgs& q = qargs[nq]; q.x = dY; q.dt = dt; q.rows = T; q.cols = N; q.ld = N; q.q = *qdY;
        q.codes_rm = cd[0]; q.ld_rm = p.pitch_n; q.scale_rm = sc[0];
        q.codes_tr = cd[1]; q.ld_tr = p.pitch_t; q.scale_tr = sc[1];
        qscr[nq++] = carve_quant_scratch(base + p.off_scratch[0], T, N);
    }
    if (N > 0 && K > 0) {      // W -> [K,N]
        QuantArgs& q = qargs[nq]; q.x = W; q.dt = dt; q.rows = N; q.cols = K; q.ld = K; q.q = *qW;
        q.codes_rm = nullptr; q.ld_rm = 0; q.scale_rm = nullptr;
        q.codes_tr = cd[2]; q.ld_tr = p.pitch_n; q.scale_tr = sc[2];
        qscr[nq++] = carve_quant_scratch(base + p.off_scratch[1], N, K);
    }
    if (T > 0 && K > 0) {      // A -> [K,T]
        QuantArgs& q = qargs[nq]; q.x = A; q.dt = dt; q.rows = T; q.cols = K; q.ld = K; q.q = *qA;
        q.codes_rm = nullptr; q.ld_rm = 0; q.scale_rm = nullptr;
        q.codes_tr = cd[3]; q.ld_tr = p.pitch_t; q.scale_tr = sc[3];
        qscr[nq++] = carve_quant_scratch(base + p.off_scratch[2], T, K);
    }
    // all operands: one pair of launches when the problem is small, else operand by operand
    if (nq > 0 && launch_quantize_batch(qargs, qscr, nq, status, st, true) != cudaSuccess) return SRQ_ERR_CUDA;

    // dA[T,K] = Q(dY)[T,N] . Q(W)^T[K,N]
    if (T > 0 && K > 0) {
        if (N == 0) {
            if (dA && !opt_in.accumulate && cudaMemset2DAsync(dA, (size_t)K * (opt_in.out_bf16 ? 2 : 4), 0, (size_t)K * (opt_in.out_bf16 ? 2 : 4), (size_t)T, st) != cudaSuccess) return SRQ_ERR_CUDA;
        } else {
            GemmArgs g;
            g.a = cd[0]; g.lda = p.pitch_n; g.b = cd[2]; g.ldb = p.pitch_n; g.M = T; g.N = K; g.Kc = N; g.kind = kind;
            g.s_row = sc[0]; g.row_stride = qdY->scale == SRQ_PER_ROW; g.s_col = sc[2]; g.col_stride = qW->scale == SRQ_PER_ROW;
            g.out = dA; g.ldo = K; g.acc_out = dbg_in ? dbg_in->acc : nullptr; g.opt = opt_in;
            g.splitk_ws = base + p.off_split[0]; g.splitk_ws_bytes = p.off_split[1] - p.off_split[0];
            if ((s = launch_gemm_i8(g, status, st)) != SRQ_OK) return s;
            if ((s = copy_debug(dbg_in, cd[0], sc[0], T, g.row_stride, cd[2], sc[2], K, g.col_stride, N, p.pitch_n, st)) != SRQ_OK) return s;
        }
    }
    // dW[N,K] = Q(dY)^T[N,T] . Q(A)^T[K,T]
    if (N > 0 && K > 0) {
        if (T == 0) {
            if (dW && !opt_w.accumulate && cudaMemset2DAsync(dW, (size_t)K * (opt_w.out_bf16 ? 2 : 4), 0, (size_t)K * (opt_w.out_bf16 ? 2 : 4), (size_t)N, st) != cudaSuccess) return SRQ_ERR_CUDA;
        } else {
            GemmArgs g;
            g.a = cd[1]; g.lda = p.pitch_t; g.b = cd[3]; g.ldb = p.pitch_t; g.M = N; g.N = K; g.Kc = T; g.kind = kind;
            g.s_row = sc[1]; g.row_stride = qdY->scale == SRQ_PER_ROW; g.s_col = sc[3]; g.col_stride = qA->scale == SRQ_PER_ROW;
            g.out = dW; g.ldo = K; g.acc_out = dbg_w ? dbg_w->acc : nullptr; g.opt = opt_w;
            g.splitk_ws = base + p.off_split[1]; g.splitk_ws_bytes = p.total - p.off_split[1];
            if ((s = launch_gemm_i8(g, status, st)) != SRQ_OK) return s;
            if ((s = copy_debug(dbg_w, cd[1], sc[1], N, g.row_stride, cd[3], sc[3], K, g.col_stride, T, p.pitch_t, st)) != SRQ_OK) return s;
        }
    }
    return SRQ_OK;
}

}  // namespace

extern "C" {

size_t srq_quantize_workspace_bytes(int64_t rows, int64_t cols) {
    if (rows < 0 || cols < 0) return 0;
    return sizeof(WsHeader) + quant_scratch_bytes(rows, cols);
}

size_t srq_gemm_workspace_bytes(int64_t M, int64_t N) {
    if (M < 0 || N < 0) return 0;
    return sizeof(WsHeader) + gemm_splitk_bytes(M, N);
}

size_t srq_workspace_bytes(int64_t T, int64_t N, int64_t K) {
    if (T < 0 || N < 0 || K < 0) return 0;
    srq_qspec_t q{};
    const Operand fa{(void*)1, T, K, false, &q}, fw{(void*)1, N, K, false, &q};
    const Operand iy{(void*)1, T, N, false, &q}, iw{(void*)1, N, K, true, &q};
    const Operand wy{(void*)1, T, N, true, &q}, wa{(void*)1, T, K, true, &q};
    size_t m = plan_layer(fa, fw).total;
    const size_t m1 = plan_layer(iy, iw).total, m2 = plan_layer(wy, wa).total;
    if (m1 > m) m = m1;
    if (m2 > m) m = m2;
    const size_t m3 = plan_bwd(T, N, K).total, m4 = plan_fp_act(N, K).total;
    if (m3 > m) m = m3;
    if (m4 > m) m = m4;
    return m;
}

srq_status_t sr_quantize(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, const srq_qspec_t* q,
                         int8_t* codes_rm, int64_t ld_rm, float* scale_rm, int8_t* codes_tr, int64_t ld_tr, float* scale_tr,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!x || !ws || rows < 0 || cols < 0 || ld < cols) return SRQ_ERR_INVALID_ARG;
    if (dt != SRQ_F32 && dt != SRQ_BF16) return SRQ_ERR_INVALID_ARG;
    srq_status_t s = check_qspec(q);
    if (s != SRQ_OK) return s;
    if (!codes_rm && !codes_tr) return SRQ_ERR_INVALID_ARG;
    if (codes_rm && (!scale_rm || ld_rm < cols)) return SRQ_ERR_INVALID_ARG;
    if (codes_tr && (!scale_tr || ld_tr < rows)) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || !aligned_to(ws, 256)) return SRQ_ERR_INVALID_ARG;
    if (ws_bytes < srq_quantize_workspace_bytes(rows, cols)) return SRQ_ERR_WORKSPACE;
    if (rows == 0 || cols == 0) return SRQ_OK;
    uint32_t* status = &((WsHeader*)ws)->status;
    if (cudaMemsetAsync(ws, 0, srq_quantize_workspace_bytes(rows, cols), st) != cudaSuccess) return SRQ_ERR_CUDA;
    QuantArgs a;
    a.x = x; a.dt = dt; a.rows = rows; a.cols = cols; a.ld = ld; a.q = *q;
    a.codes_rm = codes_rm; a.ld_rm = ld_rm; a.scale_rm = scale_rm;
    a.codes_tr = codes_tr; a.ld_tr = ld_tr; a.scale_tr = scale_tr;
    const QuantScratch sc = carve_quant_scratch((char*)ws + sizeof(WsHeader), rows, cols);
    return launch_quantize(a, sc, status, st, true) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}

srq_status_t srq_absmax(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* absmax, void* cuda_stream) {
    if (!x || !absmax || rows < 0 || cols < 0 || ld < cols) return SRQ_ERR_INVALID_ARG;
    if (dt != SRQ_F32 && dt != SRQ_BF16) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || !aligned_to(absmax, 4)) return SRQ_ERR_INVALID_ARG;
    return launch_absmax(x, dt, rows, cols, ld, absmax, (cudaStream_t)cuda_stream) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}

srq_status_t srq_absmax_cols(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* absmax_cols,
                             void* cuda_stream) {
    if (!x || !absmax_cols || rows < 0 || cols < 0 || ld < cols) return SRQ_ERR_INVALID_ARG;
    if (dt != SRQ_F32 && dt != SRQ_BF16) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || !aligned_to(absmax_cols, 4)) return SRQ_ERR_INVALID_ARG;
    return launch_absmax_cols(x, dt, rows, cols, ld, absmax_cols, (cudaStream_t)cuda_stream) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}

srq_status_t srq_gemm_i8(const int8_t* a, int64_t lda, const int8_t* b, int64_t ldb, int64_t M, int64_t N, int64_t Kc,
                         const float* s_row, int32_t row_stride, const float* s_col, int32_t col_stride,
                         float* out, int64_t ldo, int32_t* acc_out, void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!a || !b || !s_row || !s_col || !out || !ws) return SRQ_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || Kc <= 0 || lda < Kc || ldb < Kc || ldo < N) return SRQ_ERR_INVALID_ARG;
    if ((row_stride != 0 && row_stride != 1) || (col_stride != 0 && col_stride != 1)) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(a, 16) || !aligned_to(b, 16) || lda % 16 || ldb % 16 || !aligned_to(ws, 256)) return SRQ_ERR_INVALID_ARG;
    if ((double)Kc * 127.0 * 127.0 >= 2147483648.0) return SRQ_ERR_ACC_OVERFLOW;
    if (ws_bytes < sizeof(WsHeader)) return SRQ_ERR_WORKSPACE;
    if (M == 0 || N == 0) return SRQ_OK;
    uint32_t* status = &((WsHeader*)ws)->status;
    if (clear_header(ws, st) != cudaSuccess) return SRQ_ERR_CUDA;
    GemmArgs g;
    g.a = a; g.lda = lda; g.b = b; g.ldb = ldb; g.M = M; g.N = N; g.Kc = Kc; g.kind = 0;
    g.s_row = s_row; g.row_stride = row_stride; g.s_col = s_col; g.col_stride = col_stride;
    g.out = out; g.ldo = ldo; g.acc_out = acc_out;
    g.splitk_ws = (char*)ws + sizeof(WsHeader); g.splitk_ws_bytes = ws_bytes - sizeof(WsHeader);
    return launch_gemm_i8(g, status, st);
}

srq_status_t srq_gemm_e4m3(const uint8_t* a, int64_t lda, const uint8_t* b, int64_t ldb, int64_t M, int64_t N, int64_t Kc,
                           const float* s_row, int32_t row_stride, const float* s_col, int32_t col_stride,
                           float* out, int64_t ldo, float* acc_out, void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!a || !b || !s_row || !s_col || !out || !ws) return SRQ_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || Kc <= 0 || lda < Kc || ldb < Kc || ldo < N) return SRQ_ERR_INVALID_ARG;
    if ((row_stride != 0 && row_stride != 1) || (col_stride != 0 && col_stride != 1)) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(a, 16) || !aligned_to(b, 16) || lda % 16 || ldb % 16 || !aligned_to(ws, 256)) return SRQ_ERR_INVALID_ARG;
    if (ws_bytes < sizeof(WsHeader)) return SRQ_ERR_WORKSPACE;
    if (M == 0 || N == 0) return SRQ_OK;
    uint32_t* status = &((WsHeader*)ws)->status;
    if (clear_header(ws, st) != cudaSuccess) return SRQ_ERR_CUDA;
    GemmArgs g;
    g.a = (const int8_t*)a; g.lda = lda; g.b = (const int8_t*)b; g.ldb = ldb; g.M = M; g.N = N; g.Kc = Kc; g.kind = 1;
    g.s_row = s_row; g.row_stride = row_stride; g.s_col = s_col; g.col_stride = col_stride;
    g.out = out; g.ldo = ldo; g.acc_out = (int32_t*)acc_out;       // raw binary32 sums, copied bit for bit
    g.splitk_ws = nullptr; g.splitk_ws_bytes = 0;
    return launch_gemm_i8(g, status, st);
}

srq_status_t qlinear_fwd(const void* A, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                         const srq_qspec_t* qA, const srq_qspec_t* qW, float* Y, const srq_debug_out_t* dbg,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
    if (qA && qA->format == SRQ_GRID_NONE) return run_fwd_fp_act(A, W, dt, T, N, K, qW, Y, ws, ws_bytes, cuda_stream);
    const Operand a{A, T, K, false, qA}, b{W, N, K, false, qW};
    return run_layer(a, b, dt, Y, nullptr, dbg, ws, ws_bytes, cuda_stream);
}

srq_status_t qlinear_bwd_input(const void* dY, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                               const srq_qspec_t* qdY, const srq_qspec_t* qW, float* dA, const srq_debug_out_t* dbg,
                               void* ws, size_t ws_bytes, void* cuda_stream) {
    const Operand a{dY, T, N, false, qdY}, b{W, N, K, true, qW};
    return run_layer(a, b, dt, dA, nullptr, dbg, ws, ws_bytes, cuda_stream);
}

srq_status_t qlinear_bwd_weight(const void* dY, const void* A, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                                const srq_qspec_t* qdY, const srq_qspec_t* qA, float* dW, const srq_debug_out_t* dbg,
                                void* ws, size_t ws_bytes, void* cuda_stream) {
    const Operand a{dY, T, N, true, qdY}, b{A, T, K, true, qA};
    return run_layer(a, b, dt, dW, nullptr, dbg, ws, ws_bytes, cuda_stream);
}

srq_status_t qlinear_bwd(const void* dY, const void* A, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                         const srq_qspec_t* qdY, const srq_qspec_t* qA, const srq_qspec_t* qW, float* dA, float* dW,
                         const srq_debug_out_t* dbg_input, const srq_debug_out_t* dbg_weight,
                         void* ws, size_t ws_bytes, void* cuda_stream) {
    return run_bwd(dY, A, W, dt, T, N, K, qdY, qA, qW, dA, dW, nullptr, nullptr, dbg_input, dbg_weight, ws, ws_bytes, cuda_stream);
}

srq_status_t srq_gemm_i8_ex(const int8_t* a, int64_t lda, const int8_t* b, int64_t ldb, int64_t M, int64_t N, int64_t Kc,
                            const float* s_row, int32_t row_stride, const float* s_col, int32_t col_stride,
                            float* out, int64_t ldo, int32_t* acc_out, const srq_output_t* output,
                            void* ws, size_t ws_bytes, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!a || !b || !s_row || !s_col || !ws) return SRQ_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || Kc <= 0 || lda < Kc || ldb < Kc || (out && ldo < N)) return SRQ_ERR_INVALID_ARG;
    if ((row_stride != 0 && row_stride != 1) || (col_stride != 0 && col_stride != 1)) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(a, 16) || !aligned_to(b, 16) || lda % 16 || ldb % 16 || !aligned_to(ws, 256)) return SRQ_ERR_INVALID_ARG;
    if ((double)Kc * 127.0 * 127.0 >= 2147483648.0) return SRQ_ERR_ACC_OVERFLOW;
    if (ws_bytes < sizeof(WsHeader)) return SRQ_ERR_WORKSPACE;
    GemmArgs g;
    const srq_status_t so = make_out_options(output, N, out != nullptr, &g.opt);
    if (so != SRQ_OK) return so;
    if (!aligned_to(out, g.opt.out_bf16 ? 2 : 4)) return SRQ_ERR_INVALID_ARG;
    if (M == 0 || N == 0) return SRQ_OK;
    uint32_t* status = &((WsHeader*)ws)->status;
    if (clear_header(ws, st) != cudaSuccess) return SRQ_ERR_CUDA;
    g.a = a; g.lda = lda; g.b = b; g.ldb = ldb; g.M = M; g.N = N; g.Kc = Kc; g.kind = 0;
    g.s_row = s_row; g.row_stride = row_stride; g.s_col = s_col; g.col_stride = col_stride;
    g.out = out; g.ldo = ldo; g.acc_out = acc_out;
    g.splitk_ws = (char*)ws + sizeof(WsHeader); g.splitk_ws_bytes = ws_bytes - sizeof(WsHeader);
    return launch_gemm_i8(g, status, st);
}

srq_status_t qlinear_fwd_ex(const void* A, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                            const srq_qspec_t* qA, const srq_qspec_t* qW, float* Y, const srq_output_t* output,
                            const srq_debug_out_t* dbg, void* ws, size_t ws_bytes, void* cuda_stream) {
    const Operand a{A, T, K, false, qA}, b{W, N, K, false, qW};
    return run_layer(a, b, dt, Y, output, dbg, ws, ws_bytes, cuda_stream);
}

srq_status_t qlinear_bwd_ex(const void* dY, const void* A, const void* W, srq_dtype_t dt, int64_t T, int64_t N, int64_t K,
                            const srq_qspec_t* qdY, const srq_qspec_t* qA, const srq_qspec_t* qW, float* dA, float* dW,
                            const srq_output_t* output_dA, const srq_output_t* output_dW,
                            const srq_debug_out_t* dbg_input, const srq_debug_out_t* dbg_weight,
                            void* ws, size_t ws_bytes, void* cuda_stream) {
    return run_bwd(dY, A, W, dt, T, N, K, qdY, qA, qW, dA, dW, output_dA, output_dW, dbg_input, dbg_weight, ws, ws_bytes, cuda_stream);
}

srq_status_t srq_dequant_i32(const int32_t* acc, int64_t ld_acc, int64_t M, int64_t N, const float* s_row, int32_t row_stride,
                             const float* s_col, int32_t col_stride, void* out, int64_t ldo, int32_t out_bf16, void* cuda_stream) {
    if (!acc || !s_row || !s_col || !out) return SRQ_ERR_INVALID_ARG;
    if (M < 0 || N < 0 || ld_acc < N || ldo < N) return SRQ_ERR_INVALID_ARG;
    if ((row_stride != 0 && row_stride != 1) || (col_stride != 0 && col_stride != 1)) return SRQ_ERR_INVALID_ARG;
    if (out_bf16 != 0 && out_bf16 != 1) return SRQ_ERR_INVALID_ARG;
    if (!aligned_to(acc, 4) || !aligned_to(s_row, 4) || !aligned_to(s_col, 4) || !aligned_to(out, out_bf16 ? 2 : 4)) return SRQ_ERR_INVALID_ARG;
    return launch_finish_sums(acc, ld_acc, M, N, s_row, row_stride, s_col, col_stride, (float*)out, ldo, out_bf16,
                              (cudaStream_t)cuda_stream) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}

void srq_plan_splits(int64_t tiles, int32_t k_blocks, int32_t groups, int32_t* full_tiles, int32_t* splits) {
    if (!full_tiles || !splits) return;
    *full_tiles = 0; *splits = 0;
    if (tiles <= 0 || k_blocks <= 0 || groups <= 0 || tiles > 2147483647ll) return;
    gemm_plan_splits(tiles, k_blocks, groups, full_tiles, splits);
}

srq_status_t srq_selftest_bounded_wait(void* ws, size_t ws_bytes, uint32_t limit_us, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!ws || !aligned_to(ws, 256) || limit_us == 0 || limit_us > 1000000u) return SRQ_ERR_INVALID_ARG;
    if (ws_bytes < sizeof(WsHeader)) return SRQ_ERR_WORKSPACE;
    if (clear_header(ws, st) != cudaSuccess) return SRQ_ERR_CUDA;
    return launch_bounded_wait_probe(&((WsHeader*)ws)->status, (uint64_t)limit_us * 1000ull, st) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}

srq_status_t srq_set_product_timer(uint64_t* slots, int64_t n) {
    if (n < 0 || (n > 0 && (!slots || !aligned_to(slots, 8)))) return SRQ_ERR_INVALID_ARG;
    set_product_timer((unsigned long long*)slots, n);
    return SRQ_OK;
}

srq_status_t srq_selftest_mma_rate(void* ws, size_t ws_bytes, int32_t k_blocks, int64_t* ops, void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!ws || !aligned_to(ws, 256) || k_blocks < 1 || k_blocks > (1 << 22)) return SRQ_ERR_INVALID_ARG;
    if (ws_bytes < sizeof(WsHeader)) return SRQ_ERR_WORKSPACE;
    if (clear_header(ws, st) != cudaSuccess) return SRQ_ERR_CUDA;
    return launch_mma_rate(k_blocks, &((WsHeader*)ws)->status, ops, st);
}

srq_status_t srq_poll_status(void* ws, void* cuda_stream) {
    if (!ws) return SRQ_ERR_INVALID_ARG;
    uint32_t v = 0;
    if (cudaMemcpyAsync(&v, &((WsHeader*)ws)->status, 4, cudaMemcpyDeviceToHost, (cudaStream_t)cuda_stream) != cudaSuccess)
        return SRQ_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)cuda_stream) != cudaSuccess) return SRQ_ERR_CUDA;
    return (srq_status_t)v;
}

const char* srq_status_string(srq_status_t s) {
    switch (s) {
        case SRQ_OK: return "ok";
        case SRQ_ERR_INVALID_ARG: return "invalid argument";
        case SRQ_ERR_UNSUPPORTED: return "unsupported bit width";
        case SRQ_ERR_WORKSPACE: return "workspace too small";
        case SRQ_ERR_ACC_OVERFLOW: return "contraction too long for int32 accumulation";
        case SRQ_ERR_CUDA: return "CUDA call failed";
        case SRQ_ERR_NONFINITE: return "input is not finite";
        case SRQ_ERR_TIMEOUT: return "bounded wait in a kernel ran out";
    }
    return "unknown status";
}

uint64_t srq_launch_count(void) { return (uint64_t)g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
