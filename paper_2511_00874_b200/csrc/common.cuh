// Shared declarations of the CUDA side of libsrq: workspace header, launch accounting and the
// internal launchers that the C-ABI file strings together.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "srq.h"

namespace srq {

// First 256 bytes of every workspace.
struct WsHeader {
    uint32_t status;    // srq_status_t recorded by device code (first error wins)
    uint32_t pad[63];
};
static_assert(sizeof(WsHeader) == 256, "header is one 256-byte line");

constexpr size_t kAlign = 256;
__host__ __device__ inline size_t align_up(size_t v, size_t a = kAlign) { return (v + a - 1) / a * a; }

// Kernels launched by this process (host counter; entry points may be called from several threads).
extern std::atomic<unsigned long long> g_launches;
inline void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

// Programmatic dependent launch.  Every kernel of the library waits for the results of the work before
// it as its first act (griddepcontrol.wait returns once the preceding grids have finished and their
// writes are visible; it returns at once for a kernel launched the ordinary way) and then lets the
// kernel after it be launched, so that the successor's launch and start-up overlap this kernel's
// execution instead of following it.  Nothing is read or written before the wait, so the order of the
// stream is kept; a kernel two places ahead has finished as well, because the one in between only
// finishes after its own wait.  A kernel launched through launch_pdl (or with the same attribute)
// that did NOT start with pdl_enter() could read its predecessor's half-written output, so every
// __global__ function of the library starts with it; a host-side test reads the sources and fails
// for a kernel that does not.
__device__ __forceinline__ void pdl_enter() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// The two halves on their own, for a kernel whose set-up touches no global memory: it lets its successor
// be launched at once and waits for its predecessor only when the set-up is done, so that the set-up
// overlaps the predecessor's tail.  Nothing the predecessor wrote may be read, and nothing it may
// still read may be written, before pdl_wait().
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Not while the stream is being captured: in a replayed graph the ordinary kernel-to-kernel edges were
// measured faster than the programmatic ones (0.104 against 0.111 ms for a 15-kernel layer).
static inline bool pdl_allowed(cudaStream_t st) {
    cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
    return cudaStreamIsCapturing(st, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusNone;
}
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &at; cfg.numAttrs = pdl_allowed(st) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ void record_status(uint32_t* status, uint32_t code) {
    atomicCAS(status, 0u, code);
}

// ------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds, two 32x32->64 multiplies per round.
// The ten round keys (key + r * Weyl constants) are the same for every thread; the host
// computes them once and passes them in the kernel parameters.
// ------------------------------------------------------------------------------------------
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
    uint32_t tid0, tid1;     // counter words 2 and 3 (tensor_id)
};

__device__ __forceinline__ void philox_rounds(uint32_t c0, uint32_t c1, const PhiloxKeys& K, uint32_t out[4]) {
    uint32_t c2 = K.tid0, c3 = K.tid1;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;    // one wide multiply: hi and lo
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c3 = (uint32_t)p0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The same ten rounds, returning the COMPLEMENT of every output word (what the rounding rule adds):
// in the last round the two words that are low halves of products come complemented from a
// multiply-add of their own ( ~lo(M c) = lo((-M) c) - 1 ), and the two that end in an exclusive-or
// absorb the complement into that operation, so that no separate NOT is spent on any of them.
__device__ __forceinline__ void philox_rounds_not(uint32_t c0, uint32_t c1, const PhiloxKeys& K, uint32_t out[4]) {
    uint32_t c2 = K.tid0, c3 = K.tid1;
#pragma unroll
    for (int r = 0; r < 9; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        c0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        c1 = (uint32_t)p1;
        c2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c3 = (uint32_t)p0;
    }
    const uint32_t h0 = __umulhi(0xD2511F53u, c0), h1 = __umulhi(0xCD9E8D57u, c2);
    out[0] = ~(h1 ^ c1 ^ K.k0[9]);
    out[1] = c2 * 0x326172A9u + 0xFFFFFFFFu;         // -0xCD9E8D57 mod 2^32
    out[2] = ~(h0 ^ c3 ^ K.k1[9]);
    out[3] = c0 * 0x2DAEE0ADu + 0xFFFFFFFFu;         // -0xD2511F53 mod 2^32
}

// Round keys and upper counter words for one quantization point.
inline PhiloxKeys make_philox_keys(uint64_t seed, uint64_t tensor_id) {
    PhiloxKeys k;
    for (int r = 0; r < 10; ++r) {
        k.k0[r] = (uint32_t)seed + (uint32_t)r * 0x9E3779B9u;
        k.k1[r] = (uint32_t)(seed >> 32) + (uint32_t)r * 0xBB67AE85u;
    }
    k.tid0 = (uint32_t)tensor_id; k.tid1 = (uint32_t)(tensor_id >> 32);
    return k;
}

// SRQ_OK, or why the quantization point cannot be used: unknown grid, scale or rounding mode, a bit
// width outside the grid's range, a mode the grid does not have, a misaligned absmax pointer.
srq_status_t check_qspec(const srq_qspec_t* q);

// ------------------------------------------------------------------------------------------
// Quantizer (quantize.cu)
// ------------------------------------------------------------------------------------------
// Scratch carved from a workspace for one sr_quantize: absmax words and reciprocal steps for
// the row-major layout (1 or rows) and the transposed layout (1 or cols).
struct QuantScratch {
    uint32_t* counter;   // CTAs of the absmax launch that have finished, zeroed before use
    uint32_t* amax_rm;   // fp32 bit patterns, zeroed before use
    uint32_t* amax_tr;
    float* inv_rm;
    float* inv_tr;
    size_t bytes;        // total bytes carved (multiple of 256)
};
size_t quant_scratch_bytes(int64_t rows, int64_t cols);
QuantScratch carve_quant_scratch(void* base, int64_t rows, int64_t cols);

struct QuantArgs {
    const void* x; srq_dtype_t dt; int64_t rows, cols, ld;
    srq_qspec_t q;
    int8_t* codes_rm; int64_t ld_rm; float* scale_rm;
    int8_t* codes_tr; int64_t ld_tr; float* scale_tr;
};
// Enqueues: clear scratch (unless the caller has zeroed the whole scratch block already), absmax with
// step sizes, quantize.  `scratch` must be exclusively this call's until the kernels finish.
cudaError_t launch_quantize(const QuantArgs& a, const QuantScratch& scratch, uint32_t* status,
                            cudaStream_t stream, bool scratch_zeroed = false);

// The operands of one layer call (n <= 3, scratch blocks already zeroed): two launches for all of them
// together where the problem is small, else launch_quantize for each.  Same results either way.
cudaError_t launch_quantize_batch(const QuantArgs* a, const QuantScratch* s, int n, uint32_t* status, cudaStream_t stream,
                                  bool scratch_zeroed);

// max |x| of the whole matrix into *absmax (device float, overwritten).
cudaError_t launch_absmax(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* absmax, cudaStream_t stream);
// absmax_cols[c] = max over the rows of |x[r, c]| (device [cols], overwritten).
cudaError_t launch_absmax_cols(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* absmax_cols,
                               cudaStream_t stream);

// int8 codes as bfloat16 integers (pitches in elements); *one receives 1.0f.
cudaError_t launch_widen_codes(const int8_t* codes, int64_t rows, int64_t cols, int64_t ld, void* out_bf16, int64_t ld_out,
                               float* one, cudaStream_t stream);

// ------------------------------------------------------------------------------------------
// int8 GEMM (gemm_i8.cu)
// ------------------------------------------------------------------------------------------
// What else a product does with its results (all optional).
struct OutOptions {
    int32_t accumulate = 0;          // out += result instead of out = result
    int32_t out_bf16 = 0;            // out holds bfloat16 [M, ldo]: each result rounded to nearest even
    int32_t raw_sums = 0;            // out holds int32 [M, ldo]: the sums themselves, nothing is scaled
    int32_t requant = 0;             // also write Q(result) as int8 codes with a given step size
    int32_t rq_sr = 0;               // stochastic rounding (else round to nearest)
    float rq_lim = 0.0f;             // qmax * 2^24: saturation bound of the fixed-point quotient
    const float* rq_step = nullptr;  // device [1]
    int8_t* rq_codes = nullptr; int64_t rq_ld = 0;
    uint64_t rq_offset = 0;          // flat index of result [0, 0] in the threshold stream
    PhiloxKeys rq_keys = {};
    uint32_t* absmax_bits = nullptr; // device [1]: raised to the bit pattern of max |result|
};

struct GemmArgs {
    const int8_t* a; int64_t lda; const int8_t* b; int64_t ldb;
    int64_t M, N, Kc;
    int kind;                                   // 0: int8 codes, int32 sums; 1: E4M3 codes, binary32 sums;
                                                // 2: bfloat16 operands, binary32 sums (Kc, lda, ldb in BYTES)
    const float* s_row; int32_t row_stride; const float* s_col; int32_t col_stride;
    float* out; int64_t ldo; int32_t* acc_out;
    OutOptions opt;
    void* splitk_ws; size_t splitk_ws_bytes;   // int32 [M,N] partial sums
};
size_t gemm_splitk_bytes(int64_t M, int64_t N);
// Host-side planning of the split contraction (exposed for tests).
void gemm_plan_splits(int64_t tiles, int32_t num_kb, int groups, int32_t* full_tiles, int32_t* splits);
// One thread waits (at most limit_ns) on a barrier nobody signals and records SRQ_ERR_TIMEOUT.
cudaError_t launch_bounded_wait_probe(uint32_t* status, uint64_t limit_ns, cudaStream_t stream);
// out = float(acc) * (s_row * s_col) over a caller's int32 matrix (the finishing step on its own).
cudaError_t launch_finish_sums(const int32_t* acc, int64_t ld_acc, int64_t M, int64_t N, const float* s_row, int32_t row_stride,
                               const float* s_col, int32_t col_stride, float* out, int64_t ldo, int out_bf16, cudaStream_t stream);
srq_status_t launch_gemm_i8(const GemmArgs& g, uint32_t* status, cudaStream_t stream);
// Device-side timing of the next n product launches into slots[2 * i] (start) / slots[2 * i + 1] (end).
void set_product_timer(unsigned long long* slots, int64_t n);
// Tensor-pipe issue-rate microbenchmark: every CTA pair issues k_blocks x 4 kind::i8 MMAs (M256 N256 K32)
// on operands resident in shared memory; *ops receives the integer operations of the launch.
srq_status_t launch_mma_rate(int32_t k_blocks, uint32_t* status, int64_t* ops, cudaStream_t stream);

}  // namespace srq
