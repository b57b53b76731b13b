// Absmax reduction, step sizes and the SR / RTN quantizer (Def. 1-3 of the paper).
//
// Three kernels per quantized tensor:
//   amax_kernel      one read of x; max |x| per tensor, per row and/or per column, kept as the
//                    binary32 bit pattern (non-negative floats order like unsigned integers,
//                    so atomicMax on the bits is exact and order independent)
//   scales_kernel    D = m / qmax (round to nearest) and 1/D = qmax / m rounded toward zero, so
//                    that no quotient x * (1/D) of the group exceeds qmax and no clamp is needed
//   quantize_kernel  second read of x; t = x * (1/D) (one binary32 multiply), then Def. 1 on
//                    real numbers: SR rounds up iff u24 * 2^-24 < frac(t) with u24 from
//                    Philox4x32-10 keyed by (seed, tensor_id, flat index); RTN rounds up iff
//                    frac(t) >= 1/2; code = clamp(floor(t) + up).  The comparison is evaluated
//                    exactly, in fixed point with 24 fractional bits (see quantize_elem).
//                    Writes the row-major code layout directly and the transposed layout
//                    through a swizzled shared-memory tile, so that both are stored with
//                    full 128-byte lines.
//
// The two multiplies that produce the fixed-point quotient use explicit round-to-nearest
// intrinsics so that the compiler cannot merge them.
#include <cuda_bf16.h>

#include "common.cuh"

namespace srq {

std::atomic<unsigned long long> g_launches{0};

// ------------------------------------------------------------------------------------------
// scratch carving
// ------------------------------------------------------------------------------------------
static inline size_t f32_block(int64_t n) { return align_up((size_t)n * 4); }

size_t quant_scratch_bytes(int64_t rows, int64_t cols) {
    return kAlign + 2 * (f32_block(rows) + f32_block(cols));
}

QuantScratch carve_quant_scratch(void* base, int64_t rows, int64_t cols) {
    // counter and amax blocks first and contiguous, so that one memset clears them
    char* p = (char*)base;
    QuantScratch s;
    s.counter = (uint32_t*)p; p += kAlign;
    s.amax_rm = (uint32_t*)p; p += f32_block(rows);
    s.amax_tr = (uint32_t*)p; p += f32_block(cols);
    s.inv_rm = (float*)p; p += f32_block(rows);
    s.inv_tr = (float*)p; p += f32_block(cols);
    s.bytes = (size_t)(p - (char*)base);
    return s;
}

// ------------------------------------------------------------------------------------------
// element access
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) {
    return __uint_as_float((uint32_t)__bfloat16_as_ushort(v) << 16);
}

// Four consecutive elements starting at column c of one row; columns >= cols read as 0.
template <typename T>
__device__ __forceinline__ void load4(const T* row, int64_t c, int64_t cols, bool vec_ok, float v[4]) {
    if (vec_ok && c + 4 <= cols) {
        if constexpr (sizeof(T) == 4) {
            float4 q = __ldcs(reinterpret_cast<const float4*>(row + c));
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else {
            uint2 q = __ldcs(reinterpret_cast<const uint2*>(row + c));
            v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xFFFF0000u);
            v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xFFFF0000u);
        }
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) v[e] = (c + e < cols) ? to_f32(row[c + e]) : 0.0f;
    }
}

__device__ __forceinline__ uint32_t abs_bits(float v) { return __float_as_uint(v) & 0x7FFFFFFFu; }

// ------------------------------------------------------------------------------------------
// absmax
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void scale_from_bits(uint32_t bits, float qmax, float* delta, float* inv,
                                                uint32_t* status) {
    if (bits >= 0x7F800000u) record_status(status, SRQ_ERR_NONFINITE);
    const float m = __uint_as_float(bits);
    // toward zero, so that |x * r| <= qmax for the whole group; a reciprocal that overflows when
    // rounded to nearest marks a group too small to scale, which is treated as all zeros
    float r = 0.0f;
    if (m != 0.0f && fabsf(__fdiv_rn(qmax, m)) <= 3.402823466e38f) r = __fdiv_rz(qmax, m);
    *inv = r;
    *delta = (r == 0.0f) ? 0.0f : __fdiv_rn(m, qmax);
}

// What the last CTA of an absmax launch does once every CTA has contributed: the step sizes of all
// groups (saves a launch; `counter` must be zero when the launch starts).  counter == nullptr: nothing.
struct ScaleStep {
    uint32_t* counter;
    int64_t n_rm; float* inv_rm; float* delta_rm;
    int64_t n_tr; float* inv_tr; float* delta_tr;
    float qmax;
    uint32_t* status;
};

constexpr int AMAX_THREADS = 256;
constexpr int AMAX_TILE_R = 64;    // 8 warps x 8 rows
constexpr int AMAX_GROUPS = 2;     // 16-byte groups per lane and row

// Absolute-value bit patterns of the elements of one 16-byte group.
__device__ __forceinline__ void abs_bits16(const uint4& q, uint32_t (&b)[4], float) {
    b[0] = q.x & 0x7FFFFFFFu; b[1] = q.y & 0x7FFFFFFFu; b[2] = q.z & 0x7FFFFFFFu; b[3] = q.w & 0x7FFFFFFFu;
}
__device__ __forceinline__ void abs_bits16(const uint4& q, uint32_t (&b)[8], __nv_bfloat16) {
    b[0] = (q.x << 16) & 0x7FFFFFFFu; b[1] = q.x & 0x7FFF0000u; b[2] = (q.y << 16) & 0x7FFFFFFFu; b[3] = q.y & 0x7FFF0000u;
    b[4] = (q.z << 16) & 0x7FFFFFFFu; b[5] = q.z & 0x7FFF0000u; b[6] = (q.w << 16) & 0x7FFFFFFFu; b[7] = q.w & 0x7FFF0000u;
}
// Largest absolute-value bit pattern of the group (binary32 pattern in both cases).
__device__ __forceinline__ uint32_t abs_max16(const uint4& q, float) {
    return max(max(q.x & 0x7FFFFFFFu, q.y & 0x7FFFFFFFu), max(q.z & 0x7FFFFFFFu, q.w & 0x7FFFFFFFu));
}
__device__ __forceinline__ uint32_t abs_max16(const uint4& q, __nv_bfloat16) {
    // two bfloat16 per word: packed 16-bit maxima, then the larger half widened
    const uint32_t m = __vmaxu2(__vmaxu2(q.x & 0x7FFF7FFFu, q.y & 0x7FFF7FFFu), __vmaxu2(q.z & 0x7FFF7FFFu, q.w & 0x7FFF7FFFu));
    return max(m << 16, m & 0xFFFF0000u);
}

// ROWS: one word per row wanted; COLS: one word per column wanted; neither: one word for the tensor.
// A CTA covers 64 rows x (32 lanes x 2 groups x 16 bytes); four rows (eight 16-byte loads per thread)
// are in flight at a time.  vec_ok: base and pitch allow 16-byte loads.
template <typename T, bool ROWS, bool COLS>
__device__ __forceinline__ void amax_tile(const T* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, bool vec_ok,
                                          uint32_t* __restrict__ amax_rm, uint32_t* __restrict__ amax_tr, int64_t blk) {
    constexpr int EPL = 16 / (int)sizeof(T);                   // elements per 16-byte group
    constexpr int TILE_C = 32 * AMAX_GROUPS * EPL;
    __shared__ uint32_t col_max[COLS ? TILE_C : 1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_tc = (cols + TILE_C - 1) / TILE_C;
    const int64_t c0 = (blk % n_tc) * TILE_C;
    const int64_t r0 = (blk / n_tc) * AMAX_TILE_R;
    if constexpr (COLS) {
        for (int i = threadIdx.x; i < TILE_C; i += AMAX_THREADS) col_max[i] = 0u;
        __syncthreads();
    }
    uint32_t cm[COLS ? AMAX_GROUPS * EPL : 1];
#pragma unroll
    for (int i = 0; i < (COLS ? AMAX_GROUPS * EPL : 1); ++i) cm[i] = 0u;
    uint32_t all = 0u;
#pragma unroll 1
    for (int rr = 0; rr < AMAX_TILE_R / 8; rr += 4) {
        uint4 v[4][AMAX_GROUPS];
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int64_t r = r0 + warp + 8 * (rr + h);
#pragma unroll
            for (int g = 0; g < AMAX_GROUPS; ++g) {
                const int64_t c = c0 + (int64_t)(g * 32 + lane) * EPL;
                v[h][g] = make_uint4(0u, 0u, 0u, 0u);
                if (r < rows && c < cols) {
                    const T* src = x + r * ld + c;
                    if (vec_ok && c + EPL <= cols) {
                        v[h][g] = __ldcs(reinterpret_cast<const uint4*>(src));
                    } else {                                       // ragged or unaligned: element by element
                        T tmp[EPL];
#pragma unroll
                        for (int e = 0; e < EPL; ++e) tmp[e] = (c + e < cols) ? src[e] : T(0.0f);
                        memcpy(&v[h][g], tmp, 16);
                    }
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int64_t r = r0 + warp + 8 * (rr + h);
            uint32_t rmax = 0u;
#pragma unroll
            for (int g = 0; g < AMAX_GROUPS; ++g) {
                if constexpr (COLS) {
                    uint32_t b[EPL];
                    abs_bits16(v[h][g], b, T());
#pragma unroll
                    for (int e = 0; e < EPL; ++e) { rmax = max(rmax, b[e]); cm[g * EPL + e] = max(cm[g * EPL + e], b[e]); }
                } else {
                    rmax = max(rmax, abs_max16(v[h][g], T()));
                }
            }
            if constexpr (ROWS) {
                rmax = __reduce_max_sync(0xFFFFFFFFu, rmax);
                if (lane == 0 && rmax && r < rows) atomicMax(&amax_rm[r], rmax);
            } else {
                all = max(all, rmax);
            }
        }
    }
    if constexpr (!ROWS && !COLS) {
        // one word for the whole tensor: combine the CTA first, and only touch the word when this
        // CTA can raise it (atomics on one address are serialised by the memory system)
        __shared__ uint32_t warp_max[AMAX_THREADS / 32];
        all = __reduce_max_sync(0xFFFFFFFFu, all);
        if (lane == 0) warp_max[warp] = all;
        __syncthreads();
        if (threadIdx.x == 0) {
#pragma unroll
            for (int w = 1; w < AMAX_THREADS / 32; ++w) all = max(all, warp_max[w]);
            if (all > __ldcg(&amax_rm[0])) atomicMax(&amax_rm[0], all);
        }
    }
    if constexpr (COLS) {
#pragma unroll
        for (int g = 0; g < AMAX_GROUPS; ++g)
#pragma unroll
            for (int e = 0; e < EPL; ++e)
                if (cm[g * EPL + e]) atomicMax(&col_max[(g * 32 + lane) * EPL + e], cm[g * EPL + e]);
        __syncthreads();
        for (int i = threadIdx.x; i < TILE_C; i += AMAX_THREADS) {
            const int64_t c = c0 + i;
            if (c < cols && col_max[i]) atomicMax(&amax_tr[c], col_max[i]);
        }
    }
}

// True in exactly one CTA of the launch: the one that finishes last (`counter` is zero at launch).
__device__ __forceinline__ bool last_cta_of_launch(uint32_t* counter) {
    __shared__ uint32_t is_last;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(counter, 1u) == gridDim.x - 1 ? 1u : 0u;
    __syncthreads();
    if (is_last) __threadfence();
    return is_last != 0u;
}

// Step sizes of all groups of one operand from their maxima (one CTA).
__device__ __forceinline__ void scale_step(const ScaleStep& S, const uint32_t* amax_rm, const uint32_t* amax_tr) {
    for (int64_t i = threadIdx.x; i < S.n_rm; i += blockDim.x) {
        float d, r;
        scale_from_bits(__ldcg(&amax_rm[i]), S.qmax, &d, &r, S.status);
        S.inv_rm[i] = r;
        if (S.delta_rm) S.delta_rm[i] = d;
    }
    for (int64_t i = threadIdx.x; i < S.n_tr; i += blockDim.x) {
        float d, r;
        scale_from_bits(__ldcg(&amax_tr[i]), S.qmax, &d, &r, S.status);
        S.inv_tr[i] = r;
        if (S.delta_tr) S.delta_tr[i] = d;
    }
}

template <typename T, bool ROWS, bool COLS>
__global__ void __launch_bounds__(AMAX_THREADS, COLS ? 3 : 4)
amax_kernel(const T* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, bool vec_ok,
            uint32_t* __restrict__ amax_rm, uint32_t* __restrict__ amax_tr, const ScaleStep S) {
    pdl_enter();
    amax_tile<T, ROWS, COLS>(x, rows, cols, ld, vec_ok, amax_rm, amax_tr, (int64_t)blockIdx.x);
    if (S.counter == nullptr) return;
    // the CTA that arrives last sees every maximum and turns them into step sizes
    if (last_cta_of_launch(S.counter)) scale_step(S, amax_rm, amax_tr);
}

// The operands of one layer call in ONE launch (small problems, where the launches themselves are what
// takes the time): CTAs [first_block[i], first_block[i + 1]) take the tiles of operand i; an operand
// whose maxima are known contributes no tiles.  The CTA that finishes last derives every operand's
// step sizes.  Same arithmetic as amax_kernel, flags chosen at run time.
constexpr int BATCH_MAX = 3;
struct AmaxOperand {
    const void* x; int64_t rows, cols, ld;
    uint32_t* amax_rm; uint32_t* amax_tr;            // where the tiles put their maxima
    const uint32_t* src_rm; const uint32_t* src_tr;  // what the step sizes are derived from (may be given maxima)
    int32_t want_rows, want_cols, vec_ok;
    ScaleStep S;
};
struct AmaxBatch {
    AmaxOperand op[BATCH_MAX];
    uint32_t first_block[BATCH_MAX + 1];
    int32_t n;
    uint32_t* counter;
};

template <typename T>
__global__ void __launch_bounds__(AMAX_THREADS, 3)
amax_batch_kernel(const __grid_constant__ AmaxBatch Bt) {
    pdl_enter();
    int i = 0;
    while (i + 1 < Bt.n && blockIdx.x >= Bt.first_block[i + 1]) ++i;
    if (blockIdx.x < Bt.first_block[Bt.n]) {
        const AmaxOperand& o = Bt.op[i];
        const int64_t blk = (int64_t)(blockIdx.x - Bt.first_block[i]);
        const T* x = (const T*)o.x;
        if (o.want_rows && o.want_cols) amax_tile<T, true, true>(x, o.rows, o.cols, o.ld, o.vec_ok != 0, o.amax_rm, o.amax_tr, blk);
        else if (o.want_rows) amax_tile<T, true, false>(x, o.rows, o.cols, o.ld, o.vec_ok != 0, o.amax_rm, o.amax_tr, blk);
        else if (o.want_cols) amax_tile<T, false, true>(x, o.rows, o.cols, o.ld, o.vec_ok != 0, o.amax_rm, o.amax_tr, blk);
        else amax_tile<T, false, false>(x, o.rows, o.cols, o.ld, o.vec_ok != 0, o.amax_rm, o.amax_tr, blk);
    }
    if (!last_cta_of_launch(Bt.counter)) return;
    for (int k = 0; k < Bt.n; ++k) scale_step(Bt.op[k].S, Bt.op[k].src_rm, Bt.op[k].src_tr);
}

template <typename T>
static void launch_amax(const void* x, int64_t rows, int64_t cols, int64_t ld, uint32_t* amax_rm, bool want_rows,
                        uint32_t* amax_tr, bool want_cols, const ScaleStep& S, cudaStream_t st) {
    const T* p = (const T*)x;
    constexpr int tile_c = 32 * AMAX_GROUPS * (16 / (int)sizeof(T));
    const unsigned grid = (unsigned)(((cols + tile_c - 1) / tile_c) * ((rows + AMAX_TILE_R - 1) / AMAX_TILE_R));
    const bool vec_ok = ((uintptr_t)x % 16 == 0) && ((ld * (int64_t)sizeof(T)) % 16 == 0);
    if (want_rows && want_cols) launch_pdl(amax_kernel<T, true, true>, dim3(grid), dim3(AMAX_THREADS), 0, st, p, rows, cols, ld, vec_ok, amax_rm, amax_tr, S);
    else if (want_rows) launch_pdl(amax_kernel<T, true, false>, dim3(grid), dim3(AMAX_THREADS), 0, st, p, rows, cols, ld, vec_ok, amax_rm, amax_tr, S);
    else if (want_cols) launch_pdl(amax_kernel<T, false, true>, dim3(grid), dim3(AMAX_THREADS), 0, st, p, rows, cols, ld, vec_ok, amax_rm, amax_tr, S);
    else launch_pdl(amax_kernel<T, false, false>, dim3(grid), dim3(AMAX_THREADS), 0, st, p, rows, cols, ld, vec_ok, amax_rm, amax_tr, S);
}

// ------------------------------------------------------------------------------------------
// step sizes
// ------------------------------------------------------------------------------------------
// The rm and tr arrays may be the same memory (per tensor, one group serves both layouts).
__global__ void scales_kernel(const uint32_t* amax_rm, int64_t n_rm, float* inv_rm, float* delta_rm,
                              const uint32_t* amax_tr, int64_t n_tr, float* inv_tr, float* delta_tr,
                              float qmax, uint32_t* status) {
    pdl_enter();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_rm) {
        float d, r;
        scale_from_bits(amax_rm[i], qmax, &d, &r, status);
        inv_rm[i] = r;
        if (delta_rm) delta_rm[i] = d;
    }
    if (i < n_tr) {
        float d, r;
        scale_from_bits(amax_tr[i], qmax, &d, &r, status);
        inv_tr[i] = r;
        if (delta_tr) delta_tr[i] = d;
    }
}

// ------------------------------------------------------------------------------------------
// quantizer
// ------------------------------------------------------------------------------------------
// Def. 1 for one element.
// The comparison frac(t) > eps of Def. 1 is taken on real numbers, with no rounding of the
// fractional part, in fixed point with 24 fractional bits.  Let S = t * 2^24 (exact: a power-of
// -two scaling of the binary32 product t = x * (1/D)), u = u24 the 24-bit threshold.
//   SR : for an integer L, L < S  <=>  L < ceil(S); with C = ceil(S) = f' 2^24 + low,
//        0 <= low < 2^24, the code is f' + (u < low) = (C + (2^24 - 1 - u)) >> 24.
//        (When S is not an integer and C is a multiple of 2^24, f' is floor(t) + 1 and
//        low = 0: the code is f' either way, as Def. 1 gives with frac(t) > 1 - 2^-24 > eps.)
//   RTN: frac(t) >= 1/2  <=>  floor(S) - floor(t) 2^24 >= 2^23, so the code is
//        (floor(S) + 2^23) >> 24.
// |t| <= qmax for every element of a group (the reciprocal step is rounded toward zero), so
// |C| <= qmax 2^24, the sum stays inside int32 and the code inside [-qmax, qmax] without a clamp.
// NOTTED: the threshold word arrives complemented (philox_rounds_not), which saves the NOT here.
// MODE: bit 0 = stochastic rounding (else round to nearest), bit 1 = E4M3 grid (else integer grid),
// bit 2 = stochastic rounding with 8 random bits per element (integer grid only; the thresholds are
// then handed to the same arithmetic as words (b << 24) | 2^23, whose top 24 bits are (2 b + 1) 2^15).
constexpr int MODE_SR = 1, MODE_E4M3 = 2, MODE_SR8 = 4;

// Integer grid: returns the 32-bit sum whose top byte is the code (two's complement).
template <int MODE, bool NOTTED = false>
__device__ __forceinline__ uint32_t quantize_sum(float x, float inv, uint32_t word) {
    const float s = __fmul_rn(__fmul_rn(x, inv), 16777216.0f);
    if constexpr ((MODE & MODE_SR) != 0) {
        const int c = __float2int_ru(s);
        uint32_t sum;   // (~word >> 8) + c = (2^24 - 1 - u24) + c in one multiply-add (high half)
        asm("mad.hi.u32 %0, %1, 16777216, %2;" : "=r"(sum) : "r"(NOTTED ? word : ~word), "r"((uint32_t)c));
        return sum;
    } else {
        return (uint32_t)__float2int_rd(s) + 0x00800000u;
    }
}

// E4M3 grid: Def. 1 with the step of the binade of t = x * (1/D): for 2^e <= |t| < 2^(e+1) (e >= -6;
// smaller |t| use e = -6, the subnormal spacing) the step is 2^(e-3) and u = t 2^(3-e) is rounded to
// an integer q in [-16, 16] by the same exact fixed-point rule as above.  With E = e + 127 the biased
// exponent of t, the code is sign | ((E - 120) << 3) + |q| - 8: |q| = 16 carries into the exponent
// field (next binade), |q| < 8 only occurs for E = 121 and gives the subnormal codes, q = 0 gives +0.
// Returns the code in the low byte.
template <int MODE, bool NOTTED = false>
__device__ __forceinline__ uint32_t quantize_e4m3(float x, float inv, uint32_t word, uint32_t sh) {
    // sh = 3 - k for the E4Mk grid (k mantissa bits; 0 for E4M3 itself): the step of binade e is
    // 2^(e-k), q counts those steps, and q << sh is the same value in the E4M3 code's units of 2^(e-3)
    const float t = __fmul_rn(x, inv);
    const uint32_t E = max((__float_as_uint(t) >> 23) & 0xFFu, 121u);          // |t| <= 448: E <= 135
    const float s = __fmul_rn(t, __uint_as_float((281u - sh - E) << 23));       // t 2^(k-e) 2^24, exact
    uint32_t sum;
    if constexpr ((MODE & MODE_SR) != 0) {
        const int c = __float2int_ru(s);
        asm("mad.hi.u32 %0, %1, 16777216, %2;" : "=r"(sum) : "r"(NOTTED ? word : ~word), "r"((uint32_t)c));
    } else {
        sum = (uint32_t)__float2int_rd(s) + 0x00800000u;
    }
    const int q = (int)sum >> 24;
    return ((uint32_t)q & 0x80u) | ((E << 3) + ((uint32_t)abs(q) << sh) - 968u);
}

// 8-random-bit mode: the threshold words of four consecutive elements from the stream word that holds
// their four bytes.
__device__ __forceinline__ void sr8_words(uint32_t w, uint32_t rnd[4]) {
    rnd[0] = __byte_perm(w, 0x00800000u, 0x0644); rnd[1] = __byte_perm(w, 0x00800000u, 0x1644);
    rnd[2] = __byte_perm(w, 0x00800000u, 0x2644); rnd[3] = __byte_perm(w, 0x00800000u, 0x3644);
}

// Four codes packed into one word, first element in the low byte.
template <int MODE, bool NOTTED = false>
__device__ __forceinline__ uint32_t quantize4(const float v[4], float i0, float i1, float i2, float i3,
                                              const uint32_t rnd[4], uint32_t sh) {
    if constexpr ((MODE & MODE_SR8) != 0) {
        return quantize4<MODE_SR>(v, i0, i1, i2, i3, rnd, sh);
    } else if constexpr ((MODE & MODE_E4M3) != 0) {
        const uint32_t c0 = quantize_e4m3<MODE, NOTTED>(v[0], i0, rnd[0], sh), c1 = quantize_e4m3<MODE, NOTTED>(v[1], i1, rnd[1], sh);
        const uint32_t c2 = quantize_e4m3<MODE, NOTTED>(v[2], i2, rnd[2], sh), c3 = quantize_e4m3<MODE, NOTTED>(v[3], i3, rnd[3], sh);
        return __byte_perm(__byte_perm(c0, c1, 0x0040), __byte_perm(c2, c3, 0x0040), 0x5410);
    } else {
        const uint32_t s0 = quantize_sum<MODE, NOTTED>(v[0], i0, rnd[0]), s1 = quantize_sum<MODE, NOTTED>(v[1], i1, rnd[1]);
        const uint32_t s2 = quantize_sum<MODE, NOTTED>(v[2], i2, rnd[2]), s3 = quantize_sum<MODE, NOTTED>(v[3], i3, rnd[3]);
        return __byte_perm(__byte_perm(s0, s1, 0x0073), __byte_perm(s2, s3, 0x0073), 0x5410);   // top bytes
    }
}

// Same with the mode chosen at run time (general path).
__device__ __forceinline__ uint32_t quantize4_rt(int mode, const float v[4], float i0, float i1, float i2, float i3,
                                                 const uint32_t rnd[4], uint32_t sh) {
    switch (mode) {
        case 0: return quantize4<0>(v, i0, i1, i2, i3, rnd, sh);
        case 1: return quantize4<1>(v, i0, i1, i2, i3, rnd, sh);
        case 2: return quantize4<2>(v, i0, i1, i2, i3, rnd, sh);
        case 3: return quantize4<3>(v, i0, i1, i2, i3, rnd, sh);
        default: return quantize4<MODE_SR>(v, i0, i1, i2, i3, rnd, sh);      // MODE_SR8: thresholds already in word form
    }
}

// 4x4 byte transpose: w[i] holds columns c..c+3 of row i -> o[e] holds rows 0..3 of column c+e
__device__ __forceinline__ void transpose4x4(const uint32_t w[4], uint32_t o[4]) {
    const uint32_t lo01 = __byte_perm(w[0], w[1], 0x5140), hi01 = __byte_perm(w[0], w[1], 0x7362);
    const uint32_t lo23 = __byte_perm(w[2], w[3], 0x5140), hi23 = __byte_perm(w[2], w[3], 0x7362);
    o[0] = __byte_perm(lo01, lo23, 0x5410); o[1] = __byte_perm(lo01, lo23, 0x7632);
    o[2] = __byte_perm(hi01, hi23, 0x5410); o[3] = __byte_perm(hi01, hi23, 0x7632);
}

constexpr int Q_THREADS = 256;
constexpr int Q_TILE = 128;          // 128 x 128 elements per CTA

struct QuantParams {
    int64_t rows, cols, ld;
    uint64_t index_offset;
    PhiloxKeys keys;
    int sr;                       // 1 = SR, 0 = RTN
    int mode;                     // MODE_SR | MODE_E4M3
    uint32_t e4m_shift;           // E4Mk grid: 3 - k (0 for E4M3 and for the integer grid)
    int per_row;                  // step size per row of each layout
    int8_t* codes_rm; int64_t ld_rm;
    int8_t* codes_tr; int64_t ld_tr;
    const float* inv_rm;          // [1] or [rows]
    const float* inv_tr;          // [1] or [cols]
    int vec_in;                   // 4-element vector loads allowed
    int vec_rm, vec_tr;           // 4-byte code stores allowed
    int vec_tr16;                 // 16-byte stores of the transposed layout allowed
};

// Row-wise read of the transposed tile and its stores: one warp per tile column, lane = row quad.
// Only the row quads [quad_lo, quad_hi) of the tile have been written (a CTA that took a slice of the tile).
__device__ __forceinline__ void store_transposed_tile(const uint32_t* tileT, const QuantParams& P, int64_t r0, int64_t c0,
                                                      int warp, int lane, int quad_lo = 0, int quad_hi = 32) {
    const int64_t r = r0 + lane * 4;
    if (lane < quad_lo || lane >= quad_hi) return;
#pragma unroll 4
    for (int col = warp; col < Q_TILE; col += 8) {
        const int64_t cc = c0 + col;
        if (cc >= P.cols || r >= P.rows) continue;
        const uint32_t w = tileT[col * 32 + (lane ^ ((col >> 2) & 31))];
        int8_t* dst = P.codes_tr + cc * P.ld_tr + r;
        if (P.vec_tr && r + 4 <= P.rows) {
            *reinterpret_cast<uint32_t*>(dst) = w;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (r + e < P.rows) dst[e] = (int8_t)((w >> (8 * e)) & 0xFF);
        }
    }
}

// Raw 4-element group as loaded, and its widening to binary32.
template <typename T> struct Raw4;
template <> struct Raw4<float> { using type = float4; };
template <> struct Raw4<__nv_bfloat16> { using type = uint2; };

__device__ __forceinline__ void widen(const float4& q, float v[4]) { v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w; }
__device__ __forceinline__ void widen(const uint2& q, float v[4]) {
    v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xFFFF0000u);
    v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xFFFF0000u);
}

// Fast path: extents, pitches and index offset are multiples of 4, pointers are aligned, so every
// 4-element group is one vector load, one Philox block and one 4-byte store.  LAYOUT bit 0 = row-major
// codes wanted, bit 1 = transposed codes wanted.  The loads of the next row quad are issued before the
// current one is processed, which keeps two quads of loads in flight per thread.
// FULL: the 128 x 128 tile lies inside the matrix and its Philox block indices do not carry into the
// upper counter word, so rows need no bounds checks and the counter is one 32-bit multiply-add.
// TR16 (full tiles whose transposed layout allows 16-byte stores): a warp takes 16 consecutive rows
// instead of every eighth row quad, so that a thread ends up with 16 consecutive codes of each of
// its four columns, writes them to the shared tile as one 16-byte chunk and the tile leaves in
// 16-byte stores (a quarter of the instructions of the 4-byte path).
template <typename T, int MODE, int LAYOUT, bool PER_ROW, bool FULL, bool TR16>
__device__ __forceinline__ void quantize_tile(const T* __restrict__ x, const QuantParams& P, uint32_t* tileT,
                                              int64_t r0, int64_t c0) {
    using Raw = typename Raw4<T>::type;
    constexpr bool WANT_RM = (LAYOUT & 1) != 0, WANT_TR = (LAYOUT & 2) != 0;
    constexpr bool TWO_STEPS = WANT_TR && PER_ROW;     // transposed layout has its own step sizes
    constexpr bool SRM = (MODE & MODE_SR) != 0, SR8 = (MODE & MODE_SR8) != 0;
    constexpr bool NT = SRM && !SR8;                  // thresholds arrive complemented
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t c = c0 + lane * 4;
    const bool col_ok = FULL || c < P.cols;             // cols % 4 == 0: a group is all in or all out

    float ic[4] = {0.f, 0.f, 0.f, 0.f};
    if constexpr (TWO_STEPS) {
        if (col_ok) { const float4 t = *reinterpret_cast<const float4*>(P.inv_tr + c); ic[0] = t.x; ic[1] = t.y; ic[2] = t.z; ic[3] = t.w; }
    }
    const float inv_tensor = PER_ROW ? 0.0f : P.inv_rm[0];

    // element (tr, lane * 4) of the tile, tr = (warp + 8 * it) * 4 + i: 32-bit offsets from the tile corner
    const T* xt = x + r0 * P.ld + c;
    const uint32_t ld = (uint32_t)P.ld;
    int8_t* out_rm = WANT_RM ? P.codes_rm + r0 * P.ld_rm + c : nullptr;
    const uint32_t ld_rm = (uint32_t)P.ld_rm;
    // Philox block index of (row, c): (index_offset + row * cols + c) / 4 = jb + tr * j_row
    const uint64_t jb = (P.index_offset + (uint64_t)r0 * (uint64_t)P.cols + (uint64_t)c) >> 2;
    const uint32_t j_row = (uint32_t)((uint64_t)P.cols >> 2);
    const uint32_t jb_lo = (uint32_t)jb, jb_hi = (uint32_t)(jb >> 32);

    Raw cur[4], nxt[4];
    float inv_cur[4], inv_nxt[4];
    uint32_t tw[TR16 ? 4 : 1][4];                       // TR16: codes of 16 rows x 4 columns, one word per row quad
    auto load_quad = [&](int it, Raw raw[4], float inv_r[4]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t tr = (uint32_t)(TR16 ? warp * 4 + it : warp + 8 * it) * 4 + i;
            if (FULL || (col_ok && r0 + tr < P.rows)) {
                raw[i] = __ldcs(reinterpret_cast<const Raw*>(xt + tr * ld));
                if constexpr (PER_ROW && WANT_RM) inv_r[i] = P.inv_rm[r0 + tr];
            } else {
                raw[i] = Raw{};
                if constexpr (PER_ROW && WANT_RM) inv_r[i] = 0.0f;
            }
        }
    };
    load_quad(0, cur, inv_cur);

#pragma unroll
    for (int it = 0; it < 4; ++it) {
        if (it + 1 < 4) load_quad(it + 1, nxt, inv_nxt);
        const int rq = TR16 ? warp * 4 + it : warp + 8 * it;
        uint32_t wr[4], wt[4];
        uint32_t sw[4] = {0u, 0u, 0u, 0u};     // 8-bit mode: stream word of this thread's 4 elements, per row
        if constexpr (SR8) {
            // one Philox block covers 16 consecutive elements = the 4-element groups of 4 neighbouring
            // lanes.  Lane 4 g + j computes the block of row j of the quad; a 4 x 4 transpose over the four
            // lanes then gives each lane word j of the blocks of rows 0 .. 3.
            const int j4 = lane & 3;
            const uint64_t i16 = P.index_offset + (uint64_t)(r0 + rq * 4 + j4) * (uint64_t)P.cols + (uint64_t)(c0 + (lane >> 2) * 16);
            philox_rounds((uint32_t)(i16 >> 4), (uint32_t)(i16 >> 36), P.keys, sw);
            {
                const bool hi = (j4 & 2) != 0;
                const uint32_t r0w = __shfl_xor_sync(0xFFFFFFFFu, hi ? sw[0] : sw[2], 2);
                const uint32_t r1w = __shfl_xor_sync(0xFFFFFFFFu, hi ? sw[1] : sw[3], 2);
                if (hi) { sw[0] = r0w; sw[1] = r1w; } else { sw[2] = r0w; sw[3] = r1w; }
            }
            {
                const bool odd = (j4 & 1) != 0;
                const uint32_t r0w = __shfl_xor_sync(0xFFFFFFFFu, odd ? sw[0] : sw[1], 1);
                const uint32_t r1w = __shfl_xor_sync(0xFFFFFFFFu, odd ? sw[2] : sw[3], 1);
                if (odd) { sw[0] = r0w; sw[2] = r1w; } else { sw[1] = r0w; sw[3] = r1w; }
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint32_t tr = (uint32_t)rq * 4 + i;
            float v[4];
            widen(cur[i], v);
            uint32_t rnd[4] = {0u, 0u, 0u, 0u};
            if constexpr (SR8) sr8_words(sw[i], rnd);
            if constexpr (SRM) {
                if constexpr (FULL) {
                    philox_rounds_not(jb_lo + tr * j_row, jb_hi, P.keys, rnd);
                } else {
                    const uint64_t jj = jb + (uint64_t)tr * j_row;
                    philox_rounds_not((uint32_t)jj, (uint32_t)(jj >> 32), P.keys, rnd);
                }
            }
            if constexpr (WANT_RM || !TWO_STEPS) {
                const float ir = (PER_ROW && WANT_RM) ? inv_cur[i] : inv_tensor;
                wr[i] = quantize4<MODE, NT>(v, ir, ir, ir, ir, rnd, P.e4m_shift);
            }
            if constexpr (TWO_STEPS) wt[i] = quantize4<MODE, NT>(v, ic[0], ic[1], ic[2], ic[3], rnd, P.e4m_shift);
            else wt[i] = wr[i];
            if constexpr (WANT_RM) {
                if (FULL || (col_ok && r0 + tr < P.rows)) *reinterpret_cast<uint32_t*>(out_rm + tr * ld_rm) = wr[i];
            }
        }
        if constexpr (WANT_TR) {
            uint32_t o[4];
            transpose4x4(wt, o);
            if constexpr (TR16) {
#pragma unroll
                for (int e = 0; e < 4; ++e) tw[e][it] = o[e];
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) tileT[(lane * 4 + e) * 32 + (rq ^ lane)] = o[e];
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) { cur[i] = nxt[i]; inv_cur[i] = inv_nxt[i]; }
    }
    if constexpr (WANT_TR && TR16) {
        // column col of the tile is a 128-byte row of tileT; rows 16 w .. 16 w + 15 (warp w) are its 16-byte
        // chunk w, stored at chunk position w ^ ((col >> 2) & 7) so that a warp's stores spread over all banks
#pragma unroll
        for (int e = 0; e < 4; ++e)
            *reinterpret_cast<uint4*>(tileT + (lane * 4 + e) * 32 + ((warp ^ (lane & 7)) << 2)) =
                make_uint4(tw[e][0], tw[e][1], tw[e][2], tw[e][3]);
        __syncthreads();
        // a warp stores 16 columns, four per instruction: 8 lanes x 16 bytes = the 128 rows of one column
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const int col = warp * 16 + k * 4 + (lane >> 3);
            const int chunk = lane & 7;
            const uint4 v = *reinterpret_cast<const uint4*>(tileT + col * 32 + (chunk << 2));
            const int rows16 = chunk ^ ((col >> 2) & 7);           // which 16 rows this chunk holds
            *reinterpret_cast<uint4*>(P.codes_tr + (c0 + col) * P.ld_tr + r0 + rows16 * 16) = v;
        }
    } else if constexpr (WANT_TR) {
        __syncthreads();
        store_transposed_tile(tileT, P, r0, c0, warp, lane);
    }
}

template <typename T, int MODE, int LAYOUT, bool PER_ROW>
__global__ void __launch_bounds__(Q_THREADS)
quantize_fast_kernel(const T* __restrict__ x, const __grid_constant__ QuantParams P) {
    pdl_enter();
    __shared__ uint32_t tileT[(LAYOUT & 2) ? Q_TILE * (Q_TILE / 4) : 1];
    const int64_t n_tc = (P.cols + Q_TILE - 1) / Q_TILE;
    const int64_t c0 = ((int64_t)blockIdx.x % n_tc) * Q_TILE;
    const int64_t r0 = ((int64_t)blockIdx.x / n_tc) * Q_TILE;
    // last Philox block index of the tile, relative to its first: no carry if it fits in the low word
    const uint64_t j_first = (P.index_offset + (uint64_t)r0 * (uint64_t)P.cols + (uint64_t)c0) >> 2;
    const uint64_t j_span = (uint64_t)(Q_TILE - 1) * ((uint64_t)P.cols >> 2) + (Q_TILE / 4 - 1);
    const bool full = r0 + Q_TILE <= P.rows && c0 + Q_TILE <= P.cols && (j_first & 0xFFFFFFFFull) + j_span <= 0xFFFFFFFFull;
    if constexpr ((LAYOUT & 2) != 0) {
        if (full && P.vec_tr16) { quantize_tile<T, MODE, LAYOUT, PER_ROW, true, true>(x, P, tileT, r0, c0); return; }
    }
    if (full) quantize_tile<T, MODE, LAYOUT, PER_ROW, true, false>(x, P, tileT, r0, c0);
    else quantize_tile<T, MODE, LAYOUT, PER_ROW, false, false>(x, P, tileT, r0, c0);
}

// Per-row step sizes, row-major codes only: absmax and quantizer in ONE pass over the input.  A CTA
// takes whole rows; each thread holds its 4-element groups of the row in registers (G per thread,
// groups tid, tid + 256, ...), the row maximum is reduced over the CTA (two barriers per row), the
// step size is derived exactly as in the two-pass path, and the codes are formed from the registers,
// so that the input is read once (e + 1 bytes per element instead of 2 e + 1).  Several CTAs per SM
// hide one another's load latency (holding the next row in registers as well cost more in occupancy
// than it gained).  Same conditions as the fast path (groups of four line up with the flat index),
// same arithmetic, same codes.
__device__ __forceinline__ uint32_t abs_max4(const float4& q) {
    return max(max(__float_as_uint(q.x) & 0x7FFFFFFFu, __float_as_uint(q.y) & 0x7FFFFFFFu),
               max(__float_as_uint(q.z) & 0x7FFFFFFFu, __float_as_uint(q.w) & 0x7FFFFFFFu));
}
__device__ __forceinline__ uint32_t abs_max4(const uint2& q) {      // four bfloat16: packed 16-bit maxima, widened
    const uint32_t m = __vmaxu2(q.x & 0x7FFF7FFFu, q.y & 0x7FFF7FFFu);
    return max(m << 16, m & 0xFFFF0000u);
}

constexpr int ROWQ_MAX_G = 8;          // rows of up to 256 * 8 * 4 = 8192 elements

template <typename T, int MODE, int G>
__global__ void __launch_bounds__(Q_THREADS)
quantize_rows_kernel(const T* __restrict__ x, const __grid_constant__ QuantParams P, float* __restrict__ delta_out,
                     float qmax, uint32_t* status) {
    pdl_enter();
    using Raw = typename Raw4<T>::type;
    constexpr bool SRM = (MODE & MODE_SR) != 0;
    __shared__ uint32_t warp_max[2][Q_THREADS / 32];
    __shared__ float row_inv[2];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t ngroups = (uint32_t)(P.cols >> 2);
    Raw cur[G];
    auto load_row = [&](int64_t r, Raw raw[G]) {
        const Raw* src = reinterpret_cast<const Raw*>(x + r * P.ld);
#pragma unroll
        for (int k = 0; k < G; ++k) {
            const uint32_t g = (uint32_t)tid + (uint32_t)(k * Q_THREADS);
            raw[k] = g < ngroups ? __ldcs(src + g) : Raw{};
        }
    };
    int64_t r = blockIdx.x;
    for (uint32_t it = 0; r < P.rows; r += gridDim.x, ++it) {
        load_row(r, cur);
        uint32_t m = 0u;
#pragma unroll
        for (int k = 0; k < G; ++k) m = max(m, abs_max4(cur[k]));
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        if (lane == 0) warp_max[it & 1][warp] = m;
        __syncthreads();
        // one warp turns the row maximum into the step size (three divisions, done once per row instead
        // of once per warp); both shared slots alternate between rows, and the two barriers of the
        // following row separate every write from the last read of the same slot
        if (warp == 0) {
            uint32_t bits = lane < Q_THREADS / 32 ? warp_max[it & 1][lane] : 0u;
            bits = __reduce_max_sync(0xFFFFFFFFu, bits);
            if (lane == 0) {
                float delta, r_inv;
                scale_from_bits(bits, qmax, &delta, &r_inv, status);
                row_inv[it & 1] = r_inv;
                if (delta_out) delta_out[r] = delta;
            }
        }
        __syncthreads();
        const float inv = row_inv[it & 1];
        const uint64_t jb = (P.index_offset + (uint64_t)r * (uint64_t)P.cols) >> 2;     // block of the row's first group
        uint32_t* out = reinterpret_cast<uint32_t*>(P.codes_rm + r * P.ld_rm);
        // all G groups are computed without branches (groups past the row hold zeros), so that their
        // Philox chains interleave; only the stores are predicated
        uint32_t w[G];
#pragma unroll
        for (int k = 0; k < G; ++k) {
            const uint32_t g = (uint32_t)tid + (uint32_t)(k * Q_THREADS);
            float v[4];
            widen(cur[k], v);
            uint32_t rnd[4] = {0u, 0u, 0u, 0u};
            if constexpr (SRM) {
                const uint32_t lo = (uint32_t)jb + g;
                philox_rounds_not(lo, (uint32_t)(jb >> 32) + (lo < g ? 1u : 0u), P.keys, rnd);
            }
            w[k] = quantize4<MODE, SRM>(v, inv, inv, inv, inv, rnd, P.e4m_shift);
        }
#pragma unroll
        for (int k = 0; k < G; ++k) {
            const uint32_t g = (uint32_t)tid + (uint32_t)(k * Q_THREADS);
            if (g < ngroups) out[g] = w[k];
        }
    }
}

// The same one-pass scheme with a WARP per row, for rows short enough that a lane can hold its share
// in registers (GW groups of four elements per lane, groups lane, lane + 32, ...): no barriers at all,
// the row maximum is one warp reduction and every lane derives the step size itself, so the warps of
// an SM run independently and hide one another's load latency.
template <typename T, int MODE, int GW>
__global__ void __launch_bounds__(Q_THREADS)
quantize_rows_warp_kernel(const T* __restrict__ x, const __grid_constant__ QuantParams P, float* __restrict__ delta_out,
                          float qmax, uint32_t* status) {
    pdl_enter();
    using Raw = typename Raw4<T>::type;
    constexpr bool SRM = (MODE & MODE_SR) != 0;
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (Q_THREADS / 32);
    const uint32_t ngroups = (uint32_t)(P.cols >> 2);
    for (int64_t r = (int64_t)blockIdx.x * (Q_THREADS / 32) + (threadIdx.x >> 5); r < P.rows; r += warps) {
        const Raw* src = reinterpret_cast<const Raw*>(x + r * P.ld);
        Raw cur[GW];
#pragma unroll
        for (int k = 0; k < GW; ++k) {
            const uint32_t g = (uint32_t)lane + 32u * k;
            cur[k] = g < ngroups ? __ldcs(src + g) : Raw{};
        }
        uint32_t m = 0u;
#pragma unroll
        for (int k = 0; k < GW; ++k) m = max(m, abs_max4(cur[k]));
        m = __reduce_max_sync(0xFFFFFFFFu, m);
        float delta, inv;
        scale_from_bits(m, qmax, &delta, &inv, status);
        if (lane == 0 && delta_out) delta_out[r] = delta;
        const uint64_t jb = (P.index_offset + (uint64_t)r * (uint64_t)P.cols) >> 2;
        uint32_t* out = reinterpret_cast<uint32_t*>(P.codes_rm + r * P.ld_rm);
#pragma unroll
        for (int k = 0; k < GW; ++k) {
            const uint32_t g = (uint32_t)lane + 32u * k;
            float v[4];
            widen(cur[k], v);
            uint32_t rnd[4] = {0u, 0u, 0u, 0u};
            if constexpr (SRM) {
                const uint32_t lo = (uint32_t)jb + g;
                philox_rounds_not(lo, (uint32_t)(jb >> 32) + (lo < g ? 1u : 0u), P.keys, rnd);
            }
            const uint32_t w = quantize4<MODE, SRM>(v, inv, inv, inv, inv, rnd, P.e4m_shift);
            if (g < ngroups) out[g] = w;
        }
    }
}

template <typename T, int MODE, int GW>
static void launch_rows_warp_one(const T* p, const QuantParams& P, float* delta_out, float qmax, uint32_t* status,
                                 int sms, cudaStream_t st) {
    static std::atomic<int> cached{0};              // resident CTAs per SM, asked once (any thread may be first)
    int per_sm = cached.load(std::memory_order_relaxed);
    if (per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_rows_warp_kernel<T, MODE, GW>, Q_THREADS, 0) != cudaSuccess || n < 1) n = 1;
        cached.store(per_sm = n, std::memory_order_relaxed);
    }
    const int64_t resident = (int64_t)sms * per_sm;
    const int64_t need = (P.rows + Q_THREADS / 32 - 1) / (Q_THREADS / 32);
    launch_pdl(quantize_rows_warp_kernel<T, MODE, GW>, dim3((unsigned)(need < resident ? need : resident)), dim3(Q_THREADS), 0, st, p, P, delta_out, qmax, status);
}

// Groups per lane a warp may hold: 64 data registers at most.
template <typename T> constexpr int rows_warp_max_groups() { return sizeof(T) == 4 ? 16 : 32; }

template <typename T, int MODE>
static void launch_rows_warp_g(int gw, const void* x, const QuantParams& P, float* delta_out, float qmax, uint32_t* status,
                               int sms, cudaStream_t st) {
    const T* p = (const T*)x;
    if (gw <= 4) launch_rows_warp_one<T, MODE, 4>(p, P, delta_out, qmax, status, sms, st);
    else if (gw <= 8) launch_rows_warp_one<T, MODE, 8>(p, P, delta_out, qmax, status, sms, st);
    else if (gw <= 16) launch_rows_warp_one<T, MODE, 16>(p, P, delta_out, qmax, status, sms, st);
    else if constexpr (rows_warp_max_groups<T>() >= 32) launch_rows_warp_one<T, MODE, 32>(p, P, delta_out, qmax, status, sms, st);
}

// One wave of CTAs: as many as are resident at once (asked once per kernel), at most one per row.
template <typename T, int MODE, int G>
static void launch_rows_one(const T* p, const QuantParams& P, float* delta_out, float qmax, uint32_t* status,
                            int sms, cudaStream_t st) {
    static std::atomic<int> cached{0};
    int per_sm = cached.load(std::memory_order_relaxed);
    if (per_sm == 0) {
        int n = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, quantize_rows_kernel<T, MODE, G>, Q_THREADS, 0) != cudaSuccess || n < 1) n = 1;
        cached.store(per_sm = n, std::memory_order_relaxed);
    }
    const int64_t resident = (int64_t)sms * per_sm;
    const unsigned grid = (unsigned)(P.rows < resident ? P.rows : resident);
    launch_pdl(quantize_rows_kernel<T, MODE, G>, dim3(grid), dim3(Q_THREADS), 0, st, p, P, delta_out, qmax, status);
}

template <typename T, int MODE>
static void launch_rows_g(int g, const void* x, const QuantParams& P, float* delta_out, float qmax, uint32_t* status,
                          int sms, cudaStream_t st) {
    const T* p = (const T*)x;
    if (g <= 1) launch_rows_one<T, MODE, 1>(p, P, delta_out, qmax, status, sms, st);
    else if (g <= 2) launch_rows_one<T, MODE, 2>(p, P, delta_out, qmax, status, sms, st);
    else if (g <= 4) launch_rows_one<T, MODE, 4>(p, P, delta_out, qmax, status, sms, st);
    else launch_rows_one<T, MODE, 8>(p, P, delta_out, qmax, status, sms, st);
}

static void launch_rows(srq_dtype_t dt, int mode, const void* x, const QuantParams& P, float* delta_out, float qmax,
                        uint32_t* status, int sms, cudaStream_t st) {
    const int g = (int)(((P.cols >> 2) + Q_THREADS - 1) / Q_THREADS);
    const int gw = (int)(((P.cols >> 2) + 31) / 32);          // groups per lane with a warp per row
#define SRQ_ROWS_WARP(T)                                                                          \
    switch (mode) {                                                                               \
        case 0: launch_rows_warp_g<T, 0>(gw, x, P, delta_out, qmax, status, sms, st); break;      \
        case 1: launch_rows_warp_g<T, 1>(gw, x, P, delta_out, qmax, status, sms, st); break;      \
        case 2: launch_rows_warp_g<T, 2>(gw, x, P, delta_out, qmax, status, sms, st); break;      \
        default: launch_rows_warp_g<T, 3>(gw, x, P, delta_out, qmax, status, sms, st); break;     \
    }
    if (dt == SRQ_F32 && gw <= rows_warp_max_groups<float>()) { SRQ_ROWS_WARP(float) return; }
    if (dt != SRQ_F32 && gw <= rows_warp_max_groups<__nv_bfloat16>()) { SRQ_ROWS_WARP(__nv_bfloat16) return; }
#undef SRQ_ROWS_WARP
#define SRQ_ROWS(T)                                                                          \
    switch (mode) {                                                                          \
        case 0: launch_rows_g<T, 0>(g, x, P, delta_out, qmax, status, sms, st);  break;      \
        case 1: launch_rows_g<T, 1>(g, x, P, delta_out, qmax, status, sms, st);  break;      \
        case 2: launch_rows_g<T, 2>(g, x, P, delta_out, qmax, status, sms, st);  break;      \
        default: launch_rows_g<T, 3>(g, x, P, delta_out, qmax, status, sms, st);  break;     \
    }
    if (dt == SRQ_F32) { SRQ_ROWS(float) } else { SRQ_ROWS(__nv_bfloat16) }
#undef SRQ_ROWS
}

// General path: any extent, pitch, alignment and index offset; one Philox block per element
// when the groups of four do not line up with the flat index.  Same results as the fast path.
template <typename T>
__device__ __forceinline__ void quantize_general_tile(const T* __restrict__ x, const QuantParams& P, uint32_t* tileT, int64_t blk,
                                                      int it_lo = 0, int it_hi = 4) {     // 32-row slices of the tile this CTA takes
    // transposed tile: column c of the tile holds 128 row codes = 32 words; the word index is
    // XOR-ed with (c >> 2) & 31 so that both the column-wise writes and the row-wise reads
    // touch 32 different banks.
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_tc = (P.cols + Q_TILE - 1) / Q_TILE;
    const int64_t c0 = (blk % n_tc) * Q_TILE;
    const int64_t r0 = (blk / n_tc) * Q_TILE;
    const int64_t c = c0 + lane * 4;
    const bool want_rm = P.codes_rm != nullptr, want_tr = P.codes_tr != nullptr;
    const bool sr = P.sr != 0;
    const bool two_steps = want_tr && P.per_row;   // transposed layout has its own step sizes

    float inv_c[4] = {0.f, 0.f, 0.f, 0.f};
    if (two_steps) {
#pragma unroll
        for (int e = 0; e < 4; ++e) if (c + e < P.cols) inv_c[e] = P.inv_tr[c + e];
    }
    const float inv_tensor = P.per_row ? 0.0f : P.inv_rm[0];

    // the next row quad is requested before the current one is used, so that a tile costs about one
    // memory round trip instead of four (small inputs are a chain of latencies, not a stream); the loop
    // itself stays rolled, because the kernel's code must stay small for the same reason
    float cur[4][4], nxt[4][4];
    auto load_quad = [&](int it, float (&q)[4][4]) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t r = r0 + (warp + 8 * it) * 4 + i;
            if (r < P.rows && c < P.cols) load4(x + r * P.ld, c, P.cols, P.vec_in != 0, q[i]);
            else q[i][0] = q[i][1] = q[i][2] = q[i][3] = 0.0f;
        }
    };
    load_quad(it_lo, cur);

#pragma unroll 1
    for (int it = it_lo; it < it_hi; ++it) {
        if (it + 1 < it_hi) load_quad(it + 1, nxt);
        const int rq = warp + 8 * it;   // row quad of the tile
        uint32_t wr[4], wt[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t r = r0 + rq * 4 + i;
            wr[i] = 0u; wt[i] = 0u;
            if (r < P.rows && c < P.cols) {
                const float (&v)[4] = cur[i];
                uint32_t rnd[4] = {0u, 0u, 0u, 0u};
                if (sr || (P.mode & MODE_SR8)) {
                    const bool sr8 = (P.mode & MODE_SR8) != 0;        // 16 elements per block, one byte each
                    const uint64_t i0 = P.index_offset + (uint64_t)r * (uint64_t)P.cols + (uint64_t)c;
                    if (!sr8 && (i0 & 3u) == 0) {                     // the four elements share one block
                        const uint64_t jb = i0 >> 2;
                        philox_rounds((uint32_t)jb, (uint32_t)(jb >> 32), P.keys, rnd);
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint64_t ie = i0 + e, jb = sr8 ? ie >> 4 : ie >> 2;
                            uint32_t o[4];
                            philox_rounds((uint32_t)jb, (uint32_t)(jb >> 32), P.keys, o);
                            const uint32_t s = sr8 ? (uint32_t)(ie >> 2) & 3u : (uint32_t)ie & 3u;
                            const uint32_t w = s == 0 ? o[0] : s == 1 ? o[1] : s == 2 ? o[2] : o[3];
                            rnd[e] = sr8 ? ((((w >> (8 * ((uint32_t)ie & 3u))) & 0xFFu) << 24) | 0x00800000u) : w;
                        }
                    }
                }
                const float inv_r = P.per_row ? P.inv_rm[want_rm ? r : 0] : inv_tensor;
                if (want_rm || !two_steps)
                    wr[i] = quantize4_rt(P.mode, v, inv_r, inv_r, inv_r, inv_r, rnd, P.e4m_shift);
                if (two_steps)
                    wt[i] = quantize4_rt(P.mode, v, inv_c[0], inv_c[1], inv_c[2], inv_c[3], rnd, P.e4m_shift);
                else
                    wt[i] = wr[i];
                if (want_rm) {
                    int8_t* dst = P.codes_rm + r * P.ld_rm + c;
                    if (P.vec_rm && c + 4 <= P.cols) {
                        *reinterpret_cast<uint32_t*>(dst) = wr[i];
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (c + e < P.cols) dst[e] = (int8_t)((wr[i] >> (8 * e)) & 0xFF);
                    }
                }
            }
        }
        if (want_tr) {
            uint32_t o[4];
            transpose4x4(wt, o);
#pragma unroll
            for (int e = 0; e < 4; ++e) tileT[(lane * 4 + e) * 32 + (rq ^ lane)] = o[e];
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) cur[i][e] = nxt[i][e];
    }
    if (!want_tr) return;
    __syncthreads();
    store_transposed_tile(tileT, P, r0, c0, warp, lane, 8 * it_lo, 8 * it_hi);
}

template <typename T>
__global__ void __launch_bounds__(Q_THREADS)
quantize_kernel(const T* __restrict__ x, const QuantParams P) {
    pdl_enter();
    __shared__ uint32_t tileT[Q_TILE * (Q_TILE / 4)];
    quantize_general_tile<T>(x, P, tileT, (int64_t)blockIdx.x);
}

// The operands of one layer call in ONE launch (small problems): CTAs [first_block[i], first_block[i + 1])
// take the tiles of operand i.  The general path's arithmetic, so any extents and alignments; same codes.
struct QuantBatch {
    QuantParams P[BATCH_MAX];
    const void* x[BATCH_MAX];
    uint32_t first_block[BATCH_MAX + 1];
    int32_t n;
    int32_t slices;          // CTAs per 128 x 128 tile (1, 2 or 4): tiny batches are spread over more SMs
};

template <typename T>
__global__ void __launch_bounds__(Q_THREADS)
quantize_batch_kernel(const __grid_constant__ QuantBatch Bt) {
    pdl_enter();
    __shared__ uint32_t tileT[Q_TILE * (Q_TILE / 4)];
    int i = 0;
    while (i + 1 < Bt.n && blockIdx.x >= Bt.first_block[i + 1]) ++i;
    const uint32_t local = blockIdx.x - Bt.first_block[i];
    const int per = 4 / Bt.slices, it_lo = (int)(local % (uint32_t)Bt.slices) * per;
    quantize_general_tile<T>((const T*)Bt.x[i], Bt.P[i], tileT, (int64_t)(local / (uint32_t)Bt.slices), it_lo, it_lo + per);
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
template <typename T, int MODE, int LAYOUT>
static void launch_fast_pr(bool per_row, const void* x, const QuantParams& P, unsigned grid, cudaStream_t st) {
    if (per_row) launch_pdl(quantize_fast_kernel<T, MODE, LAYOUT, true>, dim3(grid), dim3(Q_THREADS), 0, st, (const T*)x, P);
    else launch_pdl(quantize_fast_kernel<T, MODE, LAYOUT, false>, dim3(grid), dim3(Q_THREADS), 0, st, (const T*)x, P);
}
template <typename T, int MODE>
static void launch_fast_layout(int layout, bool per_row, const void* x, const QuantParams& P, unsigned grid, cudaStream_t st) {
    if (layout == 1) launch_fast_pr<T, MODE, 1>(per_row, x, P, grid, st);
    else if (layout == 2) launch_fast_pr<T, MODE, 2>(per_row, x, P, grid, st);
    else launch_fast_pr<T, MODE, 3>(per_row, x, P, grid, st);
}
template <typename T>
static void launch_fast_mode(int mode, int layout, bool per_row, const void* x, const QuantParams& P, unsigned grid, cudaStream_t st) {
    switch (mode) {
        case 0: launch_fast_layout<T, 0>(layout, per_row, x, P, grid, st); break;
        case 1: launch_fast_layout<T, 1>(layout, per_row, x, P, grid, st); break;
        case 2: launch_fast_layout<T, 2>(layout, per_row, x, P, grid, st); break;
        case 3: launch_fast_layout<T, 3>(layout, per_row, x, P, grid, st); break;
        default: launch_fast_layout<T, MODE_SR8>(layout, per_row, x, P, grid, st); break;
    }
}
static void launch_fast(srq_dtype_t dt, int mode, int layout, bool per_row, const void* x, const QuantParams& P, unsigned grid,
                        cudaStream_t st) {
    if (dt == SRQ_F32) launch_fast_mode<float>(mode, layout, per_row, x, P, grid, st);
    else launch_fast_mode<__nv_bfloat16>(mode, layout, per_row, x, P, grid, st);
}

// int8 codes [rows, cols] -> the same integers as bfloat16 (exact: |code| <= 127), for the product
// of unquantized bfloat16 activations with a quantized weight.  Also writes 1.0f to *one.
__global__ void widen_codes_kernel(const int8_t* __restrict__ codes, int64_t rows, int64_t cols, int64_t ld,
                                   uint16_t* __restrict__ out, int64_t ld_out, float* one) {
    pdl_enter();
    if (blockIdx.x == 0 && threadIdx.x == 0) *one = 1.0f;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < rows * cols; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = i / cols, c = i % cols;
        out[r * ld_out + c] = (uint16_t)(__float_as_uint(__int2float_rn((int)codes[r * ld + c])) >> 16);
    }
}

cudaError_t launch_widen_codes(const int8_t* codes, int64_t rows, int64_t cols, int64_t ld, void* out_bf16, int64_t ld_out,
                               float* one, cudaStream_t stream) {
    const int64_t n = rows * cols;
    const unsigned grid = (unsigned)(n / 256 + 1 < 4096 ? n / 256 + 1 : 4096);
    launch_pdl(widen_codes_kernel, dim3(grid), dim3(256), 0, stream, codes, rows, cols, ld, (uint16_t*)out_bf16, ld_out, one);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_absmax(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* absmax, cudaStream_t stream) {
    cudaError_t e = cudaMemsetAsync(absmax, 0, sizeof(float), stream);
    if (e != cudaSuccess || rows == 0 || cols == 0) return e;
    const ScaleStep none = {};
    if (dt == SRQ_F32) launch_amax<float>(x, rows, cols, ld, (uint32_t*)absmax, false, nullptr, false, none, stream);
    else launch_amax<__nv_bfloat16>(x, rows, cols, ld, (uint32_t*)absmax, false, nullptr, false, none, stream);
    count_launch();
    return cudaGetLastError();
}

// Column maxima: absmax_cols[c] = max_r |x[r, c]| (binary32, written from zero).
cudaError_t launch_absmax_cols(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld, float* absmax_cols,
                               cudaStream_t stream) {
    if (cols == 0) return cudaSuccess;
    cudaError_t e = cudaMemsetAsync(absmax_cols, 0, (size_t)cols * sizeof(float), stream);
    if (e != cudaSuccess || rows == 0) return e;
    const ScaleStep none = {};
    if (dt == SRQ_F32) launch_amax<float>(x, rows, cols, ld, nullptr, false, (uint32_t*)absmax_cols, true, none, stream);
    else launch_amax<__nv_bfloat16>(x, rows, cols, ld, nullptr, false, (uint32_t*)absmax_cols, true, none, stream);
    count_launch();
    return cudaGetLastError();
}

// SM count of the current device (asked once per device).
static int sm_count() {
    static std::atomic<int> cached[64];             // zero-initialised; any thread may fill an entry
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        n = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// Everything launch_quantize derives from its arguments before it launches anything.
struct QuantPlan {
    QuantParams P;
    bool want_rm, want_tr, per_row, given, given_cols, fast, sr8, one_pass;
    int64_t n0, n1;               // groups whose step sizes are derived (row-major layout / transposed layout)
    float qmax;
    uint32_t* amax_rm; uint32_t* amax_tr;     // scratch words the absmax tiles write
    float* inv_rm; float* inv_tr;
};

static QuantPlan make_quant_plan(const QuantArgs& a, const QuantScratch& s) {
    QuantPlan pl;
    pl.want_rm = a.codes_rm != nullptr; pl.want_tr = a.codes_tr != nullptr;
    pl.per_row = a.q.scale == SRQ_PER_ROW;
    const bool want_rm = pl.want_rm, want_tr = pl.want_tr, per_row = pl.per_row;
    const int64_t rows = a.rows, cols = a.cols;
    const bool e4m3 = a.q.format == SRQ_GRID_E4M3;
    // E4Mk grid: bits = 5 + k; the largest value with k mantissa bits is 448 (k = 3, 2), 384 (k = 1), 256 (k = 0)
    const int mant = e4m3 ? a.q.bits - 5 : 3;
    pl.qmax = e4m3 ? (mant >= 2 ? 448.0f : (mant == 1 ? 384.0f : 256.0f)) : (float)((1 << (a.q.bits - 1)) - 1);
    const size_t esize = a.dt == SRQ_F32 ? 4 : 2;

    // group counts and where each layout's absmax lives; per tensor both layouts share word 0
    const int64_t n_rm = want_rm ? (per_row ? rows : 1) : 0;
    const int64_t n_tr = want_tr ? (per_row ? cols : 1) : 0;
    pl.amax_rm = s.amax_rm;
    pl.amax_tr = per_row ? s.amax_tr : s.amax_rm;
    pl.inv_rm = s.inv_rm;
    pl.inv_tr = per_row ? s.inv_tr : s.inv_rm;

    const bool vec_in = ((uintptr_t)a.x % (4 * esize) == 0) && (a.ld % 4 == 0);
    pl.given = a.q.absmax != nullptr && !per_row;   // per tensor: one known maximum for the whole operand
    // per row: known column maxima [cols] for the transposed layout (its groups run over the rows, i.e.
    // over the tokens, which other shards may hold); the row-major layout's row maxima are local
    pl.given_cols = a.q.absmax != nullptr && per_row && want_tr;
    // per tensor: one group feeds both layouts' scale outputs
    pl.n0 = per_row ? n_rm : 1;
    pl.n1 = per_row ? n_tr : ((want_tr && a.scale_tr) ? 1 : 0);

    QuantParams& P = pl.P;
    P.rows = rows; P.cols = cols; P.ld = a.ld;
    P.index_offset = a.q.index_offset;
    P.keys = make_philox_keys(a.q.seed, a.q.tensor_id);
    P.sr = a.q.round == SRQ_SR;
    pl.sr8 = a.q.round == SRQ_SR8;
    P.mode = pl.sr8 ? MODE_SR8 : ((P.sr ? MODE_SR : 0) | (e4m3 ? MODE_E4M3 : 0));
    P.e4m_shift = (uint32_t)(3 - mant);
    P.per_row = per_row;
    P.codes_rm = a.codes_rm; P.ld_rm = a.ld_rm;
    P.codes_tr = a.codes_tr; P.ld_tr = a.ld_tr;
    P.inv_rm = pl.inv_rm; P.inv_tr = pl.inv_tr;
    P.vec_in = vec_in;
    P.vec_rm = want_rm && ((uintptr_t)a.codes_rm % 4 == 0) && (a.ld_rm % 4 == 0);
    P.vec_tr = want_tr && ((uintptr_t)a.codes_tr % 4 == 0) && (a.ld_tr % 4 == 0);
    P.vec_tr16 = want_tr && ((uintptr_t)a.codes_tr % 16 == 0) && (a.ld_tr % 16 == 0);
    pl.fast = vec_in && (cols % 4 == 0) && (a.q.index_offset % 4 == 0) && (!pl.sr8 || (cols % 16 == 0 && a.q.index_offset % 16 == 0)) &&
              a.ld < (1 << 24) && a.ld_rm < (1 << 24) && (!want_rm || P.vec_rm) && (!want_tr || (P.vec_tr && rows % 4 == 0));
    // per-row steps and row-major codes only: one pass (rows of 512 .. 8192 elements)
    pl.one_pass = per_row && want_rm && !want_tr && pl.fast && !pl.sr8 && cols >= 512 && cols <= (int64_t)ROWQ_MAX_G * Q_THREADS * 4;
    return pl;
}

cudaError_t launch_quantize(const QuantArgs& a, const QuantScratch& s, uint32_t* status, cudaStream_t stream, bool scratch_zeroed) {
    const int64_t rows = a.rows, cols = a.cols;
    if (rows == 0 || cols == 0 || (!a.codes_rm && !a.codes_tr)) return cudaSuccess;
    const QuantPlan pl = make_quant_plan(a, s);
    const QuantParams& P = pl.P;
    const bool want_rm = pl.want_rm, want_tr = pl.want_tr, per_row = pl.per_row;
    const int64_t n0 = pl.n0, n1 = pl.n1;
    const float qmax = pl.qmax;
    uint32_t* amax_rm = pl.amax_rm;
    uint32_t* amax_tr = pl.amax_tr;
    float* inv_rm = pl.inv_rm;
    float* inv_tr = pl.inv_tr;

    if (pl.one_pass) {
        launch_rows(a.dt, P.mode, a.x, P, a.scale_rm, qmax, status, sm_count(), stream);
        count_launch();
        return cudaGetLastError();
    }

    if (pl.given_cols) {
        const int threads = 256;
        if (want_rm) {                                  // row maxima of this shard, then their step sizes
            if (!scratch_zeroed) {
                cudaError_t e = cudaMemsetAsync(s.counter, 0, (size_t)((char*)s.inv_rm - (char*)s.counter), stream);
                if (e != cudaSuccess) return e;
            }
            const ScaleStep none = {};
            if (a.dt == SRQ_F32) launch_amax<float>(a.x, rows, cols, a.ld, amax_rm, true, nullptr, false, none, stream);
            else launch_amax<__nv_bfloat16>(a.x, rows, cols, a.ld, amax_rm, true, nullptr, false, none, stream);
            count_launch();
        }
        const uint32_t* col_bits = (const uint32_t*)a.q.absmax;     // a non-negative float is its own bit pattern
        const int64_t n = n0 > n1 ? n0 : n1;
        launch_pdl(scales_kernel, dim3((unsigned)((n + threads - 1) / threads)), dim3(threads), 0, stream,
            amax_rm, n0, inv_rm, want_rm ? a.scale_rm : nullptr, col_bits, n1, inv_tr, a.scale_tr, qmax, status);
        count_launch();
    } else if (pl.given) {
        amax_rm = amax_tr = (uint32_t*)a.q.absmax;     // a non-negative float is its own bit pattern
        const int64_t n = n0 > n1 ? n0 : n1;
        const int threads = 256;
        launch_pdl(scales_kernel, dim3((unsigned)((n + threads - 1) / threads)), dim3(threads), 0, stream,
            amax_rm, n0, inv_rm, want_rm ? a.scale_rm : nullptr,
            amax_tr, n1, inv_tr, want_tr ? a.scale_tr : nullptr, qmax, status);
        count_launch();
    } else {
        if (!scratch_zeroed) {
            cudaError_t e = cudaMemsetAsync(s.counter, 0, (size_t)((char*)s.inv_rm - (char*)s.counter), stream);
            if (e != cudaSuccess) return e;
        }
        // absmax of every group; the last CTA to finish turns them into step sizes when there are few
        // (one CTA would take long over many thousands of groups: those get a launch of their own)
        const bool few = n0 + n1 <= 2048;
        const ScaleStep S = {few ? s.counter : nullptr, n0, inv_rm, want_rm ? a.scale_rm : nullptr,
                             n1, inv_tr, want_tr ? a.scale_tr : nullptr, qmax, status};
        const bool want_rows = per_row && want_rm, want_cols = per_row && want_tr;
        if (a.dt == SRQ_F32) launch_amax<float>(a.x, rows, cols, a.ld, amax_rm, want_rows, amax_tr, want_cols, S, stream);
        else launch_amax<__nv_bfloat16>(a.x, rows, cols, a.ld, amax_rm, want_rows, amax_tr, want_cols, S, stream);
        count_launch();
        if (!few) {
            const int64_t n = n0 > n1 ? n0 : n1;
            const int threads = 256;
            launch_pdl(scales_kernel, dim3((unsigned)((n + threads - 1) / threads)), dim3(threads), 0, stream,
                amax_rm, n0, inv_rm, want_rm ? a.scale_rm : nullptr,
                amax_tr, n1, inv_tr, want_tr ? a.scale_tr : nullptr, qmax, status);
            count_launch();
        }
    }
    {
        const unsigned grid = (unsigned)(((cols + Q_TILE - 1) / Q_TILE) * ((rows + Q_TILE - 1) / Q_TILE));
        if (pl.fast) launch_fast(a.dt, P.mode, (want_rm ? 1 : 0) | (want_tr ? 2 : 0), per_row, a.x, P, grid, stream);
        else if (a.dt == SRQ_F32) launch_pdl(quantize_kernel<float>, dim3(grid), dim3(Q_THREADS), 0, stream, (const float*)a.x, P);
        else launch_pdl(quantize_kernel<__nv_bfloat16>, dim3(grid), dim3(Q_THREADS), 0, stream, (const __nv_bfloat16*)a.x, P);
        count_launch();
    }
    return cudaGetLastError();
}

// The operands of one layer call.  Small problems (the launches, not the data, take the time) get two
// launches for all operands together, one for the maxima and step sizes, one for the codes; anything
// else, and anything the batched kernels do not cover, goes operand by operand.  Same results.
cudaError_t launch_quantize_batch(const QuantArgs* a, const QuantScratch* s, int n, uint32_t* status, cudaStream_t stream,
                                  bool scratch_zeroed) {
    // measured: below about four million elements per call the saved launches outweigh the general
    // kernel's lower speed; above, the specialised kernels win
    constexpr int64_t kBatchMaxElements = 1ll << 22, kBatchMaxGroups = 2048;
    int64_t elements = 0, groups = 0;
    bool ok = n >= 2 && n <= BATCH_MAX && scratch_zeroed;
    QuantPlan pl[BATCH_MAX];
    for (int i = 0; ok && i < n; ++i) {
        if (a[i].rows == 0 || a[i].cols == 0 || (!a[i].codes_rm && !a[i].codes_tr) || a[i].dt != a[0].dt) { ok = false; break; }
        pl[i] = make_quant_plan(a[i], s[i]);
        elements += a[i].rows * a[i].cols;
        groups += pl[i].n0 + pl[i].n1;
        if (a[i].ld >= (1ll << 31) || a[i].rows >= (1ll << 31)) ok = false;
    }
    if (!ok || elements > kBatchMaxElements || groups > kBatchMaxGroups) {
        for (int i = 0; i < n; ++i) {
            const cudaError_t e = launch_quantize(a[i], s[i], status, stream, scratch_zeroed);
            if (e != cudaSuccess) return e;
        }
        return cudaSuccess;
    }

    AmaxBatch ab = {};
    QuantBatch qb = {};
    ab.n = qb.n = n;
    {   // a handful of tiles would leave most SMs idle and each CTA with a long serial loop: slice the tiles
        int64_t tiles = 0;
        for (int i = 0; i < n; ++i) tiles += ((a[i].cols + Q_TILE - 1) / Q_TILE) * ((a[i].rows + Q_TILE - 1) / Q_TILE);
        const int sms = sm_count();
        qb.slices = tiles * 4 <= 8 * sms ? 4 : (tiles * 2 <= 8 * sms ? 2 : 1);
    }
    ab.counter = s[0].counter;                       // zeroed with the rest of the scratch
    uint32_t ablocks = 0, qblocks = 0;
    for (int i = 0; i < n; ++i) {
        const QuantArgs& A = a[i];
        const QuantPlan& p = pl[i];
        const size_t esize = A.dt == SRQ_F32 ? 4 : 2;
        AmaxOperand& o = ab.op[i];
        o.x = A.x; o.rows = A.rows; o.cols = A.cols; o.ld = A.ld;
        o.amax_rm = p.amax_rm; o.amax_tr = p.amax_tr;
        o.vec_ok = ((uintptr_t)A.x % 16 == 0) && ((A.ld * (int64_t)esize) % 16 == 0);
        // which maxima the tiles have to find, and which words the step sizes come from
        bool tiles = true;
        o.want_rows = p.per_row && p.want_rm; o.want_cols = p.per_row && p.want_tr;
        o.src_rm = p.amax_rm; o.src_tr = p.amax_tr;
        if (p.given) { tiles = false; o.src_rm = o.src_tr = (const uint32_t*)A.q.absmax; }
        else if (p.given_cols) { tiles = p.want_rm; o.want_cols = 0; o.src_tr = (const uint32_t*)A.q.absmax; }
        o.S = ScaleStep{nullptr, p.n0, p.inv_rm, p.want_rm ? A.scale_rm : nullptr, p.n1, p.inv_tr, p.want_tr ? A.scale_tr : nullptr, p.qmax, status};
        const int tile_c = 32 * AMAX_GROUPS * (16 / (int)esize);
        ab.first_block[i] = ablocks;
        if (tiles) ablocks += (uint32_t)(((A.cols + tile_c - 1) / tile_c) * ((A.rows + AMAX_TILE_R - 1) / AMAX_TILE_R));
        qb.P[i] = p.P; qb.x[i] = A.x;
        qb.first_block[i] = qblocks;
        qblocks += (uint32_t)(((A.cols + Q_TILE - 1) / Q_TILE) * ((A.rows + Q_TILE - 1) / Q_TILE)) * (uint32_t)qb.slices;
    }
    ab.first_block[n] = ablocks; qb.first_block[n] = qblocks;
    if (a[0].dt == SRQ_F32) launch_pdl(amax_batch_kernel<float>, dim3(ablocks ? ablocks : 1u), dim3(AMAX_THREADS), 0, stream, ab);
    else launch_pdl(amax_batch_kernel<__nv_bfloat16>, dim3(ablocks ? ablocks : 1u), dim3(AMAX_THREADS), 0, stream, ab);
    count_launch();
    if (a[0].dt == SRQ_F32) launch_pdl(quantize_batch_kernel<float>, dim3(qblocks), dim3(Q_THREADS), 0, stream, qb);
    else launch_pdl(quantize_batch_kernel<__nv_bfloat16>, dim3(qblocks), dim3(Q_THREADS), 0, stream, qb);
    count_launch();
    return cudaGetLastError();
}

}  // namespace srq
