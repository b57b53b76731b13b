// Absmax reduction, step sizes and the SR / RTN quantizer (Def. 1-3 of the paper).
//
// Three kernels per quantized tensor:
//   amax_kernel      one read of x; max |x| per tensor, per row and/or per column, kept as the
//                    binary32 bit pattern (non-negative floats order like unsigned integers,
//                    so atomicMax on the bits is exact and order independent)
//   scales_kernel    D = m / qmax and 1/D = qmax / m per group (one IEEE division each)
//   quantize_kernel  second read of x; t = x * (1/D), f = floor(t), p = t - f;
//                    SR: up iff u24 * 2^-24 < p with u24 from Philox4x32-10 keyed by
//                    (seed, tensor_id, flat index); RTN: up iff p >= 1/2; code = clamp(f + up).
//                    Writes the row-major code layout directly and the transposed layout
//                    through a swizzled shared-memory tile, so that both are stored with
//                    full 128-byte lines.
//
// Arithmetic that decides a code uses explicit round-to-nearest intrinsics so that the
// compiler cannot contract x * inv - f into a fused multiply-add.
#include <cuda_bf16.h>

#include "common.cuh"

namespace srq {

unsigned long long g_launches = 0;

// ------------------------------------------------------------------------------------------
// scratch carving
// ------------------------------------------------------------------------------------------
static inline size_t f32_block(int64_t n) { return align_up((size_t)n * 4); }

size_t quant_scratch_bytes(int64_t rows, int64_t cols) {
    return 2 * (f32_block(rows) + f32_block(cols));
}

QuantScratch carve_quant_scratch(void* base, int64_t rows, int64_t cols) {
    // amax blocks first and contiguous, so that one memset clears both
    char* p = (char*)base;
    QuantScratch s;
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
constexpr int AMAX_THREADS = 256;
constexpr int AMAX_TILE_C = 512;   // 32 lanes x 4 groups x 4 elements
constexpr int AMAX_TILE_R = 64;    // 8 warps x 8 rows

// what each layout needs: nothing, one word for the whole tensor, or one word per row (rm) / column (tr)
enum : int { AMAX_NONE = 0, AMAX_TENSOR = 1, AMAX_GROUPS = 2 };

template <typename T>
__global__ void __launch_bounds__(AMAX_THREADS)
amax_kernel(const T* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, bool vec_ok,
            uint32_t* __restrict__ amax_rm, int rm_mode, uint32_t* __restrict__ amax_tr, int tr_mode) {
    __shared__ uint32_t col_max[AMAX_TILE_C];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_tc = (cols + AMAX_TILE_C - 1) / AMAX_TILE_C;
    const int64_t c0 = ((int64_t)blockIdx.x % n_tc) * AMAX_TILE_C;
    const int64_t r0 = ((int64_t)blockIdx.x / n_tc) * AMAX_TILE_R;
    const bool want_cols = (tr_mode == AMAX_GROUPS);
    const bool want_rows = (rm_mode == AMAX_GROUPS);
    if (want_cols) {
        for (int i = threadIdx.x; i < AMAX_TILE_C; i += AMAX_THREADS) col_max[i] = 0u;
        __syncthreads();
    }
    uint32_t cm[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) cm[i] = 0u;
    uint32_t all = 0u;
    for (int rr = 0; rr < AMAX_TILE_R / 8; ++rr) {
        const int64_t r = r0 + warp + 8 * rr;
        if (r >= rows) break;
        const T* row = x + r * ld;
        uint32_t rmax = 0u;
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const int64_t c = c0 + (int64_t)(g * 32 + lane) * 4;
            if (c < cols) {
                float v[4];
                load4(row, c, cols, vec_ok, v);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint32_t b = abs_bits(v[e]);
                    rmax = max(rmax, b);
                    cm[g * 4 + e] = max(cm[g * 4 + e], b);
                }
            }
        }
        if (want_rows) {
            rmax = __reduce_max_sync(0xFFFFFFFFu, rmax);
            if (lane == 0 && rmax) atomicMax(&amax_rm[r], rmax);
        } else {
            all = max(all, rmax);
        }
    }
    if (rm_mode == AMAX_TENSOR) {
        all = __reduce_max_sync(0xFFFFFFFFu, all);
        if (lane == 0 && all) atomicMax(&amax_rm[0], all);
    }
    if (want_cols) {
#pragma unroll
        for (int g = 0; g < 4; ++g)
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (cm[g * 4 + e]) atomicMax(&col_max[(g * 32 + lane) * 4 + e], cm[g * 4 + e]);
        __syncthreads();
        for (int i = threadIdx.x; i < AMAX_TILE_C; i += AMAX_THREADS) {
            const int64_t c = c0 + i;
            if (c < cols && col_max[i]) atomicMax(&amax_tr[c], col_max[i]);
        }
    }
}

// ------------------------------------------------------------------------------------------
// step sizes
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void scale_from_bits(uint32_t bits, float qmax, float* delta, float* inv,
                                                uint32_t* status) {
    if (bits >= 0x7F800000u) record_status(status, SRQ_ERR_NONFINITE);
    const float m = __uint_as_float(bits);
    float r = (m == 0.0f) ? 0.0f : __fdiv_rn(qmax, m);
    if (!(fabsf(r) <= 3.402823466e38f)) r = 0.0f;   // overflowed reciprocal: treat the group as zero
    *inv = r;
    *delta = (r == 0.0f) ? 0.0f : __fdiv_rn(m, qmax);
}

// The rm and tr arrays may be the same memory (per tensor, one group serves both layouts).
__global__ void scales_kernel(const uint32_t* amax_rm, int64_t n_rm, float* inv_rm, float* delta_rm,
                              const uint32_t* amax_tr, int64_t n_tr, float* inv_tr, float* delta_tr,
                              float qmax, uint32_t* status) {
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
// Philox4x32-10 (Salmon et al., SC'11): ten rounds, two 32x32->64 multiplies per round
// ------------------------------------------------------------------------------------------
struct Philox {
    uint32_t k0[10], k1[10];   // round keys: key + r * Weyl constants (same for every thread)
};

__device__ __forceinline__ void philox_rounds(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t key0, uint32_t key1, uint32_t out[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t k0 = key0 + (uint32_t)r * 0x9E3779B9u;
        const uint32_t k1 = key1 + (uint32_t)r * 0xBB67AE85u;
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// ------------------------------------------------------------------------------------------
// quantizer
// ------------------------------------------------------------------------------------------
// Def. 1 for one element; returns the code as a small integer held in a float.
__device__ __forceinline__ float quantize_elem(float x, float inv, float qmax, bool sr, uint32_t word) {
    const float t = __fmul_rn(x, inv);
    const float f = floorf(t);
    const float p = __fsub_rn(t, f);
    bool up;
    if (sr) {
        // eps < p  <=>  u24 < p * 2^24 ; both sides exact in binary32
        up = __uint2float_rn(word >> 8) < __fmul_rn(p, 16777216.0f);
    } else {
        up = p >= 0.5f;
    }
    float q = up ? __fadd_rn(f, 1.0f) : f;
    return fminf(fmaxf(q, -qmax), qmax);
}

// Low byte of the two's complement integer held exactly in q (|q| <= 127).
__device__ __forceinline__ uint32_t code_bits(float q) { return __float_as_uint(__fadd_rn(q, 12582912.0f)); }

__device__ __forceinline__ uint32_t pack4(uint32_t b0, uint32_t b1, uint32_t b2, uint32_t b3) {
    return __byte_perm(__byte_perm(b0, b1, 0x0040), __byte_perm(b2, b3, 0x0040), 0x5410);
}

constexpr int Q_THREADS = 256;
constexpr int Q_TILE = 128;          // 128 x 128 elements per CTA

struct QuantParams {
    int64_t rows, cols, ld;
    uint64_t index_offset;
    uint32_t key0, key1, tid0, tid1;
    float qmax;
    int sr;                       // 1 = SR, 0 = RTN
    int per_row;                  // step size per row of each layout
    int8_t* codes_rm; int64_t ld_rm;
    int8_t* codes_tr; int64_t ld_tr;
    const float* inv_rm;          // [1] or [rows]
    const float* inv_tr;          // [1] or [cols]
    int vec_in;                   // 4-element vector loads allowed
    int vec_rm, vec_tr;           // 4-byte code stores allowed
};

template <typename T, bool ALIGNED>
__global__ void __launch_bounds__(Q_THREADS)
quantize_kernel(const T* __restrict__ x, const QuantParams P) {
    // transposed tile: column c of the tile holds 128 row codes = 32 words; the word index is
    // XOR-ed with (c >> 2) & 31 so that both the column-wise writes and the row-wise reads
    // touch 32 different banks.
    __shared__ uint32_t tileT[Q_TILE * (Q_TILE / 4)];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_tc = (P.cols + Q_TILE - 1) / Q_TILE;
    const int64_t c0 = ((int64_t)blockIdx.x % n_tc) * Q_TILE;
    const int64_t r0 = ((int64_t)blockIdx.x / n_tc) * Q_TILE;
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

#pragma unroll 1
    for (int it = 0; it < 4; ++it) {
        const int rq = warp + 8 * it;   // row quad of the tile
        uint32_t wr[4], wt[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t r = r0 + rq * 4 + i;
            wr[i] = 0u; wt[i] = 0u;
            if (r < P.rows && c < P.cols) {
                float v[4];
                load4(x + r * P.ld, c, P.cols, P.vec_in != 0, v);
                uint32_t rnd[4] = {0u, 0u, 0u, 0u};
                if (sr) {
                    const uint64_t i0 = P.index_offset + (uint64_t)r * (uint64_t)P.cols + (uint64_t)c;
                    if constexpr (ALIGNED) {
                        const uint64_t j = i0 >> 2;
                        philox_rounds((uint32_t)j, (uint32_t)(j >> 32), P.tid0, P.tid1, P.key0, P.key1, rnd);
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint64_t ie = i0 + e, j = ie >> 2;
                            uint32_t o[4];
                            philox_rounds((uint32_t)j, (uint32_t)(j >> 32), P.tid0, P.tid1, P.key0, P.key1, o);
                            const uint32_t s = (uint32_t)ie & 3u;
                            rnd[e] = s == 0 ? o[0] : s == 1 ? o[1] : s == 2 ? o[2] : o[3];
                        }
                    }
                }
                const float inv_r = P.per_row ? P.inv_rm[want_rm ? r : 0] : inv_tensor;
                if (want_rm || !two_steps) {
                    uint32_t b[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) b[e] = code_bits(quantize_elem(v[e], inv_r, P.qmax, sr, rnd[e]));
                    wr[i] = pack4(b[0], b[1], b[2], b[3]);
                }
                if (two_steps) {
                    uint32_t b[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) b[e] = code_bits(quantize_elem(v[e], inv_c[e], P.qmax, sr, rnd[e]));
                    wt[i] = pack4(b[0], b[1], b[2], b[3]);
                } else {
                    wt[i] = wr[i];
                }
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
            // 4x4 byte transpose: wt[i] holds columns c..c+3 of row i -> o[e] holds rows 0..3 of column c+e
            const uint32_t lo01 = __byte_perm(wt[0], wt[1], 0x5140), hi01 = __byte_perm(wt[0], wt[1], 0x7362);
            const uint32_t lo23 = __byte_perm(wt[2], wt[3], 0x5140), hi23 = __byte_perm(wt[2], wt[3], 0x7362);
            uint32_t o[4];
            o[0] = __byte_perm(lo01, lo23, 0x5410); o[1] = __byte_perm(lo01, lo23, 0x7632);
            o[2] = __byte_perm(hi01, hi23, 0x5410); o[3] = __byte_perm(hi01, hi23, 0x7632);
#pragma unroll
            for (int e = 0; e < 4; ++e) tileT[(lane * 4 + e) * 32 + (rq ^ lane)] = o[e];
        }
    }
    if (!want_tr) return;
    __syncthreads();
    // row-wise read of the transposed tile: one warp per tile column, lane = row quad
    const int64_t r = r0 + lane * 4;
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

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
cudaError_t launch_quantize(const QuantArgs& a, const QuantScratch& s, uint32_t* status, cudaStream_t stream) {
    const bool want_rm = a.codes_rm != nullptr, want_tr = a.codes_tr != nullptr;
    const bool per_row = a.q.scale == SRQ_PER_ROW;
    const int64_t rows = a.rows, cols = a.cols;
    if (rows == 0 || cols == 0 || (!want_rm && !want_tr)) return cudaSuccess;
    const float qmax = (float)((1 << (a.q.bits - 1)) - 1);
    const size_t esize = a.dt == SRQ_F32 ? 4 : 2;

    // group counts and where each layout's absmax lives; per tensor both layouts share word 0
    const int64_t n_rm = want_rm ? (per_row ? rows : 1) : 0;
    const int64_t n_tr = want_tr ? (per_row ? cols : 1) : 0;
    uint32_t* amax_rm = s.amax_rm;
    uint32_t* amax_tr = per_row ? s.amax_tr : s.amax_rm;
    float* inv_rm = s.inv_rm;
    float* inv_tr = per_row ? s.inv_tr : s.inv_rm;

    cudaError_t e = cudaMemsetAsync(s.amax_rm, 0, (size_t)((char*)s.inv_rm - (char*)s.amax_rm), stream);
    if (e != cudaSuccess) return e;

    const bool vec_in = ((uintptr_t)a.x % (4 * esize) == 0) && (a.ld % 4 == 0);
    {
        const unsigned grid = (unsigned)(((cols + AMAX_TILE_C - 1) / AMAX_TILE_C) * ((rows + AMAX_TILE_R - 1) / AMAX_TILE_R));
        const int rm_mode = per_row ? (want_rm ? AMAX_GROUPS : AMAX_NONE) : AMAX_TENSOR;
        const int tr_mode = per_row ? (want_tr ? AMAX_GROUPS : AMAX_NONE) : AMAX_NONE;
        if (a.dt == SRQ_F32)
            amax_kernel<float><<<grid, AMAX_THREADS, 0, stream>>>((const float*)a.x, rows, cols, a.ld, vec_in,
                                                                 amax_rm, rm_mode, amax_tr, tr_mode);
        else
            amax_kernel<__nv_bfloat16><<<grid, AMAX_THREADS, 0, stream>>>((const __nv_bfloat16*)a.x, rows, cols, a.ld,
                                                                         vec_in, amax_rm, rm_mode, amax_tr, tr_mode);
        ++g_launches;
    }
    {
        // per tensor: one group feeds both layouts' scale outputs
        const int64_t n0 = per_row ? n_rm : 1;
        const int64_t n1 = per_row ? n_tr : ((want_tr && a.scale_tr) ? 1 : 0);
        const int64_t n = n0 > n1 ? n0 : n1;
        const int threads = 256;
        scales_kernel<<<(unsigned)((n + threads - 1) / threads), threads, 0, stream>>>(
            amax_rm, n0, inv_rm, want_rm ? a.scale_rm : nullptr,
            amax_tr, n1, inv_tr, want_tr ? a.scale_tr : nullptr, qmax, status);
        ++g_launches;
    }
    {
        QuantParams P;
        P.rows = rows; P.cols = cols; P.ld = a.ld;
        P.index_offset = a.q.index_offset;
        P.key0 = (uint32_t)a.q.seed; P.key1 = (uint32_t)(a.q.seed >> 32);
        P.tid0 = (uint32_t)a.q.tensor_id; P.tid1 = (uint32_t)(a.q.tensor_id >> 32);
        P.qmax = qmax;
        P.sr = a.q.round == SRQ_SR;
        P.per_row = per_row;
        P.codes_rm = a.codes_rm; P.ld_rm = a.ld_rm;
        P.codes_tr = a.codes_tr; P.ld_tr = a.ld_tr;
        P.inv_rm = inv_rm; P.inv_tr = inv_tr;
        P.vec_in = vec_in;
        P.vec_rm = want_rm && ((uintptr_t)a.codes_rm % 4 == 0) && (a.ld_rm % 4 == 0);
        P.vec_tr = want_tr && ((uintptr_t)a.codes_tr % 4 == 0) && (a.ld_tr % 4 == 0);
        const bool aligned = (cols % 4 == 0) && (a.q.index_offset % 4 == 0);
        const unsigned grid = (unsigned)(((cols + Q_TILE - 1) / Q_TILE) * ((rows + Q_TILE - 1) / Q_TILE));
        if (a.dt == SRQ_F32) {
            if (aligned) quantize_kernel<float, true><<<grid, Q_THREADS, 0, stream>>>((const float*)a.x, P);
            else quantize_kernel<float, false><<<grid, Q_THREADS, 0, stream>>>((const float*)a.x, P);
        } else {
            if (aligned) quantize_kernel<__nv_bfloat16, true><<<grid, Q_THREADS, 0, stream>>>((const __nv_bfloat16*)a.x, P);
            else quantize_kernel<__nv_bfloat16, false><<<grid, Q_THREADS, 0, stream>>>((const __nv_bfloat16*)a.x, P);
        }
        ++g_launches;
    }
    return cudaGetLastError();
}

}  // namespace srq
