// Product of two int8 code matrices on the 5th-generation tensor cores (sm_100a), with the
// dequantizing epilogue: the paper's mixed-precision matmul (low-precision multiply, wide
// accumulate) used by Alg. 1 (forward) and Alg. 2 (both backward products).
//
//   acc[i,j] = sum_k a[i,k] * b[j,k]          int8 x int8 -> int32, exact
//   out[i,j] = float(acc[i,j]) * (s_row[i] * s_col[j])
//
// Persistent kernel, one CTA per SM, 10 warps.  Two forms of the same code (template CTAS):
//   CTAS = 2  two CTAs on neighbouring SMs (a cluster) share one 256 x 256 output tile: each stages
//             its own 128 rows of a and 128 of the 256 rows of b, and the leader CTA issues
//             tcgen05.mma.cta_group::2 (M256 x N256 x K32), which reads both CTAs' shared memory
//             and writes 128 accumulator rows into each CTA's TMEM.  Per SM this halves the b
//             traffic and the shared-memory reads per MMA; used whenever M > 128.
//   CTAS = 1  one CTA per 128 x 256 tile with tcgen05.mma.cta_group::1 (M128 x N256 x K32).
// Roles:
//   warp 0      TMA producer: 128-byte-swizzled tiles of a and b into a shared-memory ring
//               (5 stages of 32 KB, or 3 of 48 KB), signalled through mbarriers; with CTAS = 2
//               both CTAs' loads complete on the leader's barrier (no multicast is used)
//   warp 1      allocates TMEM; in the leader one thread issues the MMAs; accumulators live in
//               TMEM, two buffers of 256 columns, so the tensor pipe starts the next tile while
//               the previous one is being drained
//   warps 2-9   epilogue, two groups of four warps: group g drains accumulator buffer g, i.e. every
//               other tile of this CTA, so that one group is in the middle of its block stores
//               while the other is between tiles and the store queue never runs dry (on
//               output-bound shapes the stores, not the tensor pipe, decide the time).  A warp
//               takes one TMEM lane quarter: tcgen05.ld, convert, scale and store (through shared
//               memory and TMA block stores); or, for a split contraction, add the exact int32
//               partial sums into a zeroed workspace (TMA block reductions), which dequant_kernel
//               scales afterwards
// Ragged edges rely on TMA zero fill for loads and on bounds checks for stores.
// Every wait is bounded by a wall-clock limit; on expiry the CTA records SRQ_ERR_TIMEOUT,
// stops issuing work, waits (bounded) for what it has in flight, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "common.cuh"

namespace srq {

constexpr int BM = 128, BN = 256, BK = 128;          // per-CTA rows, tile columns, k-block (bytes = int8 elements)
constexpr int UMMA_K = 32;                             // bytes of K per tcgen05.mma.kind::i8
constexpr int A_STAGE_BYTES = BM * BK;
constexpr int TMEM_COLS = 512;                         // two accumulator buffers of BN columns
constexpr int EPI_GROUPS = 2;                          // epilogue warp groups; group g drains accumulator buffer g
constexpr int GEMM_THREADS = 64 + 128 * EPI_GROUPS;
constexpr uint64_t WAIT_LIMIT_NS = 2000000000ull;      // 2 s

template <int CTAS>
struct Cfg {
    static constexpr int B_ROWS = BN / CTAS;                         // rows of b staged by each CTA
    static constexpr int B_STAGE_BYTES = B_ROWS * BK;
    static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    static constexpr int STAGES = CTAS == 1 ? 3 : 5;
};

template <int STAGES>
struct SharedTail {                                    // after the stage ring
    uint64_t full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain;
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
    alignas(16) float s_col[2 * EPI_GROUPS][BN];   // read as float4; two per epilogue group, used in turn
};
constexpr int OUT_STAGE_BYTES = 32 * 32 * 4;           // one 32 x 32 block of 32-bit results per epilogue warp
template <int CTAS>
constexpr size_t gemm_smem() {
    return 1024 /*alignment slack*/ + (size_t)Cfg<CTAS>::STAGES * Cfg<CTAS>::STAGE_BYTES + 4 * EPI_GROUPS * OUT_STAGE_BYTES +
           sizeof(SharedTail<Cfg<CTAS>::STAGES>);
}

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Non-blocking look at a phase (never suspends the thread).
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if the limit passed or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint64_t limit_ns = WAIT_LIMIT_NS) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_ns();
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 63u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > limit_ns) return false;
        }
    }
}

// Cluster helpers (CTAS = 2): rank of this CTA in its pair, the pair-wide barrier, and the address
// of a shared-memory object of the pair's CTA `rank` in the shared::cluster window.
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
    return r;
}
// Arrival on a barrier of the pair (possibly the other CTA's).  What it orders here are TMEM reads
// against the MMAs that overwrite the accumulator, which the tcgen05 fences on both sides of the
// barrier take care of; a cluster-scope release on top of that made the arriving thread wait for its
// outstanding memory traffic (about 2 800 cycles per tile at the end of a tile's stores).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// Tile load into this CTA's shared memory.  CTAS = 2: the completion bytes are counted on the
// barrier at `bar_addr`, which may belong to the other CTA of the pair (no multicast).
template <int CTAS>
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int32_t x, int32_t y, uint32_t bar_addr) {
    if constexpr (CTAS == 1) {
        asm volatile(
            "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
            ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(bar_addr) : "memory");
    } else {
        asm volatile(
            "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
            ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(bar_addr) : "memory");
    }
}

// Block of results from shared memory to global memory; elements outside the tensor are clipped.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src_smem, int32_t x, int32_t y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src_smem), "r"(x), "r"(y) : "memory");
}
// Same, added into global memory (32-bit integer adds performed by the memory system).
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src_smem, int32_t x, int32_t y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 ::"l"(map), "r"(src_smem), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }   // source reusable
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }         // writes performed
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Thread `lane` holds 32 consecutive 32-bit results of row `lane` of a 32 x 32 block: writes them as a
// dense block with 128-byte rows in the 128-byte swizzle the tensor maps of the outputs use (16-byte
// chunk index xor row mod 8), which also spreads each 16-byte store of a warp over all banks.
__device__ __forceinline__ void stage_block(uint32_t stage, int lane, const uint32_t w[32]) {
    const uint32_t row = stage + (uint32_t)lane * 128u;
#pragma unroll
    for (int q = 0; q < 8; ++q)
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row + (uint32_t)((q ^ (lane & 7)) << 4)),
                     "r"(w[4 * q]), "r"(w[4 * q + 1]), "r"(w[4 * q + 2]), "r"(w[4 * q + 3]) : "memory");
}

// Two binary32 numbers rounded to nearest even bfloat16, the first in the low half.
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// One warp per CTA; with CTAS = 2 the same warp of both CTAs of the pair, same shared-memory offset.
template <int CTAS>
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t cols) {
    if constexpr (CTAS == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    } else {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
}
template <int CTAS>
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
    if constexpr (CTAS == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem], issued by one thread (of the leader CTA when CTAS = 2; the
// descriptors then address the same offsets in both CTAs).  KIND 0: int8 operands, int32
// accumulators (kind::i8); KIND 1: E4M3 operands, binary32 accumulators (kind::f8f6f4); KIND 2:
// bfloat16 operands, binary32 accumulators (kind::f16; 16 elements = 32 bytes of K per instruction).
template <int CTAS, int KIND>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
#define SRQ_UMMA(GROUP, KINDSTR)                                                                   \
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\n"                                        \
                 "tcgen05.mma.cta_group::" GROUP ".kind::" KINDSTR " [%0], %1, %2, %3, p;\n}"        \
                 ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory")
    if constexpr (CTAS == 1 && KIND == 0) SRQ_UMMA("1", "i8");
    else if constexpr (CTAS == 2 && KIND == 0) SRQ_UMMA("2", "i8");
    else if constexpr (CTAS == 1 && KIND == 1) SRQ_UMMA("1", "f8f6f4");
    else if constexpr (CTAS == 2 && KIND == 1) SRQ_UMMA("2", "f8f6f4");
    else if constexpr (CTAS == 1 && KIND == 2) SRQ_UMMA("1", "f16");
    else SRQ_UMMA("2", "f16");
#undef SRQ_UMMA
}
// The mbarrier gets one arrival once every MMA issued so far by this thread has completed.
// CTAS = 2, both = true: the barrier at the same offset in both CTAs of the pair gets it.
template <int CTAS>
__device__ __forceinline__ void umma_commit(uint64_t* bar, bool both) {
    if constexpr (CTAS == 1) {
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
    } else {
        if (both) {
            const uint16_t mask = 3;
            asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                         ::"r"(smem_u32(bar)), "h"(mask) : "memory");
        } else {
            asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
        }
    }
}

// 32 lanes x 32 consecutive 32-bit columns: thread t of the warp receives lane (base + t).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t v[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile written by TMA with the 128-byte
// swizzle: rows are 128 bytes, eight rows form a 1024-byte swizzle atom, so the stride between
// 8-row groups is 1024 bytes; the leading-dimension offset is not used for this layout.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                               // leading byte offset (unused), 16-byte units
    d |= (uint64_t)(1024 >> 4) << 32;                     // stride byte offset
    d |= (uint64_t)1 << 46;                               // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                               // 128-byte swizzle
    return d;
}

// Instruction descriptor: dense, no saturation, both operands K-major, N x M; KIND 0: D = s32,
// A = B = s8; KIND 1: D = f32, A = B = E4M3 (format 0); KIND 2: D = f32, A = B = bfloat16.
__device__ __forceinline__ constexpr uint32_t make_idesc(int kind, int m, int n) {
    const uint32_t types = kind == 0 ? ((2u << 4) | (1u << 7) | (1u << 10))          // s32 <- s8 x s8
                         : kind == 1 ? (1u << 4)                                   // f32 <- e4m3 x e4m3
                                     : ((1u << 4) | (1u << 7) | (1u << 10));       // f32 <- bf16 x bf16
    return types | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// Accumulator word to binary32: an exact int32 -> float conversion for integer codes, the bits
// themselves for binary32 accumulators.
template <int KIND>
__device__ __forceinline__ float acc_to_float(uint32_t v) {
    if constexpr (KIND == 0) return __int2float_rn((int)v);
    else return __uint_as_float(v);
}

// ------------------------------------------------------------------------------------------
// kernel
// ------------------------------------------------------------------------------------------
struct GemmParams {
    int64_t M, N;
    int32_t num_kb;            // 128-byte blocks along the contraction
    int32_t splits;            // parts the contraction of the LAST tiles is cut into (1 = none)
    int32_t full_tiles;        // tiles [0, full_tiles) are not split; the rest are, their sums going to `part`
    int32_t tiles_m, tiles_n;  // tiles of (128 * CTAS) x 256
    const float* s_row; int32_t row_stride;
    const float* s_col; int32_t col_stride;
    float* out; int64_t ldo;
    int32_t* acc_out;          // optional raw sums [M, N]
    int32_t* part;             // split tiles: zeroed int32 [(tiles - full_tiles) * 128 * CTAS, 256], tile after tile
    uint32_t* status;
    unsigned long long* timer; // optional: [0] lowered to the time the first CTA starts its work, [1] raised to the time the last one ends
    int32_t vec_out;           // 16-byte stores to out allowed
    int32_t tma_out;           // out is written with TMA stores (map_out valid, no acc_out)
    int32_t write_out;         // out is wanted (it may be left out when only codes are)
    int32_t rq_vec;            // 16-byte stores of codes allowed
    OutOptions opt;
};

// Re-quantization of 32 consecutive results of one row (columns col0 .. col0 + 31) with the
// caller's step size, saturating, by the quantizer's fixed-point rule; and their absmax.
// o holds binary32 bit patterns.  Thresholds follow the flat index rq_offset + row * N + col.
__device__ __forceinline__ void output_options(const GemmParams& P, const uint32_t (&o)[32], int64_t row, int64_t col0,
                                               float rq_inv, uint32_t& amax) {
    if (row >= P.M || col0 >= P.N) return;
    if (P.opt.absmax_bits) {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < P.N) amax = max(amax, o[i] & 0x7FFFFFFFu);
    }
    if (!P.opt.requant) return;
    const uint64_t i0 = P.opt.rq_offset + (uint64_t)row * (uint64_t)P.N + (uint64_t)col0;
    const bool aligned = (i0 & 3u) == 0;
    const float lim = P.opt.rq_lim;
    uint32_t words[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        uint32_t rnd[4] = {0u, 0u, 0u, 0u};
        if (P.opt.rq_sr) {
            if (aligned) {
                const uint64_t jb = (i0 >> 2) + q;
                philox_rounds((uint32_t)jb, (uint32_t)(jb >> 32), P.opt.rq_keys, rnd);
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint64_t ie = i0 + 4 * q + e, jb = ie >> 2;
                    uint32_t w[4];
                    philox_rounds((uint32_t)jb, (uint32_t)(jb >> 32), P.opt.rq_keys, w);
                    const uint32_t sel = (uint32_t)ie & 3u;
                    rnd[e] = sel == 0 ? w[0] : sel == 1 ? w[1] : sel == 2 ? w[2] : w[3];
                }
            }
        }
        uint32_t sums[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float s = __fmul_rn(__fmul_rn(__uint_as_float(o[4 * q + e]), rq_inv), 16777216.0f);
            s = fminf(fmaxf(s, -lim), lim);                                  // saturation
            if (P.opt.rq_sr) {
                asm("mad.hi.u32 %0, %1, 16777216, %2;" : "=r"(sums[e]) : "r"(~rnd[e]), "r"((uint32_t)__float2int_ru(s)));
            } else {
                sums[e] = (uint32_t)__float2int_rd(s) + 0x00800000u;
            }
        }
        words[q] = __byte_perm(__byte_perm(sums[0], sums[1], 0x0073), __byte_perm(sums[2], sums[3], 0x0073), 0x5410);
    }
    int8_t* dst = P.opt.rq_codes + row * P.opt.rq_ld + col0;
    if (P.rq_vec && col0 + 32 <= P.N) {
        *reinterpret_cast<uint4*>(dst) = make_uint4(words[0], words[1], words[2], words[3]);
        *reinterpret_cast<uint4*>(dst + 16) = make_uint4(words[4], words[5], words[6], words[7]);
    } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (col0 + i < P.N) dst[i] = (int8_t)((words[i >> 2] >> (8 * (i & 3))) & 0xFF);
    }
}

template <int STAGES>
__device__ __forceinline__ void give_up(SharedTail<STAGES>* T, uint32_t* status) {
    T->abort_flag = 1u;
    record_status(status, SRQ_ERR_TIMEOUT);
}

template <int CTAS, int KIND>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_i8_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_part, const GemmParams P) {
    pdl_trigger();                                   // the wait follows the set-up below, which touches only shared memory and TMEM
    using C = Cfg<CTAS>;
    constexpr int STAGES = C::STAGES, STAGE_BYTES = C::STAGE_BYTES;
    using Tail = SharedTail<STAGES>;
    static_assert(4 * EPI_GROUPS * 4 * OUT_STAGE_BYTES <= STAGES * STAGE_BYTES, "the ring must hold one staging buffer per block of a shared tile");
    extern __shared__ uint8_t smem_raw[];
    // the dynamic window starts at the same offset in every CTA, so the aligned layouts coincide
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    uint8_t* out_stage = smem + (size_t)STAGES * STAGE_BYTES;          // 1024-byte aligned, 4 KB per epilogue warp
    Tail* T = (Tail*)(out_stage + 4 * EPI_GROUPS * OUT_STAGE_BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = CTAS == 1 ? 0u : cluster_ctarank();   // position in the CTA pair
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&T->full[s], 1); mbar_init(&T->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&T->tmem_full[b], 1); mbar_init(&T->tmem_empty[b], 4 * CTAS); }
        mbar_init(&T->drain, 1);
        T->abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (warp == 1) tmem_alloc<CTAS>(&T->tmem_base, TMEM_COLS);
    tc_fence_before();
    if constexpr (CTAS == 1) __syncthreads(); else cluster_sync();   // the peer's barriers exist from here on
    tc_fence_after();
    const uint32_t tmem_base = T->tmem_base;
    pdl_wait();                                      // from here on the work before this kernel has finished and is visible
    if (P.timer && threadIdx.x == 0) atomicMin(&P.timer[0], (unsigned long long)global_ns());

    const int64_t groups = gridDim.x / CTAS, group = blockIdx.x / CTAS;   // a group = the CTAs of one tile
    // work units: the first full_tiles tiles whole, then every remaining tile in `splits` parts
    const int64_t tiles_all = (int64_t)P.tiles_m * P.tiles_n;
    const int64_t units = P.full_tiles + (tiles_all - P.full_tiles) * P.splits;
    const int32_t kb_per_split = (P.num_kb + P.splits - 1) / P.splits;
    auto decode = [&](int64_t u, int64_t& tile, int32_t& kb0, int32_t& kb1) {
        if (u < P.full_tiles) { tile = u; kb0 = 0; kb1 = P.num_kb; return; }
        const int64_t v = u - P.full_tiles;
        tile = P.full_tiles + v / P.splits;
        kb0 = (int32_t)(v % P.splits) * kb_per_split;
        kb1 = min(kb0 + kb_per_split, P.num_kb);
    };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_a) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(&map_b) : "memory");
            uint32_t it = 0;
            bool ok = true;
            for (int64_t u = group; u < units && ok; u += groups) {
                int64_t tile; int32_t kb0, kb1;
                decode(u, tile, kb0, kb1);
                const int32_t tn = (int32_t)(tile % P.tiles_n), tm = (int32_t)(tile / P.tiles_n);
                const int32_t row_a = (tm * CTAS + (int32_t)rank) * BM;
                const int32_t row_b = tn * BN + (int32_t)rank * C::B_ROWS;
                for (int32_t kb = kb0; kb < kb1; ++kb, ++it) {
                    const uint32_t s = it % STAGES, ph = (it / STAGES) & 1u;
                    if (!mbar_wait(&T->empty[s], ph ^ 1u, &T->abort_flag)) { give_up(T, P.status); ok = false; break; }
                    // the bytes of every CTA of the group are counted on the leader's barrier
                    if (leader) mbar_expect_tx(&T->full[s], STAGE_BYTES * CTAS);
                    const uint32_t bar = CTAS == 1 ? smem_u32(&T->full[s]) : map_to_cta(smem_u32(&T->full[s]), 0);
                    uint8_t* sa = smem + (size_t)s * STAGE_BYTES;
                    tma_load_2d<CTAS>(sa, &map_a, kb * BK, row_a, bar);
                    tma_load_2d<CTAS>(sa + A_STAGE_BYTES, &map_b, kb * BK, row_b, bar);
                }
            }
            if (!ok) {
                // loads already issued must land before the CTA may leave
                if (leader) {
                    const uint32_t back = it < (uint32_t)STAGES ? it : (uint32_t)STAGES;
                    for (uint32_t j = 1; j <= back; ++j) {
                        const uint32_t jt = it - j;
                        const uint64_t t0 = global_ns();
                        while (!mbar_try_wait(&T->full[jt % STAGES], (jt / STAGES) & 1u) && global_ns() - t0 < WAIT_LIMIT_NS) {}
                    }
                } else {
                    const uint64_t t0 = global_ns();          // their barrier is not ours to wait on: give them time
                    while (global_ns() - t0 < 1000000ull) {}
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && leader) {
            const uint32_t idesc = make_idesc(KIND, BM * CTAS, BN);
            uint32_t lt = 0;
            bool ok = true;
            // Whatever this thread does between the last MMA of one k-block and the first of the next can show
            // up as idle pipe cycles, so the loop keeps stage index, phase and descriptors in registers and
            // looks at the next stage's barrier while the current k-block's MMAs are still queued (worth
            // about half a percent on long contractions).
            uint32_t s = 0, ph = 0;                                   // ring position of the next k-block
            const uint64_t desc0 = make_smem_desc(smem_u32(smem));    // stage 0, operand a; stages are STAGE_BYTES apart
            uint64_t da = desc0;
            bool ready = false;                                       // stage s is known to be full
            for (int64_t u = group; u < units && ok; u += groups, ++lt) {
                int64_t tile; int32_t kb0, kb1;
                decode(u, tile, kb0, kb1);
                const uint32_t buf = lt & 1u, use = lt >> 1;
                if (!mbar_wait(&T->tmem_empty[buf], (use & 1u) ^ 1u, &T->abort_flag)) { give_up(T, P.status); ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + buf * BN;
                for (int32_t kb = kb0; kb < kb1; ++kb) {
                    if (!ready && !mbar_wait(&T->full[s], ph, &T->abort_flag)) { give_up(T, P.status); ok = false; break; }
                    tc_fence_after();
                    const uint64_t db = da + (uint64_t)(A_STAGE_BYTES >> 4);
                    const uint32_t ns = s + 1 == (uint32_t)STAGES ? 0u : s + 1, nph = ns == 0u ? ph ^ 1u : ph;
                    // advancing K inside the swizzle atom = advancing the start address
                    umma<CTAS, KIND>(d_tmem, da, db, idesc, kb > kb0 ? 1u : 0u);
                    ready = mbar_test_wait(&T->full[ns], nph);      // usually true already: the ring runs ahead
#pragma unroll
                    for (int k = 1; k < BK / UMMA_K; ++k)
                        umma<CTAS, KIND>(d_tmem, da + (uint64_t)((k * UMMA_K) >> 4), db + (uint64_t)((k * UMMA_K) >> 4), idesc, 1u);
                    umma_commit<CTAS>(&T->empty[s], true);       // stage reusable (in every CTA) once these MMAs have read it
                    s = ns; ph = nph;
                    da = ns == 0u ? desc0 : da + (uint64_t)(STAGE_BYTES >> 4);
                }
                if (ok) umma_commit<CTAS>(&T->tmem_full[buf], true);   // accumulator complete
            }
            if (!ok) {
                umma_commit<CTAS>(&T->drain, false);
                const uint64_t t0 = global_ns();
                while (!mbar_try_wait(&T->drain, 0u) && global_ns() - t0 < WAIT_LIMIT_NS) {}
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quarter = warp & 3;                    // TMEM lanes this warp may read
        const int egrp = (warp - 2) >> 2;                // this warp's group: it takes the units that use accumulator buffer egrp
        const int etid = (threadIdx.x - 64) & 127;       // 0..127 within the epilogue group
        // the MMA issuer's barriers (in the leader CTA)
        const uint32_t empty_bar0 = CTAS == 1 ? smem_u32(&T->tmem_empty[0]) : map_to_cta(smem_u32(&T->tmem_empty[0]), 0);
        const uint32_t empty_bar1 = CTAS == 1 ? smem_u32(&T->tmem_empty[1]) : map_to_cta(smem_u32(&T->tmem_empty[1]), 0);
        float rq_inv = 0.0f;                                  // reciprocal of the caller's step size
        if (P.opt.requant) {
            const float d = *P.opt.rq_step;
            rq_inv = d == 0.0f ? 0.0f : __fdiv_rn(1.0f, d);
            if (!(fabsf(rq_inv) <= 3.402823466e38f)) rq_inv = 0.0f;
        }
        uint32_t amax = 0u;
        uint32_t lt = 0;
        bool ok = true;
        // Where a unit's tile lies (one division per unit; 32-bit when the tile index allows).
        auto locate = [&](int64_t u, int64_t& tile, int32_t& tn, int32_t& tm) {
            int32_t kb0_unused, kb1_unused;
            decode(u, tile, kb0_unused, kb1_unused);
            if (tile < (1ll << 32)) {
                tm = (int32_t)((uint32_t)tile / (uint32_t)P.tiles_n);
                tn = (int32_t)((uint32_t)tile - (uint32_t)tm * (uint32_t)P.tiles_n);
            } else {
                tm = (int32_t)(tile / P.tiles_n);
                tn = (int32_t)(tile % P.tiles_n);
            }
        };
        // Step sizes of a unit's tile: this thread's row and two of the 256 columns (etid, etid + 128).
        // They are fetched one unit ahead, so that their latency falls into the previous tile's work.
        float sc_next[2] = {0.0f, 0.0f}, sr_next = 0.0f;
        int64_t tile_next = 0; int32_t tn_next = 0, tm_next = 0;
        auto fetch_steps = [&](int64_t u) {
            locate(u, tile_next, tn_next, tm_next);
            const int64_t col_base = (int64_t)tn_next * BN;
            const int64_t row = ((int64_t)tm_next * CTAS + rank) * BM + quarter * 32 + lane;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int64_t c = col_base + etid + 128 * h;
                sc_next[h] = (c < P.N) ? __ldg(P.s_col + c * P.col_stride) : 0.0f;
            }
            sr_next = (row < P.M) ? __ldg(P.s_row + row * P.row_stride) : 0.0f;
        };
        // the MMA warp alternates the two accumulators unit by unit, so group g owns this CTA's units g, g + 2, ...
        // A launch in which no CTA has more than one unit is all latency: there both groups drain that
        // one unit, half of its columns each.
        const bool share = units <= groups;
        const int64_t u_first = share ? group : group + (int64_t)egrp * groups, u_step = share ? groups : (int64_t)EPI_GROUPS * groups;
        if (u_first < units) fetch_steps(u_first);
        for (int64_t u = u_first; u < units && ok; u += u_step, ++lt) {
            const int64_t tile = tile_next;
            const int32_t tn = tn_next, tm = tm_next;
            const bool whole = u < P.full_tiles;              // this unit holds the complete sums of its tile
            const uint32_t buf = share ? 0u : (uint32_t)egrp, use = lt;
            const bool releases = !share || egrp == 0;           // one arrival per warp on the accumulator's barrier
            const int j_lo = share ? egrp * (BN / 64) : 0, j_hi = share ? j_lo + BN / 64 : BN / 32;     // 32-column blocks
            const int64_t row0 = ((int64_t)tm * CTAS + rank) * BM;      // first row of this CTA's half
            const int64_t row = row0 + quarter * 32 + lane;
            const int64_t col_base = (int64_t)tn * BN;
            // stage this tile's column step sizes (the group's other buffer may still be read by slower
            // warps; this one was last read two of the group's tiles ago, which every warp has left)
            const uint32_t cbuf = (uint32_t)egrp * 2u + (lt & 1u);
            T->s_col[cbuf][etid] = sc_next[0];
            T->s_col[cbuf][etid + 128] = sc_next[1];
            const float sr = sr_next;
            if (u + u_step < units) fetch_steps(u + u_step);
            bool mine = mbar_wait(&T->tmem_full[buf], use & 1u, &T->abort_flag);
            if (!mine) give_up(T, P.status);
            // the four warps of a group must leave together (they share named barrier 1 + group): one barrier makes the
            // staged step sizes visible and tells every thread whether any of them gave up
            uint32_t any_gave_up;
            asm volatile("{\n.reg .pred p, q;\nsetp.ne.u32 q, %1, 0;\nbar.red.or.pred p, %2, 128, q;\nselp.u32 %0, 1, 0, p;\n}"
                         : "=r"(any_gave_up) : "r"((uint32_t)(!mine || T->abort_flag != 0u)), "r"(1 + egrp) : "memory");
            if (any_gave_up) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + buf * BN;
            const uint32_t stage = smem_u32(out_stage + (warp - 2) * OUT_STAGE_BYTES);
            // A CTA with a single unit has no further use for its operand ring once the accumulator is
            // complete: its blocks are staged there, one buffer per block, so that no block waits for the
            // previous block's store to have read the staging buffer (8 warps x 4 blocks x 4 KB).
            const uint32_t ring_stage = smem_u32(smem) + (uint32_t)((warp - 2) * 4) * (uint32_t)OUT_STAGE_BYTES;
            const int32_t wrow = (int32_t)(row0 + quarter * 32);           // first row of this warp's blocks
            // The accumulator is free as soon as this warp's last TMEM load has completed: the MMAs of the
            // tile after next start while the last block is still being scaled, staged and stored.
            auto release_acc = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && releases) mbar_arrive_cluster(buf ? empty_bar1 : empty_bar0);
            };
            if (whole && P.tma_out && P.opt.out_bf16) {
                // two 32-column blocks at a time: 64 bfloat16 results per row fill the 128-byte rows
                // of the staging block, stored as one 32 x 64 box
#pragma unroll 1
                for (int j = j_lo / 2; j < j_hi / 2; ++j) {
                    uint32_t w[32];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        uint32_t v[32];
                        tmem_ld32(taddr + j * 64 + h * 32, v);
                        tmem_ld_wait();
                        if (h == 1 && j == j_hi / 2 - 1) release_acc();
                        const float* sc = &T->s_col[cbuf][j * 64 + h * 32];
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            v[i] = __float_as_uint(__fmul_rn(acc_to_float<KIND>(v[i]), __fmul_rn(sr, sc[i])));
                        output_options(P, v, row, (int32_t)col_base + j * 64 + h * 32, rq_inv, amax);
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[h * 16 + i] = pack_bf16(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
                    }
                    const int32_t col0 = (int32_t)col_base + j * 64;
                    const uint32_t stg = share ? ring_stage + (uint32_t)(j - j_lo / 2) * (uint32_t)OUT_STAGE_BYTES : stage;
                    if (!share && lane == 0) bulk_wait_read();
                    __syncwarp();
                    stage_block(stg, lane, w);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0 && wrow < P.M && col0 < P.N) { tma_store_2d(&map_out, stg, col0, wrow); bulk_commit(); }
                }
            } else if (whole && P.tma_out) {
                // registers -> swizzled shared-memory block -> one TMA store per 32 x 32 block
#pragma unroll 1
                for (int j = j_lo; j < j_hi; ++j) {
                    uint32_t v[32];
                    tmem_ld32(taddr + j * 32, v);
                    tmem_ld_wait();
                    if (j == j_hi - 1) release_acc();
                    const float* sc = &T->s_col[cbuf][j * 32];
                    if (!P.opt.raw_sums) {                    // raw sums leave as the int32 words they are
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const float4 c4 = *reinterpret_cast<const float4*>(sc + 4 * q);
                            v[4 * q + 0] = __float_as_uint(__fmul_rn(acc_to_float<KIND>(v[4 * q + 0]), __fmul_rn(sr, c4.x)));
                            v[4 * q + 1] = __float_as_uint(__fmul_rn(acc_to_float<KIND>(v[4 * q + 1]), __fmul_rn(sr, c4.y)));
                            v[4 * q + 2] = __float_as_uint(__fmul_rn(acc_to_float<KIND>(v[4 * q + 2]), __fmul_rn(sr, c4.z)));
                            v[4 * q + 3] = __float_as_uint(__fmul_rn(acc_to_float<KIND>(v[4 * q + 3]), __fmul_rn(sr, c4.w)));
                        }
                    }
                    const int32_t col0 = (int32_t)col_base + j * 32;
                    output_options(P, v, row, col0, rq_inv, amax);
                    const uint32_t stg = share ? ring_stage + (uint32_t)(j - j_lo) * (uint32_t)OUT_STAGE_BYTES : stage;
                    if (!share && lane == 0) bulk_wait_read();          // the previous block has left the staging buffer
                    __syncwarp();
                    stage_block(stg, lane, v);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0 && wrow < P.M && col0 < P.N) {
                        if (P.opt.accumulate == 1) tma_reduce_add_2d(&map_out, stg, col0, wrow);   // binary32 adds in memory
                        else tma_store_2d(&map_out, stg, col0, wrow);
                        bulk_commit();
                    }
                }
            } else if (whole) {
#pragma unroll 1
                for (int j = j_lo; j < j_hi; ++j) {
                    uint32_t v[32];
                    tmem_ld32(taddr + j * 32, v);
                    tmem_ld_wait();
                    const int64_t col0 = col_base + j * 32;
                    if (row < P.M && col0 < P.N) {
                        const float* sc = &T->s_col[cbuf][j * 32];
                        if (P.acc_out) {
                            int32_t* ad = P.acc_out + row * P.N + col0;
                            if (P.opt.accumulate == 2) {
                                // running int32 sums over calls (exact while they fit): acc_out += sums, and the
                                // result below is formed from the total
                                bool wrapped = false;
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (col0 + i < P.N) {
                                        const int32_t before = ad[i], add = (int32_t)v[i];
                                        const int32_t total = (int32_t)((uint32_t)before + (uint32_t)add);
                                        wrapped |= ((before ^ total) & (add ^ total)) < 0;
                                        ad[i] = total;
                                        v[i] = (uint32_t)total;
                                    }
                                if (wrapped) record_status(P.status, SRQ_ERR_ACC_OVERFLOW);
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (col0 + i < P.N) ad[i] = (int32_t)v[i];
                            }
                        }
                        if (P.opt.raw_sums) {                   // the sums themselves, element by element
                            uint32_t* dst = reinterpret_cast<uint32_t*>(P.out) + row * P.ldo + col0;
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (col0 + i < P.N) dst[i] = v[i];
                            continue;
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            v[i] = __float_as_uint(__fmul_rn(acc_to_float<KIND>(v[i]), __fmul_rn(sr, sc[i])));
                        output_options(P, v, row, col0, rq_inv, amax);
                        if (P.write_out && P.opt.out_bf16) {
                            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(P.out) + row * P.ldo + col0;
#pragma unroll
                            for (int i = 0; i < 32; ++i)
                                if (col0 + i < P.N) dst[i] = __float2bfloat16_rn(__uint_as_float(v[i]));
                        } else if (P.write_out) {
                            float* dst = P.out + row * P.ldo + col0;
                            if (P.vec_out && col0 + 32 <= P.N) {
#pragma unroll
                                for (int q = 0; q < 8; ++q) {
                                    float4 o = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                           __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                                    if (P.opt.accumulate == 1) {
                                        const float4 p = *reinterpret_cast<const float4*>(dst + 4 * q);
                                        o.x = __fadd_rn(p.x, o.x); o.y = __fadd_rn(p.y, o.y); o.z = __fadd_rn(p.z, o.z); o.w = __fadd_rn(p.w, o.w);
                                    }
                                    __stcs(reinterpret_cast<float4*>(dst + 4 * q), o);
                                }
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i)
                                    if (col0 + i < P.N)
                                        dst[i] = P.opt.accumulate == 1 ? __fadd_rn(dst[i], __uint_as_float(v[i])) : __uint_as_float(v[i]);
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && releases) mbar_arrive_cluster(buf ? empty_bar1 : empty_bar0);
            } else {
                // exact partial sums: integer adds commute, so any arrival order gives the same total.
                // `part` holds the split tiles one after another, 128 * CTAS rows of 256 sums each.
                const int32_t prow = (int32_t)((tile - P.full_tiles) * (BM * CTAS) + rank * BM + quarter * 32);
#pragma unroll 1
                for (int j = j_lo; j < j_hi; ++j) {
                    uint32_t v[32];
                    tmem_ld32(taddr + j * 32, v);
                    tmem_ld_wait();
                    if (j == j_hi - 1) release_acc();
                    const uint32_t stg = share ? ring_stage + (uint32_t)(j - j_lo) * (uint32_t)OUT_STAGE_BYTES : stage;
                    if (!share && lane == 0) bulk_wait_read();
                    __syncwarp();
                    stage_block(stg, lane, v);
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) { tma_reduce_add_2d(&map_part, stg, j * 32, prow); bulk_commit(); }
                }
            }
        }
        if (P.opt.absmax_bits) {      // absmax of everything this warp produced: one guarded atomic
            amax = __reduce_max_sync(0xFFFFFFFFu, amax);
            if (lane == 0 && amax > __ldcg(P.opt.absmax_bits)) atomicMax(P.opt.absmax_bits, amax);
        }
    }

    if (warp >= 2 && lane == 0) bulk_wait_all();      // stores still reading the staging buffers
    // nobody leaves while the other CTA of the pair may still address this one's barriers, shared
    // memory or TMEM
    __syncwarp();
    tc_fence_before();
    if constexpr (CTAS == 1) __syncthreads(); else cluster_sync();
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc<CTAS>(tmem_base, TMEM_COLS);
    }
    if (P.timer && threadIdx.x == 0) atomicMax(&P.timer[1], (unsigned long long)global_ns());
}

// Second step of a split contraction: out = float(sum) * (s_row * s_col) over the finished sums of the
// split tiles.  `part` holds them tile after tile ([tile_rows, 256] each); tile t of it is output tile
// first_tile + t in row-major tile order.  One thread per four consecutive columns.
__global__ void __launch_bounds__(256)
dequant_kernel(const int32_t* __restrict__ part, int64_t n_tiles, int64_t first_tile, int32_t tiles_n, int32_t tile_rows,
               int64_t M, int64_t N, const float* __restrict__ s_row, int32_t row_stride,
               const float* __restrict__ s_col, int32_t col_stride, float* __restrict__ out, int64_t ldo,
               int32_t* __restrict__ acc_out, int vec, int accumulate, int out_bf16, int raw_sums, uint32_t* status) {
    pdl_enter();
    const int64_t per_tile = (int64_t)tile_rows * (BN / 4);
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < n_tiles * per_tile; g += (int64_t)gridDim.x * blockDim.x) {
        const int64_t t = g / per_tile, in_tile = g % per_tile;
        const int64_t tile = first_tile + t;
        const int64_t r = (tile / tiles_n) * tile_rows + in_tile / (BN / 4);
        const int64_t c = (tile % tiles_n) * BN + (in_tile % (BN / 4)) * 4;
        if (r >= M || c >= N) continue;
        const int4 a = __ldcg(reinterpret_cast<const int4*>(part + g * 4));
        int32_t av[4] = {a.x, a.y, a.z, a.w};
        if (accumulate == 2) {             // running int32 sums over calls: the result is formed from the total
            for (int e = 0; e < 4 && c + e < N; ++e) {
                const int32_t before = acc_out[r * N + c + e];
                const int32_t total = (int32_t)((uint32_t)before + (uint32_t)av[e]);
                if (((before ^ total) & (av[e] ^ total)) < 0) record_status(status, SRQ_ERR_ACC_OVERFLOW);
                av[e] = total;
            }
        }
        if (raw_sums) {                        // the caller wants the sums themselves
            int32_t* dst = reinterpret_cast<int32_t*>(out) + r * ldo + c;
            if (vec && c + 4 <= N) *reinterpret_cast<int4*>(dst) = make_int4(av[0], av[1], av[2], av[3]);
            else for (int e = 0; e < 4 && c + e < N; ++e) dst[e] = av[e];
            continue;
        }
        const float sr = s_row[r * row_stride];
        float o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            o[e] = (c + e < N) ? __fmul_rn(__int2float_rn(av[e]), __fmul_rn(sr, s_col[(c + e) * col_stride])) : 0.0f;
        if (out_bf16) {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out) + r * ldo + c;
            if (vec && c + 4 <= N) {
                *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3]));
            } else {
                for (int e = 0; e < 4 && c + e < N; ++e) dst[e] = __float2bfloat16_rn(o[e]);
            }
            if (acc_out)
                for (int e = 0; e < 4 && c + e < N; ++e) acc_out[r * N + c + e] = av[e];
            continue;
        }
        float* dst = out + r * ldo + c;
        if (vec && c + 4 <= N) {
            float4 w = make_float4(o[0], o[1], o[2], o[3]);
            if (accumulate == 1) {
                const float4 p = *reinterpret_cast<const float4*>(dst);
                w.x = __fadd_rn(p.x, w.x); w.y = __fadd_rn(p.y, w.y); w.z = __fadd_rn(p.z, w.z); w.w = __fadd_rn(p.w, w.w);
            }
            *reinterpret_cast<float4*>(dst) = w;
        } else {
            for (int e = 0; e < 4 && c + e < N; ++e) dst[e] = accumulate == 1 ? __fadd_rn(dst[e], o[e]) : o[e];
        }
        if (acc_out)
            for (int e = 0; e < 4 && c + e < N; ++e) acc_out[r * N + c + e] = av[e];
    }
}

// The finishing step on its own, over a caller's int32 matrix: out = float(sum) * (s_row * s_col), the
// same two binary32 multiplies in the same order as the epilogue.  For sums that were added up
// elsewhere (over token shards on several devices) before they are scaled once.  One thread per four
// consecutive columns; vec: 16-byte loads and 16-byte (binary32) or 8-byte (bfloat16) stores allowed.
__global__ void __launch_bounds__(256)
finish_sums_kernel(const int32_t* __restrict__ acc, int64_t ld_acc, int64_t M, int64_t N,
                   const float* __restrict__ s_row, int32_t row_stride, const float* __restrict__ s_col, int32_t col_stride,
                   float* __restrict__ out, int64_t ldo, int vec, int out_bf16) {
    pdl_enter();
    const int64_t per_row = (N + 3) / 4;
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < M * per_row; g += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = g / per_row, c = (g % per_row) * 4;
        const int32_t* src = acc + r * ld_acc + c;
        int32_t av[4] = {0, 0, 0, 0};
        if (vec && c + 4 <= N) {
            const int4 a = __ldcs(reinterpret_cast<const int4*>(src));
            av[0] = a.x; av[1] = a.y; av[2] = a.z; av[3] = a.w;
        } else {
            for (int e = 0; e < 4 && c + e < N; ++e) av[e] = src[e];
        }
        const float sr = s_row[r * row_stride];
        float o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
            o[e] = (c + e < N) ? __fmul_rn(__int2float_rn(av[e]), __fmul_rn(sr, s_col[(c + e) * col_stride])) : 0.0f;
        if (out_bf16) {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out) + r * ldo + c;
            if (vec && c + 4 <= N) *reinterpret_cast<uint2*>(dst) = make_uint2(pack_bf16(o[0], o[1]), pack_bf16(o[2], o[3]));
            else for (int e = 0; e < 4 && c + e < N; ++e) dst[e] = __float2bfloat16_rn(o[e]);
        } else {
            float* dst = out + r * ldo + c;
            if (vec && c + 4 <= N) __stcs(reinterpret_cast<float4*>(dst), make_float4(o[0], o[1], o[2], o[3]));
            else for (int e = 0; e < 4 && c + e < N; ++e) dst[e] = o[e];
        }
    }
}

// Self-test of the bounded wait: one thread waits on a barrier that nothing ever arrives on, with a
// short limit; the wait gives up, the status word receives SRQ_ERR_TIMEOUT and the kernel returns.
__global__ void bounded_wait_probe_kernel(uint32_t* status, uint64_t limit_ns) {
    __shared__ uint64_t bar;
    __shared__ volatile uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait(&bar, 0u, &abort_flag, limit_ns)) record_status(status, SRQ_ERR_TIMEOUT);
    }
}

cudaError_t launch_bounded_wait_probe(uint32_t* status, uint64_t limit_ns, cudaStream_t stream) {
    bounded_wait_probe_kernel<<<1, 32, 0, stream>>>(status, limit_ns);
    count_launch();
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    });
    return fn;
}

// [rows, kc] int8 matrix with row pitch ld bytes, boxes of box_rows x 128 bytes, 128-byte swizzle.
static bool encode_operand(CUtensorMap* map, const int8_t* base, int64_t rows, int64_t kc, int64_t ld, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {(cuuint64_t)kc, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld};
    cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, (void*)base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// [rows, cols] matrix of 32-bit (or bfloat16) elements with row pitch ld elements, boxes of 32 rows x
// 128 bytes, 128-byte swizzle.
static bool encode_output(CUtensorMap* map, void* base, CUtensorMapDataType dt, int64_t rows, int64_t cols, int64_t ld) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const unsigned esize = dt == CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 ? 2 : 4;     // rows of a box are 128 bytes
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * esize};
    cuuint32_t box[2] = {128 / esize, 32};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, dt, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
               CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Per device: SM count, the number of CTA pairs that can be resident at once, and the one-time
// opt-in to the large dynamic shared-memory carve-out.
struct DeviceInfo { bool ready = false; int sms = 1; int pairs = 0; };

static bool device_info(DeviceInfo** out) {
    static DeviceInfo info[64];
    static std::mutex mu;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
    std::lock_guard<std::mutex> lock(mu);
    DeviceInfo& d = info[dev];
    if (!d.ready) {
        if (cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || d.sms <= 0) return false;
        if (cudaFuncSetAttribute(gemm_i8_kernel<1, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem<1>()) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(gemm_i8_kernel<2, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem<2>()) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(gemm_i8_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem<1>()) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(gemm_i8_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem<2>()) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(gemm_i8_kernel<1, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem<1>()) != cudaSuccess) return false;
        if (cudaFuncSetAttribute(gemm_i8_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)gemm_smem<2>()) != cudaSuccess) return false;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(d.sms / 2 * 2)); cfg.blockDim = dim3(GEMM_THREADS); cfg.dynamicSmemBytes = gemm_smem<2>();
        cudaLaunchAttribute at;
        at.id = cudaLaunchAttributeClusterDimension; at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
        cfg.attrs = &at; cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, gemm_i8_kernel<2, 0>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
        d.pairs = n < d.sms / 2 ? n : d.sms / 2;
        d.ready = true;
    }
    *out = &d;
    return true;
}

cudaError_t launch_finish_sums(const int32_t* acc, int64_t ld_acc, int64_t M, int64_t N, const float* s_row, int32_t row_stride,
                               const float* s_col, int32_t col_stride, float* out, int64_t ldo, int out_bf16, cudaStream_t stream) {
    if (M == 0 || N == 0) return cudaSuccess;
    DeviceInfo* dev = nullptr;
    if (!device_info(&dev)) return cudaErrorUnknown;
    const int vec = (uintptr_t)acc % 16 == 0 && ld_acc % 4 == 0 && (uintptr_t)out % (out_bf16 ? 8 : 16) == 0 && ldo % 4 == 0;
    const int64_t work = M * ((N + 3) / 4), blocks = (work + 255) / 256;
    const unsigned grid = (unsigned)(blocks < 16 * (int64_t)dev->sms ? blocks : 16 * (int64_t)dev->sms);
    launch_pdl(finish_sums_kernel, dim3(grid), dim3(256), 0, stream, acc, ld_acc, M, N, s_row, row_stride, s_col, col_stride, out, ldo,
               vec, out_bf16);
    count_launch();
    return cudaGetLastError();
}

// Issue-rate microbenchmark of the tensor pipe: every CTA pair multiplies operand blocks that already sit
// in shared memory (pseudo-random bytes, written once by the CTA itself), k_blocks times, with
// tcgen05.mma.cta_group::2.kind::i8 M256 N256 K32 into its two TMEM accumulators.  Nothing is loaded
// from or stored to global memory, so the time is what the kind::i8 pipe needs for those operations at
// the clock the power cap allows: the ceiling the product kernel's main loop is compared with.  The
// issuing thread stays at most two chunks of eight k-blocks ahead of the pipe (bounded waits).
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int32_t k_blocks, uint32_t* status) {
    pdl_enter();
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = (uint8_t*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);    // a: 128 x 128 bytes, b: 128 x 128 bytes
    __shared__ uint64_t done[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ volatile uint32_t abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool leader = cluster_ctarank() == 0;
    for (uint32_t i = threadIdx.x; i < (uint32_t)(A_STAGE_BYTES + Cfg<2>::B_STAGE_BYTES) / 4; i += blockDim.x) {
        uint32_t h = (i + 1u) * 2654435761u ^ (blockIdx.x * 40503u);     // any byte pattern that toggles the multipliers
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        reinterpret_cast<uint32_t*>(smem)[i] = h;
    }
    fence_async_smem();
    if (threadIdx.x == 0) {
        mbar_init(&done[0], 1); mbar_init(&done[1], 1);
        abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (warp == 1) tmem_alloc<2>(&tmem_base_s, TMEM_COLS);
    tc_fence_before();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    if (warp == 0 && lane == 0 && leader) {
        const uint32_t idesc = make_idesc(0, BM * 2, BN);
        const uint64_t da = make_smem_desc(smem_u32(smem)), db = make_smem_desc(smem_u32(smem) + A_STAGE_BYTES);
        bool ok = true;
        const int32_t chunks = (k_blocks + 7) / 8;
        for (int32_t c = 0; c < chunks && ok; ++c) {
            if (c >= 2 && !mbar_wait(&done[c & 1], (uint32_t)((c >> 1) - 1) & 1u, &abort_flag)) { ok = false; break; }
            const uint32_t d_tmem = tmem_base + (uint32_t)((c >> 2) & 1) * BN;      // both accumulators take turns
            const int32_t kb_end = min(8, k_blocks - 8 * c);
            for (int32_t kb = 0; kb < kb_end; ++kb)
#pragma unroll
                for (int k = 0; k < BK / UMMA_K; ++k)
                    umma<2, 0>(d_tmem, da + (uint64_t)((k * UMMA_K) >> 4), db + (uint64_t)((k * UMMA_K) >> 4), idesc, (c >= 8 || kb > 0 || k > 0) ? 1u : 0u);
            umma_commit<2>(&done[c & 1], false);
        }
        // everything issued must have left the pipe before TMEM is freed
        for (int32_t c = chunks > 2 ? chunks - 2 : 0; c < chunks && ok; ++c)
            if (!mbar_wait(&done[c & 1], (uint32_t)(c >> 1) & 1u, &abort_flag)) ok = false;
        if (!ok) record_status(status, SRQ_ERR_TIMEOUT);
    }
    __syncwarp();
    tc_fence_before();
    cluster_sync();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc<2>(tmem_base, TMEM_COLS);
    }
}

srq_status_t launch_mma_rate(int32_t k_blocks, uint32_t* status, int64_t* ops, cudaStream_t stream) {
    DeviceInfo* dev = nullptr;
    if (!device_info(&dev)) return SRQ_ERR_CUDA;
    if (dev->pairs <= 0) return SRQ_ERR_UNSUPPORTED;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)dev->pairs * 2); cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = 1024 + A_STAGE_BYTES + Cfg<2>::B_STAGE_BYTES; cfg.stream = stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = pdl_allowed(stream) ? 2 : 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, mma_rate_kernel, k_blocks, status);
    count_launch();
    if (ops) *ops = (int64_t)dev->pairs * k_blocks * (2ll * (BM * 2) * BN * BK);
    return e == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}

// Optional device-side timing of the product launches (srq_set_product_timer): launch i of the calls
// that follow writes its start and end times into slot i of a caller-owned device array.
static std::mutex g_timer_mu;
static unsigned long long* g_timer_slots = nullptr;
static int64_t g_timer_n = 0, g_timer_next = 0;

void set_product_timer(unsigned long long* slots, int64_t n) {
    std::lock_guard<std::mutex> lock(g_timer_mu);
    g_timer_slots = n > 0 ? slots : nullptr; g_timer_n = n > 0 ? n : 0; g_timer_next = 0;
}
static unsigned long long* next_timer_slot() {
    std::lock_guard<std::mutex> lock(g_timer_mu);
    if (!g_timer_slots || g_timer_next >= g_timer_n) return nullptr;
    return g_timer_slots + 2 * g_timer_next++;
}

// Which tiles are split, and into how many parts.  `groups` tiles run at a time.  Too few tiles to fill
// the machine: all of them are split.  Several rounds of tiles with a last, partly empty round: only
// the tiles of that round are split, so that it takes a fraction of a round.  Each part keeps at least
// 8 k-blocks.
static void plan_splits(int64_t tiles, int32_t num_kb, int groups, int32_t* full_tiles, int32_t* splits) {
    *full_tiles = (int32_t)tiles; *splits = 1;
    if (num_kb < 16 || tiles > 8 * (int64_t)groups) return;
    const int64_t full = tiles / groups * groups, rem = tiles - full;
    if (rem == 0) return;
    int s = (int)(groups / rem);
    if (s > num_kb / 8) s = num_kb / 8;
    if (s < 2) return;
    const int per = (num_kb + s - 1) / s;                   // no part may be empty
    s = (num_kb + per - 1) / per;
    if (s < 2) return;
    *full_tiles = (int32_t)full; *splits = s;
}

void gemm_plan_splits(int64_t tiles, int32_t num_kb, int groups, int32_t* full_tiles, int32_t* splits) {
    plan_splits(tiles, num_kb, groups, full_tiles, splits);
}

// What launch_gemm_i8 may use: int32 partial sums of the split tiles (fewer than one round of tiles,
// i.e. at most 160 blocks of 128 x 256 on any device this runs on).
size_t gemm_splitk_bytes(int64_t M, int64_t N) {
    int64_t blocks = 2 * ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
    if (blocks > 160) blocks = 160;
    return align_up((size_t)blocks * BM * BN * 4);
}

template <int CTAS, int KIND>
static cudaError_t launch_kernel(unsigned groups, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_out,
                                 const CUtensorMap& map_part, const GemmParams& P, cudaStream_t stream) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(groups * CTAS); cfg.blockDim = dim3(GEMM_THREADS);
    cfg.dynamicSmemBytes = gemm_smem<CTAS>(); cfg.stream = stream;
    cudaLaunchAttribute at[2];
    at[0].id = cudaLaunchAttributeClusterDimension; at[0].val.clusterDim.x = CTAS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization; at[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = pdl_allowed(stream) ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, gemm_i8_kernel<CTAS, KIND>, map_a, map_b, map_out, map_part, P);
}

srq_status_t launch_gemm_i8(const GemmArgs& g, uint32_t* status, cudaStream_t stream) {
    if (g.opt.accumulate == 2 && (g.acc_out == nullptr || g.kind != 0)) return SRQ_ERR_INVALID_ARG;   // int32 sums need their matrix
    if (g.opt.raw_sums && (g.kind != 0 || !g.out || g.acc_out || g.opt.accumulate || g.opt.out_bf16 || g.opt.requant || g.opt.absmax_bits))
        return SRQ_ERR_UNSUPPORTED;                       // the sums are the only result of such a call
    if (g.M == 0 || g.N == 0) return SRQ_OK;
    DeviceInfo* dev = nullptr;
    if (!device_info(&dev)) return SRQ_ERR_CUDA;
    const int ctas = (g.M > BM && dev->pairs > 0) ? 2 : 1;
    const int groups_max = ctas == 2 ? dev->pairs : dev->sms;

    CUtensorMap map_a, map_b;
    if (!encode_operand(&map_a, g.a, g.M, g.Kc, g.lda, BM)) return SRQ_ERR_CUDA;
    if (!encode_operand(&map_b, g.b, g.N, g.Kc, g.ldb, BN / ctas)) return SRQ_ERR_CUDA;

    GemmParams P;
    P.M = g.M; P.N = g.N;
    P.num_kb = (int32_t)((g.Kc + BK - 1) / BK);
    P.tiles_m = (int32_t)((g.M + BM * ctas - 1) / (BM * ctas));
    P.tiles_n = (int32_t)((g.N + BN - 1) / BN);
    const int64_t tiles = (int64_t)P.tiles_m * P.tiles_n;
    // binary32 accumulators do not add exactly: the E4M3 and bf16 products are never split; nor is a
    // product whose results are re-quantized or whose absmax is wanted (done in the epilogue)
    P.full_tiles = (int32_t)tiles; P.splits = 1;
    if (g.kind == 0 && !g.opt.requant && !g.opt.absmax_bits) plan_splits(tiles, P.num_kb, groups_max, &P.full_tiles, &P.splits);
    P.part = nullptr;
    const int64_t split_tiles = tiles - P.full_tiles;
    const size_t part_bytes = (size_t)split_tiles * BM * ctas * BN * 4;
    if (P.splits > 1) {
        if (g.splitk_ws == nullptr || g.splitk_ws_bytes < part_bytes || tiles * BM * ctas >= (1ll << 31)) {
            P.full_tiles = (int32_t)tiles; P.splits = 1;   // no room: run unsplit (same result)
        } else {
            P.part = (int32_t*)g.splitk_ws;
            if (cudaMemsetAsync(g.splitk_ws, 0, part_bytes, stream) != cudaSuccess) return SRQ_ERR_CUDA;
        }
    }
    P.s_row = g.s_row; P.row_stride = g.row_stride;
    P.s_col = g.s_col; P.col_stride = g.col_stride;
    P.out = g.out; P.ldo = g.ldo; P.acc_out = g.acc_out;
    P.status = status;
    P.timer = next_timer_slot();
    const int out_vec_elems = g.opt.out_bf16 ? 8 : 4;      // elements per 16 bytes of output
    P.vec_out = g.out && ((uintptr_t)g.out % 16 == 0) && (g.ldo % out_vec_elems == 0);

    // results leave through TMA stores when the output (and the partial sums) meet the 16-byte rules
    CUtensorMap map_out = map_a, map_part = map_a;       // placeholders when unused
    P.opt = g.opt;
    P.write_out = g.out != nullptr;
    P.rq_vec = g.opt.requant && ((uintptr_t)g.opt.rq_codes % 16 == 0) && (g.opt.rq_ld % 16 == 0);
    // (a row must also END on a 16-byte boundary: a store that reaches over the edge of the tensor map
    // was seen to write the whole last 16-byte piece of the row, into the columns of a wider buffer)
    P.tma_out = P.write_out && P.vec_out && g.N % out_vec_elems == 0 && !g.acc_out && g.M < (1ll << 31) && g.N < (1ll << 31) &&
                encode_output(&map_out, g.out, g.opt.out_bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : g.opt.raw_sums ? CU_TENSOR_MAP_DATA_TYPE_INT32 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, g.M, g.N, g.ldo);
    if (P.splits > 1 && !encode_output(&map_part, P.part, CU_TENSOR_MAP_DATA_TYPE_INT32, split_tiles * BM * ctas, BN, BN))
        return SRQ_ERR_CUDA;

    const int64_t units = P.full_tiles + split_tiles * P.splits;
    const unsigned groups = (unsigned)(units < groups_max ? units : groups_max);
    cudaError_t e;
    if (g.kind == 0) e = ctas == 2 ? launch_kernel<2, 0>(groups, map_a, map_b, map_out, map_part, P, stream)
                                   : launch_kernel<1, 0>(groups, map_a, map_b, map_out, map_part, P, stream);
    else if (g.kind == 1) e = ctas == 2 ? launch_kernel<2, 1>(groups, map_a, map_b, map_out, map_part, P, stream)
                                        : launch_kernel<1, 1>(groups, map_a, map_b, map_out, map_part, P, stream);
    else e = ctas == 2 ? launch_kernel<2, 2>(groups, map_a, map_b, map_out, map_part, P, stream)
                       : launch_kernel<1, 2>(groups, map_a, map_b, map_out, map_part, P, stream);
    count_launch();
    if (e != cudaSuccess) return SRQ_ERR_CUDA;
    if (P.splits > 1) {
        const int vec = g.ldo % 4 == 0 && (uintptr_t)g.out % 16 == 0;     // 16-byte (binary32) or 8-byte (bfloat16) stores
        const int64_t work = split_tiles * BM * ctas * (BN / 4);
        const int64_t blocks = (work + 255) / 256;
        const unsigned grid = (unsigned)(blocks < 8 * (int64_t)dev->sms ? blocks : 8 * (int64_t)dev->sms);
        launch_pdl(dequant_kernel, dim3(grid), dim3(256), 0, stream, P.part, split_tiles, P.full_tiles, P.tiles_n, BM * ctas, g.M, g.N, g.s_row,
                                                 g.row_stride, g.s_col, g.col_stride, g.out, g.ldo, g.acc_out, vec,
                                                 g.opt.accumulate, g.opt.out_bf16, g.opt.raw_sums, status);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return SRQ_ERR_CUDA;
    }
    return SRQ_OK;
}

}  // namespace srq
