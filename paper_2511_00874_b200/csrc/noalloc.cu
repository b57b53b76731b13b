// sr_quantize_static: the quantizer for callers that cannot obtain device memory.
//
// sr_quantize needs a few words of scratch per scale group (absmax bit patterns and reciprocal
// step sizes) and normally carves them from a workspace the caller allocated.  Some callers have
// no way to allocate: code running inside a memory pool that is already fully handed out, a
// plug-in that is only ever given its input and output tensors, a real-time loop in which
// cudaMalloc's implicit synchronisation is not acceptable.  For them the scratch lives in the
// fixed array below, which is part of the library image: every device that loads the library
// reserves it once, for the life of the process, and nothing is allocated at call time.
//
// Consequences of the scratch being one shared array per device:
//   - inputs whose scratch does not fit in it are refused (SRQ_ERR_WORKSPACE);
//   - the array still holds whatever the previous call left there, so each call clears the words
//     that must start at zero before its kernels use them;
//   - two calls whose kernels can overlap on one device (different streams, no ordering between
//     them) race on the array; order them, or use sr_quantize with separate workspaces.
#include <mutex>

#include "common.cuh"

using namespace srq;

namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;   // 1 MiB, see sr_quantize_static in srq.h

// In host code this name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device code may name the array directly: clears the status word kept in its first bytes.
__global__ void clear_static_status() { reinterpret_cast<WsHeader*>(g_static_scratch)->status = 0u; }

constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the array on the current device, looked up once per device.
cudaError_t static_scratch(void** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        if (!p) return cudaErrorInvalidSymbol;
        g_scratch_ptr[dev] = p;
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" srq_status_t sr_quantize_static(const void* x, srq_dtype_t dt, int64_t rows, int64_t cols, int64_t ld,
                                           const srq_qspec_t* q, int8_t* codes_rm, int64_t ld_rm, float* scale_rm,
                                           int8_t* codes_tr, int64_t ld_tr, float* scale_tr, uint32_t* device_status,
                                           void* cuda_stream) {
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (!x || rows < 0 || cols < 0 || ld < cols) return SRQ_ERR_INVALID_ARG;
    if (dt != SRQ_F32 && dt != SRQ_BF16) return SRQ_ERR_INVALID_ARG;
    const srq_status_t sq = check_qspec(q);            // the same rules as sr_quantize: grid, widths, modes, absmax pointer
    if (sq != SRQ_OK) return sq;
    if (!codes_rm && !codes_tr) return SRQ_ERR_INVALID_ARG;
    if (codes_rm && (!scale_rm || ld_rm < cols)) return SRQ_ERR_INVALID_ARG;
    if (codes_tr && (!scale_tr || ld_tr < rows)) return SRQ_ERR_INVALID_ARG;
    if ((uintptr_t)x % 16 != 0 || (uintptr_t)device_status % 4 != 0) return SRQ_ERR_INVALID_ARG;
    // the first 256 bytes of the array hold the status word when the caller passes none
    if (sizeof(WsHeader) + quant_scratch_bytes(rows, cols) > kStaticScratchBytes) return SRQ_ERR_WORKSPACE;
    if (rows == 0 || cols == 0) return SRQ_OK;

    void* base = nullptr;
    if (static_scratch(&base) != cudaSuccess) return SRQ_ERR_CUDA;
    uint32_t* status = device_status ? device_status : &((WsHeader*)base)->status;
    if (device_status) {
        if (cudaMemsetAsync(status, 0, sizeof(uint32_t), st) != cudaSuccess) return SRQ_ERR_CUDA;
    } else {
        clear_static_status<<<1, 1, 0, st>>>();
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return SRQ_ERR_CUDA;
    }

    QuantArgs a;
    a.x = x; a.dt = dt; a.rows = rows; a.cols = cols; a.ld = ld; a.q = *q;
    a.codes_rm = codes_rm; a.ld_rm = ld_rm; a.scale_rm = scale_rm;
    a.codes_tr = codes_tr; a.ld_tr = ld_tr; a.scale_tr = scale_tr;
    // launch_quantize zeroes the absmax words of this call's groups before the reduction runs
    const QuantScratch sc = carve_quant_scratch((char*)base + sizeof(WsHeader), rows, cols);
    return launch_quantize(a, sc, status, st) == cudaSuccess ? SRQ_OK : SRQ_ERR_CUDA;
}
