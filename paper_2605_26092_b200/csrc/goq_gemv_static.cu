// goq_gemv_static: the decode GEMV for callers that cannot provide scratch memory.
//
// goq_gemv needs a small scratch buffer (tile counters and parked partial sums for tiles that two CTAs
// share). Some callers have no way to get one: a plugin that runs inside an inference server which has
// already handed every byte of device memory to its own arena, a decode loop that must never hit the
// implicit device synchronisation of cudaMalloc / cudaFree, host code that has no torch (or other)
// allocator at hand. For them this file keeps one fixed scratch array inside the library image itself.
//
// The array is a file-scope __device__ array: every GPU that loads the library holds
// GOQ_STATIC_SCRATCH_BYTES of it until the process exits. In host code the array's name is only a
// host-side stand-in for the symbol, not a device address, so it is never passed to a kernel; its
// device address is looked up with cudaGetSymbolAddress, once per device, with that device current.
#include <mutex>
#include "goq_common.cuh"
#include "goq_internal.h"

namespace {

constexpr size_t kStaticScratchBytes = GOQ_STATIC_SCRATCH_BYTES;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];  // device address of g_static_scratch on each device, once known
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device (looked up on first use on that device).
goq_status static_scratch_address(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GOQ_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return GOQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        if (cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch)) return goq::status_from_cuda(e);
        if (!ptr) return GOQ_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return GOQ_OK;
}

bool ptr_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace

extern "C" goq_status goq_gemv_static(const goq_desc* desc, const void* packed, const void* x_bf16, int batch,
                                      void* y, int y_dtype, void* stream) {
    goq::Geometry g;
    if (!goq::make_geometry(desc, &g) || !packed || !x_bf16 || !y) return GOQ_ERR_INVALID_ARG;
    if (batch < 1 || batch > 16) return GOQ_ERR_INVALID_ARG;
    if (y_dtype != GOQ_BF16 && y_dtype != GOQ_F32) return GOQ_ERR_INVALID_ARG;
    if (!ptr_aligned(packed, 128) || !ptr_aligned(x_bf16, 16) || !ptr_aligned(y, y_dtype == GOQ_F32 ? 4 : 2))
        return GOQ_ERR_ALIGNMENT;
    if (!goq::gemv_stream_supported(g) || !goq::stream_hash_is_bijective()) return GOQ_ERR_UNSUPPORTED;
    const size_t need = goq::gemv_stream_workspace(g);
    if (need > kStaticScratchBytes) return GOQ_ERR_WORKSPACE;  // layer has too many 16-row tiles for the fixed array
    int major = 0, dev = 0;
    if (cudaError_t e = cudaGetDevice(&dev)) return goq::status_from_cuda(e);
    if (cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev)) return goq::status_from_cuda(e);
    if (major != 10) return GOQ_ERR_ARCH;
    void* scratch = nullptr;
    if (goq_status s = static_scratch_address(&scratch)) return s;
    cudaStream_t st = (cudaStream_t)stream;
    // The array keeps whatever the previous call left. The status word and the tile counters must start
    // at zero, so clear exactly that prefix; the parked partial sums behind it are always written before
    // they are read.
    if (cudaError_t e = cudaMemsetAsync(scratch, 0, goq::gemv_stream_zeroed_prefix(g), st)) return goq::status_from_cuda(e);
    return goq::status_from_cuda(goq::launch_gemv_stream(g, packed, x_bf16, batch, y, y_dtype, scratch, st));
}

extern "C" goq_status goq_gemv_static_status(void* stream, int* status_out) {
    if (!status_out) return GOQ_ERR_INVALID_ARG;
    void* scratch = nullptr;
    if (goq_status s = static_scratch_address(&scratch)) return s;
    int v = 0;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaError_t e = cudaMemcpyAsync(&v, scratch, sizeof(int), cudaMemcpyDeviceToHost, st)) return goq::status_from_cuda(e);
    if (cudaError_t e = cudaStreamSynchronize(st)) return goq::status_from_cuda(e);
    *status_out = v;
    return GOQ_OK;
}
