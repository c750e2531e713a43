// Internal launcher declarations shared by the translation units of libgoq.
#pragma once
#include <cuda_runtime.h>
#include "goq_common.cuh"

namespace goq {

// GOQ_OK, or GOQ_ERR_CUDA after remembering the error for goq_last_cuda_error and clearing a non-sticky one.
goq_status status_from_cuda(cudaError_t e);

// The dynamic shared memory limit of a kernel is a per-device attribute: remember, per device, the largest size it
// has been raised to (one cache object per kernel instantiation, a function-local static at the call site).
struct SmemAttrCache { size_t set[64] = {}; };
template <class Kernel>
inline cudaError_t ensure_dynamic_smem(Kernel kernel, size_t smem, SmemAttrCache& cache) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    const bool tracked = dev >= 0 && dev < 64;
    if (tracked && smem <= cache.set[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess && tracked) cache.set[dev] = smem;
    return e;
}

cudaError_t launch_pack(const Geometry& g, const uint8_t* codes, const uint8_t* meta, const uint16_t* coef,
                        void* packed, cudaStream_t st);
cudaError_t launch_unpack(const Geometry& g, const void* packed, uint8_t* b1, uint8_t* b2, uint16_t* coef,
                          cudaStream_t st);

// Float-activation layer, scalar exponent-add kernel (any group size, batch <= 16).
cudaError_t launch_gemv_scalar(const Geometry& g, const void* packed, const void* x_bf16, int batch, void* y,
                               int y_dtype, cudaStream_t st);
// Float-activation layer, tensor-core fragment kernel (group >= 32); m may exceed 16.
cudaError_t launch_linear_mma(const Geometry& g, const void* packed, const void* x_bf16, int m, void* y,
                              int y_dtype, cudaStream_t st);
bool linear_mma_supported(const Geometry& g);

// Decode GEMV, streaming kernel (group >= 32, wbits <= 3, m <= 16). `ws` holds gemv_stream_workspace(g)
// bytes whose tile counters are zero on entry (goq_workspace_init) and are left zero on return.
bool gemv_stream_supported(const Geometry& g);
size_t gemv_stream_workspace(const Geometry& g);
size_t gemv_stream_zeroed_prefix(const Geometry& g);  // leading bytes of the scratch that must be zero on entry
bool stream_hash_is_bijective();
cudaError_t launch_gemv_stream(const Geometry& g, const void* packed, const void* x_bf16, int m, void* y, int y_dtype,
                               void* ws, cudaStream_t st);

// A chain of decode GEMVs in one persistent cooperative kernel (group >= 32, wbits <= 3, batch <= 8, the staged
// activations of each linear fit in shared memory; every linear has the same wbits and group). `ws` holds
// gemv_seq_workspace(n) bytes whose first gemv_seq_zeroed_prefix(n) bytes are zero on entry and left zero on return.
// spin_limit > 0 replaces the bound of every device-side wait (tests make waits run out with it).
constexpr int kSeqMaxItems = 256;
struct SeqCall {
    Geometry g;
    const void* packed;
    const void* x;
    void* y;
    int m, y_dtype, depends;
};
// Ordering of one item of a sequence launch, decided on the host from the address ranges
enum { kSeqOrderNone = 0, kSeqOrderData = 1, kSeqOrderBarrier = 2 };
struct SeqOrder {
    int kind;               // kSeqOrder...
    int source;             // kSeqOrderData: the earlier item whose output holds this item's activations
    unsigned word_offset;   // ... and where they start in that item's tagged copy (64-bit words)
};
void plan_sequence(const SeqCall* calls, int n, SeqOrder* out);
bool gemv_seq_supported(const Geometry& g, int m);
size_t gemv_seq_workspace(int n_items);
size_t gemv_seq_zeroed_prefix(int n_items);
cudaError_t launch_gemv_seq(const SeqCall* calls, int n, int wbits, int group, int unit_bytes, void* ws, int spin_limit,
                            cudaStream_t st);

// Prefill GEMM on tcgen05 tensor cores (wbits <= 3). `ws` holds gemm_tc_workspace(g, m) bytes: status word and
// (split-K) tile counters in the common areas, then the per-token scales, the fp16 copy of the m x k_in activations
// and the split-K partial tiles.
bool gemm_tc_supported(const Geometry& g);
size_t gemm_tc_workspace(const Geometry& g, int m);
cudaError_t launch_gemm_tc(const Geometry& g, const void* packed, const void* x_bf16, int m, void* y, int y_dtype,
                           void* ws, cudaStream_t st);

// Integer-activation layer.
// amax (optional, with y): per-token largest |y|, combined into the array with an integer max (zero it before the launch).
cudaError_t launch_gemm_a8(const Geometry& g, const void* packed, const int8_t* x, int m, const float* sx,
                           const int8_t* cq, const float* sc, void* y, int y_dtype, int32_t* acc, float* amax, cudaStream_t st);

// The steps before the inner product (goq_quant.cu).
cudaError_t launch_quantize_geo(const Geometry& g, const float* w, uint8_t* codes, uint8_t* meta, uint16_t* coef, cudaStream_t st);
cudaError_t launch_solve_ref(const Geometry& g, const float* w, const uint8_t* codes, const uint8_t* meta, const float* x_calib,
                             int m, double lambda, uint16_t* coef, double* c_out, cudaStream_t st);
cudaError_t launch_quantize_act(const void* x, int x_dtype, int m, int k, int abits, const float* amax, int8_t* xq, float* sx,
                                cudaStream_t st);

}  // namespace goq
