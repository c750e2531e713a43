// C ABI of libgoq: argument checks on the host, then one launcher per call.
#include <atomic>
#include <cstdlib>
#include <vector>
#include "goq_common.cuh"
#include "goq_internal.h"

using goq::Geometry;

namespace {

std::atomic<int> g_gemv_variant{0};
std::atomic<int> g_wait_limit{0};   // 0: the kernels' own bound on device-side waits
constexpr int kGemmViaGemvMaxTokens = 32;   // above: the tcgen05 GEMM (split-K) is faster than 16-token GEMV launches

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// compute capability 10.x of the current device, cached per device index
goq_status check_arch() {
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GOQ_ERR_CUDA;
    if (dev >= 0 && dev < 64) {
        int c = cached[dev].load(std::memory_order_relaxed);
        if (c == 1) return GOQ_OK;
        if (c == 2) return GOQ_ERR_ARCH;
    }
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GOQ_ERR_CUDA;
    const bool ok = (major == 10);
    if (dev >= 0 && dev < 64) cached[dev].store(ok ? 1 : 2, std::memory_order_relaxed);
    return ok ? GOQ_OK : GOQ_ERR_ARCH;
}

std::atomic<int> g_last_cuda_error{0};
goq_status from_cuda(cudaError_t e) { return goq::status_from_cuda(e); }

}  // namespace

namespace goq {
goq_status status_from_cuda(cudaError_t e) {
    if (e == cudaSuccess) return GOQ_OK;
    (void)cudaGetLastError();  // do not leave a non-sticky error behind for the next call to trip over
    g_last_cuda_error.store((int)e, std::memory_order_relaxed);
    return GOQ_ERR_CUDA;
}
}  // namespace goq

extern "C" {

const char* goq_status_string(goq_status s) {
    switch (s) {
        case GOQ_OK: return "ok";
        case GOQ_ERR_INVALID_ARG: return "invalid argument";
        case GOQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case GOQ_ERR_ALIGNMENT: return "misaligned pointer";
        case GOQ_ERR_WORKSPACE: return "buffer too small";
        case GOQ_ERR_OVERFLOW_BOUND: return "int32 accumulator bound exceeded";
        case GOQ_ERR_ARCH: return "device is not sm_100";
        case GOQ_ERR_CUDA: return "CUDA runtime error";
        case GOQ_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

size_t goq_packed_bytes(const goq_desc* desc) {
    Geometry g;
    return goq::make_geometry(desc, &g) ? g.total_bytes : 0;
}

size_t goq_algorithmic_bytes(const goq_desc* desc) {
    Geometry g;
    if (!goq::make_geometry(desc, &g)) return 0;
    if (g.k1) return (size_t)g.n_out * g.k_in * g.wbits / 8 + (size_t)g.n_out * (g.k_in / g.group) * 2;   // codes + one fp16 scale
    // (wbits + 0.75) bits per weight = (4*wbits + 3) / 32 bytes
    return (size_t)g.n_out * g.k_in * (4 * g.wbits + 3) / 32 + (size_t)g.n_out * (g.k_in / g.group) * 4;
}

size_t goq_workspace_bytes(const goq_desc* desc, int op, int m) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || m <= 0) return 0;
    if (op == GOQ_OP_GEMV && m <= 16) {
        size_t need = 0;
        if (goq::gemv_stream_supported(g)) need = goq::gemv_stream_workspace(g);
        if (m <= 4 && goq::gemv_seq_supported(g, m) && goq::gemv_seq_workspace(1) > need) need = goq::gemv_seq_workspace(1);
        return need;
    }
    if (op == GOQ_OP_GEMM) {
        // covers both kernels a call with these arguments may take (few tokens: the streaming GEMV, unless a variant is forced)
        size_t need = goq::gemm_tc_supported(g) ? goq::gemm_tc_workspace(g, m) : 0;
        if (m <= kGemmViaGemvMaxTokens && goq::gemv_stream_supported(g) && goq::gemv_stream_workspace(g) > need)
            need = goq::gemv_stream_workspace(g);
        return need;
    }
    return 0;
}

goq_status goq_pack(const goq_desc* desc, const uint8_t* codes, const uint8_t* meta, const uint16_t* coef_f16,
                    void* packed, size_t packed_bytes, void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !codes || !meta || !coef_f16 || !packed) return GOQ_ERR_INVALID_ARG;
    if (!aligned(packed, 128) || !aligned(coef_f16, 2)) return GOQ_ERR_ALIGNMENT;
    if (packed_bytes < g.total_bytes) return GOQ_ERR_WORKSPACE;
    if (goq_status s = check_arch()) return s;
    return from_cuda(goq::launch_pack(g, codes, meta, coef_f16, packed, (cudaStream_t)stream));
}

goq_status goq_unpack(const goq_desc* desc, const void* packed, uint8_t* codes_b1, uint8_t* codes_b2,
                      uint16_t* coef_f16, void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !packed) return GOQ_ERR_INVALID_ARG;
    if (!codes_b1 && !codes_b2 && !coef_f16) return GOQ_ERR_INVALID_ARG;
    if (!aligned(packed, 128) || !aligned(coef_f16, 2)) return GOQ_ERR_ALIGNMENT;
    if (goq_status s = check_arch()) return s;
    return from_cuda(goq::launch_unpack(g, packed, codes_b1, codes_b2, coef_f16, (cudaStream_t)stream));
}

goq_status goq_gemv(const goq_desc* desc, const void* packed, const void* x_bf16, int batch, void* y, int y_dtype,
                    void* ws, size_t ws_bytes, void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !packed || !x_bf16 || !y) return GOQ_ERR_INVALID_ARG;
    if (batch < 1 || batch > 16) return GOQ_ERR_INVALID_ARG;
    if (y_dtype != GOQ_BF16 && y_dtype != GOQ_F32) return GOQ_ERR_INVALID_ARG;
    if (!aligned(packed, 128) || !aligned(x_bf16, 16) || !aligned(y, y_dtype == GOQ_F32 ? 4 : 2))
        return GOQ_ERR_ALIGNMENT;
    if (goq_status s = check_arch()) return s;
    const int variant = g_gemv_variant.load(std::memory_order_relaxed);
    bool use_stream = goq::gemv_stream_supported(g) && (variant == 0 || variant == 3);
    if (variant == 3 && !use_stream) return GOQ_ERR_UNSUPPORTED;
    if (use_stream) {
        if (!ws || !aligned(ws, 256)) return ws ? GOQ_ERR_ALIGNMENT : GOQ_ERR_WORKSPACE;
        if (ws_bytes < goq::gemv_stream_workspace(g)) return GOQ_ERR_WORKSPACE;
        if (!goq::stream_hash_is_bijective()) return GOQ_ERR_UNSUPPORTED;
        // Up to 4 tokens whose activations fit the chain kernel's staging buffer: that kernel as a one-linear chain
        // is the faster one. A refused cooperative launch falls through to the streaming kernel.
        if (variant == 0 && batch <= 4 && goq::gemv_seq_supported(g, batch) && ws_bytes >= goq::gemv_seq_workspace(1)) {
            goq::SeqCall c{g, packed, x_bf16, y, batch, y_dtype, 0};
            if (goq::launch_gemv_seq(&c, 1, g.wbits, g.group, g.unit_bytes, ws, g_wait_limit.load(std::memory_order_relaxed),
                                     (cudaStream_t)stream) == cudaSuccess)
                return GOQ_OK;
            (void)cudaGetLastError();
        }
        return from_cuda(goq::launch_gemv_stream(g, packed, x_bf16, batch, y, y_dtype, ws, (cudaStream_t)stream));
    }
    bool use_mma = goq::linear_mma_supported(g);
    if (variant == 1) use_mma = false;
    if (variant == 2 && !use_mma) return GOQ_ERR_UNSUPPORTED;
    if (use_mma) return from_cuda(goq::launch_linear_mma(g, packed, x_bf16, batch, y, y_dtype, (cudaStream_t)stream));
    return from_cuda(goq::launch_gemv_scalar(g, packed, x_bf16, batch, y, y_dtype, (cudaStream_t)stream));
}

goq_status goq_gemm(const goq_desc* desc, const void* packed, const void* x, int m, int x_dtype, const float* sx,
                    const int8_t* cq, const float* sc, void* y, int y_dtype, int32_t* acc, void* ws, size_t ws_bytes,
                    void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !packed || !x || m < 1) return GOQ_ERR_INVALID_ARG;
    if (y && y_dtype != GOQ_BF16 && y_dtype != GOQ_F32) return GOQ_ERR_INVALID_ARG;
    if (!aligned(packed, 128) || !aligned(x, 16)) return GOQ_ERR_ALIGNMENT;
    if (y && !aligned(y, y_dtype == GOQ_F32 ? 4 : 2)) return GOQ_ERR_ALIGNMENT;
    if (x_dtype == GOQ_BF16) {
        if (!y) return GOQ_ERR_INVALID_ARG;
        if (goq_status s = check_arch()) return s;
        const int variant = g_gemv_variant.load(std::memory_order_relaxed);
        // Few tokens (17..32): the streaming GEMV kernel, 16 tokens per launch (36 us each on 8192 x 8192, so 72 us at
        // 32 tokens), against ~89 us for the tensor-core kernel with split-K, which takes over from 33 tokens.
        if (m <= kGemmViaGemvMaxTokens && variant == 0 && goq::gemv_stream_supported(g)) {
            if (!ws || !aligned(ws, 256)) return ws ? GOQ_ERR_ALIGNMENT : GOQ_ERR_WORKSPACE;
            if (ws_bytes < goq::gemv_stream_workspace(g)) return GOQ_ERR_WORKSPACE;
            if (!goq::stream_hash_is_bijective()) return GOQ_ERR_UNSUPPORTED;
            const size_t ybytes = (y_dtype == GOQ_F32) ? 4 : 2;
            for (int t0 = 0; t0 < m; t0 += 16) {
                const int nb = (m - t0 < 16) ? (m - t0) : 16;
                cudaError_t e = goq::launch_gemv_stream(g, packed, (const uint16_t*)x + (size_t)t0 * g.k_in, nb,
                                                        (uint8_t*)y + (size_t)t0 * g.n_out * ybytes, y_dtype, ws,
                                                        (cudaStream_t)stream);
                if (e != cudaSuccess) return from_cuda(e);
            }
            return GOQ_OK;
        }
        // W4 has no streaming GEMV: up to 32 tokens its mma.sync kernel is the faster one (41 us at 16 tokens on
        // 8192 x 8192 against ~92 us for the tensor-core kernel), so the tensor-core kernel takes W4 from 33 tokens on
        const bool w4_few = g.wbits == 4 && m <= kGemmViaGemvMaxTokens && variant == 0 && goq::linear_mma_supported(g);
        if (goq::gemm_tc_supported(g) && variant != 2 && !w4_few) {
            if (!ws || !aligned(ws, 256)) return ws ? GOQ_ERR_ALIGNMENT : GOQ_ERR_WORKSPACE;
            if (ws_bytes < goq::gemm_tc_workspace(g, m)) return GOQ_ERR_WORKSPACE;
            return from_cuda(goq::launch_gemm_tc(g, packed, x, m, y, y_dtype, ws, (cudaStream_t)stream));
        }
        if (goq::linear_mma_supported(g))
            return from_cuda(goq::launch_linear_mma(g, packed, x, m, y, y_dtype, (cudaStream_t)stream));
        // remaining configurations (macro-blocks narrower than 32): the scalar kernel, 16 tokens at a time
        const size_t ybytes = (y_dtype == GOQ_F32) ? 4 : 2;
        for (int t0 = 0; t0 < m; t0 += 16) {
            const int nb = (m - t0 < 16) ? (m - t0) : 16;
            cudaError_t e = goq::launch_gemv_scalar(g, packed, (const uint16_t*)x + (size_t)t0 * g.k_in, nb,
                                                    (uint8_t*)y + (size_t)t0 * g.n_out * ybytes, y_dtype,
                                                    (cudaStream_t)stream);
            if (e != cudaSuccess) return from_cuda(e);
        }
        return GOQ_OK;
    }
    if (x_dtype == GOQ_I8) {
        if (!cq || (!y && !acc)) return GOQ_ERR_INVALID_ARG;
        if (y && (!sx || !sc)) return GOQ_ERR_INVALID_ARG;
        if (!aligned(acc, 4) || !aligned(sx, 4) || !aligned(sc, 4) || !aligned(cq, 2)) return GOQ_ERR_ALIGNMENT;
        if (g.group < 16 || (g.k_in % 16)) return GOQ_ERR_UNSUPPORTED;
        // |ACC| <= k_in * 127 (x~) * 127 (c~) * 2^emax must stay below 2^31
        const long long bound = (long long)g.k_in * 127 * 127 * (1ll << ((1 << (g.wbits - 1)) - 1));
        if (bound >= (1ll << 31)) return GOQ_ERR_OVERFLOW_BOUND;
        if (goq_status s = check_arch()) return s;
        return from_cuda(goq::launch_gemm_a8(g, packed, (const int8_t*)x, m, sx, cq, sc, y, y_dtype, acc, nullptr,
                                             (cudaStream_t)stream));
    }
    return GOQ_ERR_INVALID_ARG;
}

goq_status goq_gemm_i8_requant(const goq_desc* desc, const void* packed, const int8_t* x, int m, const float* sx,
                               const int8_t* cq, const float* sc, float* y, float* amax, int8_t* yq, float* sy, void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !packed || !x || m < 1 || !sx || !cq || !sc || !y || !amax) return GOQ_ERR_INVALID_ARG;
    if ((yq == nullptr) != (sy == nullptr)) return GOQ_ERR_INVALID_ARG;
    if (!aligned(packed, 128) || !aligned(x, 16) || !aligned(y, 4) || !aligned(amax, 4) || !aligned(sx, 4) || !aligned(sc, 4) ||
        !aligned(cq, 2) || !aligned(sy, 4))
        return GOQ_ERR_ALIGNMENT;
    if (g.group < 16 || (g.k_in % 16)) return GOQ_ERR_UNSUPPORTED;
    const long long bound = (long long)g.k_in * 127 * 127 * (1ll << ((1 << (g.wbits - 1)) - 1));
    if (bound >= (1ll << 31)) return GOQ_ERR_OVERFLOW_BOUND;
    if (goq_status s = check_arch()) return s;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaError_t e = cudaMemsetAsync(amax, 0, (size_t)m * sizeof(float), st)) return from_cuda(e);
    if (cudaError_t e = goq::launch_gemm_a8(g, packed, x, m, sx, cq, sc, y, GOQ_F32, nullptr, amax, st)) return from_cuda(e);
    if (yq) return from_cuda(goq::launch_quantize_act(y, GOQ_F32, m, g.n_out, 8, amax, yq, sy, st));
    return GOQ_OK;
}

goq_status goq_quantize_activations(const void* x, int x_dtype, int m, int k, int abits, const float* amax, int8_t* xq,
                                    float* sx, void* stream) {
    if (!x || !xq || !sx || m < 1 || k < 1 || abits < 2 || abits > 8) return GOQ_ERR_INVALID_ARG;
    if (x_dtype != GOQ_F32 && x_dtype != GOQ_BF16) return GOQ_ERR_INVALID_ARG;
    if (!aligned(x, x_dtype == GOQ_F32 ? 4 : 2) || !aligned(sx, 4) || !aligned(amax, 4)) return GOQ_ERR_ALIGNMENT;
    if (goq_status s = check_arch()) return s;
    return from_cuda(goq::launch_quantize_act(x, x_dtype, m, k, abits, amax, xq, sx, (cudaStream_t)stream));
}

goq_status goq_quantize_geo(const goq_desc* desc, const float* w, uint8_t* codes, uint8_t* meta, uint16_t* coef_f16,
                            void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !w || !codes || !meta || !coef_f16) return GOQ_ERR_INVALID_ARG;
    if (!aligned(w, 16) || !aligned(codes, 4) || !aligned(coef_f16, 2)) return GOQ_ERR_ALIGNMENT;
    if (goq_status s = check_arch()) return s;
    return from_cuda(goq::launch_quantize_geo(g, w, codes, meta, coef_f16, (cudaStream_t)stream));
}

goq_status goq_solve_ref(const goq_desc* desc, const float* w, const uint8_t* codes, const uint8_t* meta,
                         const float* x_calib, int m, double lambda, uint16_t* coef_f16, double* c_f64, void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !w || !codes || !meta || !x_calib || !coef_f16 || m < 1 || !(lambda >= 0.0))
        return GOQ_ERR_INVALID_ARG;
    if (g.k1) return GOQ_ERR_UNSUPPORTED;
    if (!aligned(w, 4) || !aligned(x_calib, 4) || !aligned(coef_f16, 2) || !aligned(c_f64, 8)) return GOQ_ERR_ALIGNMENT;
    if (goq_status s = check_arch()) return s;
    return from_cuda(goq::launch_solve_ref(g, w, codes, meta, x_calib, m, lambda, coef_f16, c_f64, (cudaStream_t)stream));
}

size_t goq_sequence_workspace_bytes(int n_items) { return n_items > 0 ? goq::gemv_seq_workspace(n_items) : 0; }

goq_status goq_gemv_sequence(const goq_gemv_item* items, int n_items, void* ws, size_t ws_bytes, void* stream) {
    if (!items || n_items < 1) return GOQ_ERR_INVALID_ARG;
    static thread_local std::vector<goq::SeqCall> calls;
    calls.resize((size_t)n_items);
    for (int i = 0; i < n_items; ++i) {
        const goq_gemv_item& it = items[i];
        goq::SeqCall& c = calls[(size_t)i];
        if (!goq::make_geometry(&it.desc, &c.g) || !it.packed || !it.x_bf16 || !it.y) return GOQ_ERR_INVALID_ARG;
        if (it.batch < 1 || it.batch > 16) return GOQ_ERR_INVALID_ARG;
        if (it.y_dtype != GOQ_BF16 && it.y_dtype != GOQ_F32) return GOQ_ERR_INVALID_ARG;
        if (!aligned(it.packed, 128) || !aligned(it.x_bf16, 16) || !aligned(it.y, it.y_dtype == GOQ_F32 ? 4 : 2))
            return GOQ_ERR_ALIGNMENT;
        if (!goq::gemv_seq_supported(c.g, it.batch)) return GOQ_ERR_UNSUPPORTED;
        if (c.g.wbits != calls[0].g.wbits || c.g.group != calls[0].g.group) return GOQ_ERR_UNSUPPORTED;
        c.packed = it.packed; c.x = it.x_bf16; c.y = it.y; c.m = it.batch; c.y_dtype = it.y_dtype; c.depends = it.depends ? 1 : 0;
    }
    if (!ws || !aligned(ws, 256)) return ws ? GOQ_ERR_ALIGNMENT : GOQ_ERR_WORKSPACE;
    if (ws_bytes < goq::gemv_seq_workspace(n_items)) return GOQ_ERR_WORKSPACE;
    if (goq_status s = check_arch()) return s;
    if (!goq::stream_hash_is_bijective()) return GOQ_ERR_UNSUPPORTED;
    for (int i0 = 0; i0 < n_items; i0 += goq::kSeqMaxItems) {
        const int n = (n_items - i0 < goq::kSeqMaxItems) ? (n_items - i0) : goq::kSeqMaxItems;
        // a chunk boundary is a kernel boundary on the stream: the first item of a chunk needs no counter wait
        cudaError_t e = goq::launch_gemv_seq(&calls[(size_t)i0], n, calls[0].g.wbits, calls[0].g.group, calls[0].g.unit_bytes, ws,
                                             g_wait_limit.load(std::memory_order_relaxed), (cudaStream_t)stream);
        if (e != cudaSuccess) return from_cuda(e);
    }
    return GOQ_OK;
}

goq_status goq_sequence_order(const goq_gemv_item* items, int n_items, int32_t* kind_out, int32_t* source_out) {
    if (!items || n_items < 1 || !kind_out) return GOQ_ERR_INVALID_ARG;
    std::vector<goq::SeqCall> calls((size_t)n_items);
    for (int i = 0; i < n_items; ++i) {
        const goq_gemv_item& it = items[i];
        goq::SeqCall& c = calls[(size_t)i];
        if (!goq::make_geometry(&it.desc, &c.g) || !it.x_bf16 || !it.y || it.batch < 1) return GOQ_ERR_INVALID_ARG;
        if (it.y_dtype != GOQ_BF16 && it.y_dtype != GOQ_F32) return GOQ_ERR_INVALID_ARG;
        c.packed = it.packed; c.x = it.x_bf16; c.y = it.y; c.m = it.batch; c.y_dtype = it.y_dtype; c.depends = it.depends ? 1 : 0;
    }
    std::vector<goq::SeqOrder> order((size_t)n_items);
    // a launch holds at most kSeqMaxItems items: a later chunk starts after the earlier ones have completed
    for (int i0 = 0; i0 < n_items; i0 += goq::kSeqMaxItems) {
        const int n = (n_items - i0 < goq::kSeqMaxItems) ? (n_items - i0) : goq::kSeqMaxItems;
        goq::plan_sequence(&calls[(size_t)i0], n, &order[(size_t)i0]);
        for (int j = 0; j < n; ++j) {
            kind_out[i0 + j] = order[(size_t)(i0 + j)].kind;
            if (source_out) source_out[i0 + j] = order[(size_t)(i0 + j)].source < 0 ? -1 : i0 + order[(size_t)(i0 + j)].source;
        }
    }
    return GOQ_OK;
}

goq_status goq_gemv_sequence_host(const goq_gemv_item* items, int n_items, const void* x_host, void* x_stage,
                                  size_t x_bytes, void* y_host, void* y_stage, size_t y_bytes, void* ws,
                                  size_t ws_bytes, void* stream) {
    if (!items || n_items < 1 || !x_host || !x_stage || !y_host || !y_stage || !x_bytes || !y_bytes) return GOQ_ERR_INVALID_ARG;
    const uintptr_t xs = (uintptr_t)x_stage, ys = (uintptr_t)y_stage;
    for (int i = 0; i < n_items; ++i) {
        const goq_gemv_item& it = items[i];
        if (it.batch < 1 || it.desc.k_in <= 0 || it.desc.n_out <= 0) return GOQ_ERR_INVALID_ARG;
        const size_t xb = (size_t)it.batch * it.desc.k_in * 2;
        const size_t yb = (size_t)it.batch * it.desc.n_out * (it.y_dtype == GOQ_F32 ? 4 : 2);
        const uintptr_t x = (uintptr_t)it.x_bf16, y = (uintptr_t)it.y;
        const bool x_in_x = x >= xs && x + xb <= xs + x_bytes, x_in_y = x >= ys && x + xb <= ys + y_bytes;
        if (!(x_in_x || (x_in_y && i > 0)) || !(y >= ys && y + yb <= ys + y_bytes)) return GOQ_ERR_INVALID_ARG;
    }
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(x_stage, x_host, x_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return from_cuda(cudaGetLastError());
    goq_status s = goq_gemv_sequence(items, n_items, ws, ws_bytes, stream);
    if (s != GOQ_OK) return s;
    if (cudaMemcpyAsync(y_host, y_stage, y_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return from_cuda(cudaGetLastError());
    return GOQ_OK;
}

goq_status goq_gemv_host(const goq_desc* desc, const void* packed, const void* x_host, int batch, void* y_host,
                         int y_dtype, void* x_stage, void* y_stage, void* ws, size_t ws_bytes, void* stream) {
    Geometry g;
    if (!goq::make_geometry(desc, &g) || !x_host || !y_host || !x_stage || !y_stage) return GOQ_ERR_INVALID_ARG;
    if (batch < 1 || batch > 16) return GOQ_ERR_INVALID_ARG;
    if (y_dtype != GOQ_BF16 && y_dtype != GOQ_F32) return GOQ_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t xb = (size_t)batch * g.k_in * 2, yb = (size_t)batch * g.n_out * (y_dtype == GOQ_F32 ? 4 : 2);
    if (cudaMemcpyAsync(x_stage, x_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return GOQ_ERR_CUDA;
    goq_status s = goq_gemv(desc, packed, x_stage, batch, y_stage, y_dtype, ws, ws_bytes, stream);
    if (s != GOQ_OK) return s;
    if (cudaMemcpyAsync(y_host, y_stage, yb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return GOQ_ERR_CUDA;
    return GOQ_OK;
}

goq_status goq_workspace_init(void* ws, size_t ws_bytes, void* stream) {
    if (!ws || ws_bytes == 0) return GOQ_ERR_INVALID_ARG;
    return from_cuda(cudaMemsetAsync(ws, 0, ws_bytes, (cudaStream_t)stream));
}

goq_status goq_workspace_status(const void* ws, void* stream, int* status_out) {
    if (!ws || !status_out) return GOQ_ERR_INVALID_ARG;
    int v = 0;
    if (cudaMemcpyAsync(&v, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess)
        return GOQ_ERR_CUDA;
    if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return GOQ_ERR_CUDA;
    *status_out = v;
    return GOQ_OK;
}

int goq_last_cuda_error(void) { return g_last_cuda_error.load(std::memory_order_relaxed); }

int goq_set_gemv_variant(int variant) { return g_gemv_variant.exchange(variant); }

int goq_set_wait_limit(int polls) { return g_wait_limit.exchange(polls > 0 ? polls : 0); }

}  // extern "C"
