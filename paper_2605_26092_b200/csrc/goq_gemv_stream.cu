// Decode GEMV (batch <= 16), streaming kernel.
//
// Eq. 4 of the paper read per macro-block:  y[m,n] = sum_j ( c1[n,j] S1 + c2[n,j] S2 ),
// S1 = sum_{k in j} b1[n,k] x[m,k], S2 likewise with b2. b1 and b2 enter the bf16 tensor-core MMA as
// exact PoT operands (a PoT factor only shifts the activation's exponent, so no product rounds), the
// sums are fp32, and the coefficient multiply happens once per macro-block outside the MMA.
//
// Work decomposition. The packed buffer is one contiguous array of unit records (1 KiB of codes plus
// the coefficients of 16 rows x 128 k). CTA i takes the contiguous range [U*i/G, U*(i+1)/G) of the U
// records, so every SM streams the same number of bytes whatever the shape. A producer thread moves the
// range through a ring of shared-memory stages with 1-D bulk async copies (mbarrier completion); eight
// consumer warps each take one record per stage. Lane (g,t) of a consumer owns whole micro-blocks of
// rows g and g+8, so the Strided Dual-Exchange of Section 3.3 never leaves the thread. A 16-row tile
// that straddles CTAs is finished by whichever CTA arrives last, adding the parked partial sums in CTA
// order: results do not depend on timing. The weight prefetch starts before the wait on the preceding
// kernel in the stream (programmatic dependent launch); activations, outputs and the scratch buffer are
// touched only after it.
//
// Every mbarrier wait is bounded. On expiry the CTA raises an abort flag, records GOQ_ERR_TIMEOUT in
// the scratch status word and runs out its control flow (all barriers are still reached) without
// touching data.
#include "goq_stream_core.cuh"
#include "goq_internal.h"

namespace goq {

// ------------------------------------------------------------------------------------------------
// scratch layout: [status 256 B][tile counters, in the common counter area][partials kMaxCtas x 2 x 256 floats]
// ------------------------------------------------------------------------------------------------
constexpr int kMaxCtas = 512;
constexpr int kStatusBytes = 256;
constexpr int kPartialFloats = 16 * 16;  // one 16-row tile x up to 16 tokens

struct StreamWs {
    size_t counters_off, partials_off, total;
};
__host__ inline StreamWs stream_ws_layout(const Geometry& g) {
    StreamWs w;
    w.counters_off = kStatusBytes;
    w.partials_off = kWsScratchOff;
    w.total = w.partials_off + (size_t)kMaxCtas * 2 * kPartialFloats * sizeof(float);
    return w;
}

// ------------------------------------------------------------------------------------------------
// streaming kernel
// ------------------------------------------------------------------------------------------------
constexpr int kConsumerWarps = 16;
constexpr int kStreamThreads = (kConsumerWarps + 1) * 32;
constexpr int kStageUnits = kConsumerWarps;
__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); }

struct StreamParams {
    const uint8_t* packed;
    const uint16_t* x;
    void* y;
    int* status;
    int* counters;
    float* partials;
    int n_units, unit_bytes, k_blocks, k_in, n_out, m_total, y_dtype, n_stages;
    int x_smem_bytes;  // > 0: the activations (m_total x k_in bf16) are staged in shared memory once per CTA
};

__device__ __forceinline__ int owner_of_unit(int u, int n_units, int n_ctas) {
    return (int)((((long long)u + 1) * n_ctas - 1) / n_units);
}
__device__ __forceinline__ int range_begin(int i, int n_units, int n_ctas) {
    return (int)((long long)n_units * i / n_ctas);
}

constexpr int kRedSlots = 2;  // ring of per-tile reduction buffers inside a CTA

// WB: weight bits (2, 3); NT: 8-token column tiles (1, 2); CPG: 32-wide chunks per macro-block (1, 2, 4)
// XS: activations staged in shared memory (small batches) or read from global memory
template <int WB, int NT, int CPG, bool XS>
__global__ void __launch_bounds__(kStreamThreads, (NT == 1) ? 2 : 1) gemv_stream_kernel(const StreamParams p) {
    extern __shared__ __align__(128) unsigned char smem[];
    // carve-up: [ring stages][red: kRedSlots x warps x 32 lanes x NT*4 floats][barriers][activations]
    // The record table (8 bank-disjoint copies, 8 KiB) sits at the first 8 KiB boundary of the dynamic
    // shared memory so that a slot offset can be OR-ed into its address; the launch reserves the slack.
    unsigned char* lut = smem + ((8192u - (smem_u32(smem) & 8191u)) & 8191u);
    const int stage_bytes = kStageUnits * p.unit_bytes;
    unsigned char* ring = lut + kLutBytes;
    float* red = reinterpret_cast<float*>(ring + (size_t)p.n_stages * stage_bytes);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(red + kRedSlots * kConsumerWarps * 32 * NT * 4);
    uint64_t* empty_bar = full_bar + p.n_stages;
    uint64_t* x_bar = empty_bar + p.n_stages;
    const uint16_t* xs = reinterpret_cast<const uint16_t*>(x_bar + 2);  // 16-byte aligned: barriers come in pairs
    __shared__ volatile int abort_flag;
    __shared__ int arrive_cnt[kRedSlots];  // warps that have parked their sums for the tile using the slot
    __shared__ int done_gen[kRedSlots];    // 1 + local index of the last tile fully reduced out of the slot

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_ctas = gridDim.x;
    const int u_begin = range_begin(blockIdx.x, p.n_units, n_ctas), u_end = range_begin(blockIdx.x + 1, p.n_units, n_ctas);
    const int my_units = u_end - u_begin;
    const int my_stages = (my_units + kStageUnits - 1) / kStageUnits;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < kRedSlots; ++i) { arrive_cnt[i] = 0; done_gen[i] = 0; }
        for (int s = 0; s < p.n_stages; ++s) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], kConsumerWarps);
        }
        mbar_init(x_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // the next kernel in the stream may begin its own prologue and weight prefetch
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == kConsumerWarps) {
        // ---------------- producer: one thread streams this CTA's records through the ring -------------
        if (lane == 0) {
            const uint8_t* src = p.packed + (size_t)u_begin * p.unit_bytes;
            int slot = 0, round = 0;
            bool x_issued = (p.x_smem_bytes == 0);
            int issued = 0;
            for (int s = 0; s < my_stages; ++s) {
                if (round > 0) {
                    if (!mbar_wait_bounded(&empty_bar[slot], (round - 1) & 1, &abort_flag)) break;
                }
                issued = s + 1;
                const int units = min(kStageUnits, my_units - s * kStageUnits);
                const uint32_t bytes = (uint32_t)units * p.unit_bytes;
                mbar_arrive_expect_tx(&full_bar[slot], bytes);
                bulk_copy_g2s(ring + (size_t)slot * stage_bytes, src + (size_t)s * stage_bytes, bytes, &full_bar[slot]);
                if (++slot == p.n_stages) { slot = 0; ++round; }
                if (!x_issued && (s + 1 == my_stages || s + 1 == p.n_stages)) {
                    // the ring is primed: now the activations, which the preceding kernel may have produced
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    const uint32_t row_bytes = (uint32_t)p.k_in * 2;
                    mbar_arrive_expect_tx(x_bar, row_bytes * p.m_total);
                    for (int r = 0; r < p.m_total; ++r)
                        bulk_copy_g2s(const_cast<uint16_t*>(xs) + (size_t)r * p.k_blocks * kBlockK, p.x + (size_t)r * p.k_in,
                                      row_bytes, x_bar);
                    x_issued = true;
                }
            }
            if (abort_flag) drain_issued_stages(full_bar, issued, p.n_stages);
        }
        return;
    }

    // ---------------- consumers ---------------------------------------------------------------------
    // replicate the record table (8 bank-disjoint copies), while the first stages are in flight
    for (int i = tid; i < 64 * kLutCopies; i += kConsumerWarps * 32) {
        const uint32_t* e = c_exchange_lut.v[i / kLutCopies];
        *reinterpret_cast<uint4*>(lut + (size_t)i * 16) = make_uint4(e[0], e[1], e[2], e[3]);
    }
    if (p.x_smem_bytes) {  // zero the padding [k_in, k_pad) of every staged activation row
        const int kp = p.k_blocks * kBlockK, tail = kp - p.k_in;
        uint16_t* xw = const_cast<uint16_t*>(xs);
        for (int i = tid; i < tail * p.m_total; i += kConsumerWarps * 32) xw[(size_t)(i / tail) * kp + p.k_in + (i % tail)] = 0;
    }
    consumer_bar_sync();

    const int g = lane >> 2, t = lane & 3;
    const uint32_t lut_lane = smem_u32(lut) + (lane & (kLutCopies - 1)) * 16;
    const int k_blocks = p.k_blocks;
    const int k_pad = k_blocks * kBlockK;

    // everything below reads activations or writes outputs / scratch: wait for the preceding kernel
    asm volatile("griddepcontrol.wait;" ::: "memory");

    // per-lane activation row (token nt*8+g). Lanes whose token does not exist read the last token's
    // row instead of zeros: an MMA output column depends only on its own B column, and columns of
    // missing tokens are never stored.
    const uint16_t* xrow[NT];
    uint32_t xrow_s[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int row = min(nt * 8 + g, p.m_total - 1);
        xrow[nt] = p.x + (size_t)row * p.k_in + t * 8;
        xrow_s[nt] = smem_u32(xs) + (uint32_t)(row * k_pad + t * 8) * 2;
    }
    constexpr bool x_staged = XS;
    const bool k_ragged = (p.k_in & (kBlockK - 1)) != 0;  // the last k-block is partly padding
    if (x_staged) {
        mbar_wait_bounded(x_bar, 0, &abort_flag);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) xrow_s[nt] = order_after_wait(xrow_s[nt]);
    }
    // This warp takes records u_begin + warp, + 8, ... (record i of the range sits in stage i / 8).
    const int tile_first = (my_units > 0) ? u_begin / k_blocks : 0;
    int slot = 0, phase = 0;
    int T = -1, tile_u0 = 0, tile_u1 = 0;  // tile of the sums currently held in acc
    float acc[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[nt][r] = 0.f;

    for (int i = warp;; i += kStageUnits) {
        const int u = u_begin + i;
        const bool more = (i < my_units) && (abort_flag == 0);
        const int Tn = more ? u / k_blocks : -1;
        if (Tn != T && T >= 0) {
            {
                // ---- park this warp's sums for tile T; the last warp to do so finishes the tile ----
                const int lt = T - tile_first, rs = lt % kRedSlots;
                const int a = max(u_begin, tile_u0) - u_begin, b = min(u_end, tile_u1) - u_begin;  // range-relative segment
                const int contributors = min(kConsumerWarps, b - a);
                bool ok = true;
                if (lt >= kRedSlots) {  // the slot's previous tile must be fully reduced
                    volatile int* dg = &done_gen[rs];
                    int it = 0;
                    while (*dg != lt - kRedSlots + 1) {
                        if (abort_flag || ++it > kSpinLimit) { abort_flag = 1; ok = false; break; }
                        __nanosleep(40);
                    }
                }
                if (ok) {
                    float* rb = red + (size_t)rs * kConsumerWarps * 32 * NT * 4;
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                        for (int r = 0; r < 4; ++r) rb[(warp * 32 + lane) * (NT * 4) + nt * 4 + r] = acc[nt][r];
                    __threadfence_block();
                    __syncwarp();
                    int old = 0;
                    if (lane == 0) old = atomicAdd(&arrive_cnt[rs], 1);
                    old = __shfl_sync(0xFFFFFFFFu, old, 0);
                    if (old == contributors - 1) {
                        __threadfence_block();
                        float out[NT * 4];
#pragma unroll
                        for (int q = 0; q < NT * 4; ++q) out[q] = 0.f;
                        for (int w = 0; w < kConsumerWarps; ++w) {
                            // warp w holds a record of the segment iff some i in [a, b) has i % 16 == w
                            const int first = a + ((w - a) & (kStageUnits - 1));
                            if (first < b) {
#pragma unroll
                                for (int q = 0; q < NT * 4; ++q) out[q] += rb[(w * 32 + lane) * (NT * 4) + q];
                            }
                        }
                        const bool full_tile = (a + u_begin == tile_u0) && (b + u_begin == tile_u1);
                        if (!full_tile) {
                            // park the CTA's sums; the CTA that arrives last at this tile adds them in CTA order
                            const int slot_id = (T == tile_first) ? 0 : 1;
                            float* mine_p = p.partials + ((size_t)blockIdx.x * 2 + slot_id) * kPartialFloats;
#pragma unroll
                            for (int q = 0; q < NT * 4; ++q) __stcg(mine_p + lane * (NT * 4) + q, out[q]);
                            __syncwarp();
                            const int i_lo = owner_of_unit(tile_u0, p.n_units, n_ctas);
                            const int i_hi = owner_of_unit(tile_u1 - 1, p.n_units, n_ctas);
                            int prev = 0;
                            if (lane == 0) prev = atomic_add_acq_rel_gpu(&p.counters[T], 1);
                            prev = __shfl_sync(0xFFFFFFFFu, prev, 0);
                            if (prev == i_hi - i_lo) {
#pragma unroll
                                for (int q = 0; q < NT * 4; ++q) out[q] = 0.f;
                                for (int c = i_lo; c <= i_hi; ++c) {
                                    const int first_tile_c = range_begin(c, p.n_units, n_ctas) / k_blocks;
                                    const float* pp = p.partials + ((size_t)c * 2 + ((T == first_tile_c) ? 0 : 1)) * kPartialFloats;
#pragma unroll
                                    for (int q = 0; q < NT * 4; ++q) out[q] += __ldcg(pp + lane * (NT * 4) + q);
                                }
                                if (lane == 0) p.counters[T] = 0;  // leave the scratch clean for the next call
                            } else {
                                T = -2;  // not the last CTA: nothing to store
                            }
                        }
                        if (T >= 0 && abort_flag == 0) {
#pragma unroll
                            for (int q = 0; q < NT * 4; ++q) {
                                const int nt = q >> 2, r = q & 3;
                                const int row = T * 16 + g + ((r & 2) ? 8 : 0);
                                const int tok = nt * 8 + t * 2 + (r & 1);
                                if (row < p.n_out && tok < p.m_total) {
                                    if (p.y_dtype == GOQ_F32) reinterpret_cast<float*>(p.y)[(size_t)tok * p.n_out + row] = out[q];
                                    else reinterpret_cast<uint16_t*>(p.y)[(size_t)tok * p.n_out + row] = f32_to_bf16_rne(out[q]);
                                }
                            }
                        }
                        __syncwarp();
                        if (lane == 0) {
                            arrive_cnt[rs] = 0;
                            __threadfence_block();
                            done_gen[rs] = lt + 1;
                        }
                    }
                }
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int r = 0; r < 4; ++r) acc[nt][r] = 0.f;
            }
        }
        if (!more) break;  // every path out of the loop: i only grows, so this is reached
        if (Tn != T) {
            T = Tn;
            tile_u0 = T * k_blocks;
            tile_u1 = tile_u0 + k_blocks;
        }

        if (mbar_wait_bounded(&full_bar[slot], phase, &abort_flag)) {
            const uint32_t unit = order_after_wait(smem_u32(ring) + slot * stage_bytes + warp * p.unit_bytes + lane * 16);
            const int kb0 = (u - tile_u0) * kBlockK;
            const uint4 wv0 = lds128(unit), wv1 = lds128(unit + 512);
            const uint32_t coef_addr = unit - lane * 16 + kCodeBytesPerUnit + g * 4;
            const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
            float d1[NT][4], d2[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int r = 0; r < 4; ++r) d1[nt][r] = d2[nt][r] = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int k0 = kb0 + c * 32;
                uint4 xa[NT];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    if constexpr (XS) {
                        xa[nt] = lds128(xrow_s[nt] + k0 * 2);  // rows are padded with zeros up to k_pad
                    } else {
                        // beyond k_in the weights are zero-valued padding: feed zeros
                        xa[nt] = make_uint4(0, 0, 0, 0);
                        if (!k_ragged || (k0 + t * 8) < p.k_in) xa[nt] = *reinterpret_cast<const uint4*>(xrow[nt] + k0);
                    }
                }
                uint32_t R0[4], Q0[4], R1[4], Q1[4];
                expand_word<WB>(w0[c], lut_lane, R0, Q0);
                expand_word<WB>(w1[c], lut_lane, R1, Q1);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16(d1[nt], R0[0], R1[0], R0[1], R1[1], xa[nt].x, xa[nt].y);
                    mma_bf16(d2[nt], Q0[0], Q1[0], Q0[1], Q1[1], xa[nt].x, xa[nt].y);
                    mma_bf16(d1[nt], R0[2], R1[2], R0[3], R1[3], xa[nt].z, xa[nt].w);
                    mma_bf16(d2[nt], Q0[2], Q1[2], Q0[3], Q1[3], xa[nt].z, xa[nt].w);
                }
                if (((c + 1) % CPG) == 0) {
                    const int jj = c / CPG;
                    const uint32_t cfa = lds32(coef_addr + jj * 64), cfb = lds32(coef_addr + jj * 64 + 32);
                    const float c1a = __half2float(__ushort_as_half((unsigned short)(cfa & 0xFFFFu)));
                    const float c2a = __half2float(__ushort_as_half((unsigned short)(cfa >> 16)));
                    const float c1b = __half2float(__ushort_as_half((unsigned short)(cfb & 0xFFFFu)));
                    const float c2b = __half2float(__ushort_as_half((unsigned short)(cfb >> 16)));
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) {
                        acc[nt][0] += c1a * d1[nt][0] + c2a * d2[nt][0];
                        acc[nt][1] += c1a * d1[nt][1] + c2a * d2[nt][1];
                        acc[nt][2] += c1b * d1[nt][2] + c2b * d2[nt][2];
                        acc[nt][3] += c1b * d1[nt][3] + c2b * d2[nt][3];
#pragma unroll
                        for (int r = 0; r < 4; ++r) d1[nt][r] = d2[nt][r] = 0.f;
                    }
                }
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[slot]);
        if (++slot == p.n_stages) { slot = 0; phase ^= 1; }
    }
    if (lane == 0 && abort_flag) atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
}

bool gemv_stream_supported(const Geometry& g) { return g.group >= 32 && g.wbits <= 3 && (size_t)g.n_tiles * 4 <= kWsCounterBytes; }

size_t gemv_stream_workspace(const Geometry& g) { return stream_ws_layout(g).total; }
size_t gemv_stream_zeroed_prefix(const Geometry& g) { return stream_ws_layout(g).counters_off + (size_t)g.n_tiles * 4; }

bool stream_hash_is_bijective() {
    bool seen[64] = {};
    for (uint32_t meta = 0; meta < 64; ++meta) {
        uint32_t s = record_slot(meta);
        if (seen[s]) return false;
        seen[s] = true;
    }
    return true;
}

static int sm_count() {
    static int cached[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (cached[dev] == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        cached[dev] = n > 0 ? n : 148;
    }
    return cached[dev];
}

bool g_stream_pdl = true;  // programmatic dependent launch on the streaming kernel
int g_stream_grid_per_sm = 0;  // 0: as many CTAs per SM as fit; 1: leave room for the next kernel's CTAs

template <int WB, int NT, int CPG>
static cudaError_t launch_stream(const Geometry& g, const StreamParams& p0, cudaStream_t st) {
    StreamParams p = p0;
    constexpr int kCtasPerSm = (NT == 1) ? 2 : 1;
    int grid = sm_count() * ((g_stream_grid_per_sm > 0 && g_stream_grid_per_sm < kCtasPerSm) ? g_stream_grid_per_sm : kCtasPerSm);
    if (grid > kMaxCtas) grid = kMaxCtas;
    if (grid > p.n_units) grid = p.n_units;
    // ring depth: what fits in ~70 KB, at most what one CTA will ever use
    const int stage_bytes = kStageUnits * g.unit_bytes;
    const int x_bytes = p.m_total * g.k_pad * 2;
    p.x_smem_bytes = (x_bytes <= 40 * 1024) ? x_bytes : 0;
    int n_stages = ((kCtasPerSm == 2 ? 56 : 100) * 1024) / stage_bytes;
    const int need = (p.n_units / grid + 1 + kStageUnits - 1) / kStageUnits + 1;
    if (n_stages > need) n_stages = need;
    if (n_stages < 2) n_stages = 2;
    p.n_stages = n_stages;
    const size_t smem = (size_t)2 * kLutBytes + (size_t)n_stages * stage_bytes +
                        (size_t)kRedSlots * kConsumerWarps * 32 * NT * 4 * sizeof(float) +
                        (size_t)(2 * n_stages + 2) * sizeof(uint64_t) + (size_t)p.x_smem_bytes;
    auto kernel = p.x_smem_bytes ? gemv_stream_kernel<WB, NT, CPG, true> : gemv_stream_kernel<WB, NT, CPG, false>;
    static SmemAttrCache smem_attr[2];
    if (cudaError_t e = ensure_dynamic_smem(kernel, 160 * 1024, smem_attr[p.x_smem_bytes ? 1 : 0])) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kStreamThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_stream_pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int WB, int NT>
static cudaError_t launch_stream_cpg(const Geometry& g, const StreamParams& p, cudaStream_t st) {
    switch (g.group) {
        case 32: return launch_stream<WB, NT, 1>(g, p, st);
        case 64: return launch_stream<WB, NT, 2>(g, p, st);
        default: return launch_stream<WB, NT, 4>(g, p, st);
    }
}

cudaError_t launch_gemv_stream(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype,
                               void* ws, cudaStream_t st) {
    const StreamWs L = stream_ws_layout(g);
    auto* wsb = (uint8_t*)ws;
    StreamParams p;
    p.packed = (const uint8_t*)packed;
    p.x = (const uint16_t*)x;
    p.y = y;
    p.status = (int*)wsb;
    p.counters = (int*)(wsb + L.counters_off);
    p.partials = (float*)(wsb + L.partials_off);
    p.n_units = (int)g.n_units;
    p.unit_bytes = g.unit_bytes;
    p.k_blocks = g.k_blocks;
    p.k_in = g.k_in;
    p.n_out = g.n_out;
    p.m_total = m;
    p.y_dtype = y_dtype;
    p.n_stages = 0;
    p.x_smem_bytes = 0;
    if (g.wbits == 3) return m <= 8 ? launch_stream_cpg<3, 1>(g, p, st) : launch_stream_cpg<3, 2>(g, p, st);
    return m <= 8 ? launch_stream_cpg<2, 1>(g, p, st) : launch_stream_cpg<2, 2>(g, p, st);
}

}  // namespace goq
