// A sequence of decode GEMVs (batch <= 8) in ONE persistent kernel.
//
// A decode step is a chain of small linears (Eq. 4 of the paper per layer): each streams a few MB of
// packed weights, far too little to hide a kernel's launch, prologue, first-byte latency and tail. Here the
// whole chain runs in one cooperative launch: every CTA stays resident, its producer thread keeps the
// weight stream going across the boundary between two linears (weights never depend on an earlier result),
// and a linear whose activations do depend on earlier outputs waits on a device-wide completion counter
// before it reads them - only that wait and the activation fetch are serial.
//
// Work unit = one 16-row tile of one linear, all of K (no split across CTAs, hence no partial-sum hand-off):
// tile number base_p + T goes to CTA (base_p + T) mod G. Inside the CTA the tile's unit records (16 rows x
// 128 k each, contiguous in the packed buffer) are streamed 16 at a time into a ring of shared-memory
// stages by 1-D bulk async copies; consumer warp w takes record w of each stage, so the warps split K. The
// math per record is that of the streaming kernel: b1 and b2 as exact bf16 PoT operands of mma.sync
// (the exchange of Section 3.3 stays inside a lane), fp32 sums, coefficient multiply once per macro-block.
// The last warp to finish a tile adds the 16 partial sums in warp order and stores the outputs.
//
// Every wait is bounded (mbarriers, the completion counters); on expiry the CTA raises an abort flag, keeps
// its control flow (all barriers are still reached), touches no more data and reports GOQ_ERR_TIMEOUT.
#include "goq_stream_core.cuh"
#include "goq_internal.h"

namespace goq {
namespace seq {

constexpr int kConsumerWarps = 16;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kStageUnits = kConsumerWarps;
constexpr int kRedSlots = 2;
constexpr int kXBufBytes = 22 * 1024 + 512;   // staged activations of one linear (batch * k_pad * 2 bytes) with two CTAs per SM
constexpr int kXBufBytesMax = 136 * 1024;      // ... with one CTA per SM, for the batches and widths that need more
constexpr int kScaleFloats = 96 * 4;           // (integer form) one 2^-s per k-block and token: k_blocks <= 90, batch <= 4
constexpr int kGlobalSpin = 1 << 20;          // polls (with a short sleep) of a completion counter

struct Item {
    const uint8_t* packed;
    const uint16_t* x;
    void* y;
    int n_tiles, k_blocks, k_in, n_out, m_total, y_dtype, depends, tile_base;
};
struct Params {
    Item item[kSeqMaxItems];
    int n_items, unit_bytes, n_stages;
    int* status;
    int* done;   // [n_items] CTAs that have finished each linear; zero on entry, left zero
    // 255, read from the constant bank: 0/1 bytes times a value the compiler cannot see stays one multiply (on the
    // multiply-add pipe) instead of a shift and a subtract on the logic pipe, which bounds the decode. (The same
    // trick for the right shifts, as mul.hi by 2^16 and 2^13, was measured slower.)
    uint32_t mul_255;
};

__device__ __forceinline__ void consumer_bar_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory"); }
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// ---- integer operands (batch <= 4) -------------------------------------------------------------------
// Every PoT state times 2^emax is a small integer, so b1 and b2 can feed the int8 tensor-core MMA as bytes
// straight out of the byte-table lookup: no 16-bit operand registers to assemble (the largest share of the
// logic-pipe work of the bf16 form), and half as many MMAs (k = 32). The activations are made integers too:
// per token and 128-wide k-block, Q = rne(x * 2^s) with s chosen so that the block's largest magnitude lands in
// [2^14, 2^15), split as Q = 256 q0 + q1 into two int8 rows of the B operand (columns 2t and 2t+1 of token t).
// bf16 has 8 significant bits, so Q is exact for every element within 2^-7 of the block's largest; smaller ones
// are rounded at 2^-15 of it. Integer sums are exact; 256 S0 + S1 is formed in int32 and converted once.
template <int WB> struct IntTables;
template <> struct IntTables<3> {  // codes 0..7 -> 8 4 2 0 -8 -4 -2 -1 and the negated table
    static constexpr uint32_t P0 = 0x00020408u, P1 = 0xFFFEFCF8u, N0 = 0x00FEFCF8u, N1 = 0x01020408u;
};
template <> struct IntTables<2> {  // codes 0..3 -> 2 0 -2 -1
    static constexpr uint32_t P0 = 0xFFFE0002u, P1 = 0u, N0 = 0x010200FEu, N1 = 0u;
};
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// The record table holds sign-bit masks (bit 7 of each flipped byte); >> 7 leaves a 1 in each flipped byte.
__device__ __forceinline__ uint32_t flip_ones(uint32_t sign_bits) { return sign_bits >> 7; }
// One micro-block word -> b1 bytes (pa: weights 0..3, pb: 4..7), int8 = value * 2^emax, and b2 as two operands:
// the permuted b1 bytes with every flipped byte complemented (ra, rb), and a 1 in every flipped byte (za, zb).
// ~v = -v - 1, so sum_i (~v_i) x_i + sum_i 1 x_i = -sum_i v_i x_i over the flipped positions: accumulating both
// operands against the same activations gives the signed sum exactly (a flipped zero contributes -x + x = 0),
// for one xor per register in place of a second table lookup, a second permute and a select.
template <int WB>
__device__ __forceinline__ void decode_i8(const Params& p, uint32_t w, uint32_t lut_lane, uint32_t& pa, uint32_t& pb,
                                          uint32_t& ra, uint32_t& rb, uint32_t& za, uint32_t& zb) {
    const uint32_t m = w & 0x77777777u, mh = m >> 16;
    pa = prmt_b32(IntTables<WB>::P0, IntTables<WB>::P1, m);
    pb = prmt_b32(IntTables<WB>::P0, IntTables<WB>::P1, mh);
    const uint32_t h = (w - m) * kHashMul;
    const uint4 e = lds128(((h >> 19) & 0x1F80u) | lut_lane);   // selectors x, y; ones at the flipped bytes z, w
    za = e.z;
    zb = e.w;
    ra = prmt_b32(pa, pb, e.x) ^ (e.z * p.mul_255);
    rb = prmt_b32(pa, pb, e.y) ^ (e.w * p.mul_255);
}

// first tile of linear `it` that belongs to CTA `cta` (tiles cta-congruent modulo the grid, numbered across linears)
__device__ __forceinline__ int first_tile(const Item& it, int cta, int n_ctas) {
    int r = (cta - it.tile_base) % n_ctas;
    return r < 0 ? r + n_ctas : r;
}

#ifdef GOQ_TRACE
__device__ unsigned long long g_seq_trace[512][8][8];   // [cta][item][event], warp 0 lane 0, SM cycle counter
#define GOQ_ST(item, ev) do { if (threadIdx.x == 0 && (item) >= GOQ_TRI0 && (item) < GOQ_TRI0 + 8) { unsigned long long t_; \
    asm volatile("mov.u64 %0, %%clock64;" : "=l"(t_) :: "memory"); g_seq_trace[blockIdx.x][(item) - GOQ_TRI0][ev] = t_; } } while (0)
#else
#define GOQ_ST(item, ev) do { } while (0)
#endif
#ifndef GOQ_TRI0
#define GOQ_TRI0 0
#endif

template <int WB, int CPG, bool I8>
__global__ void __launch_bounds__(kThreads, 2) gemv_seq_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* lut = smem + ((8192u - (smem_u32(smem) & 8191u)) & 8191u);   // 8 KiB boundary: slot offsets are OR-ed in
    const int stage_bytes = kStageUnits * p.unit_bytes;
    unsigned char* ring = lut + kLutBytes;
    float* red = reinterpret_cast<float*>(ring + (size_t)p.n_stages * stage_bytes);
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(red + kRedSlots * kConsumerWarps * 32 * 4);
    uint64_t* empty_bar = full_bar + p.n_stages;
    uint64_t* x_bar = empty_bar + p.n_stages;
    float* xscale = reinterpret_cast<float*>(x_bar + 2);   // (I8) [k-block][4 tokens]
    uint16_t* xs = reinterpret_cast<uint16_t*>(xscale + kScaleFloats);   // bf16 rows, or (I8) int8 rows 2*token + slice; last: its size varies per launch
    __shared__ volatile int abort_flag;
    __shared__ int arrive_cnt[kRedSlots];
    __shared__ int done_gen[kRedSlots];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_ctas = (int)gridDim.x, cta = (int)blockIdx.x;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < kRedSlots; ++i) { arrive_cnt[i] = 0; done_gen[i] = 0; }
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kConsumerWarps); }
        mbar_init(x_bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp == kConsumerWarps) {
        // ---------------- producer: the weight stream of every tile this CTA owns, linear after linear ----------------
        if (lane == 0) {
            int slot = 0, round = 0, issued = 0;
            bool ok = true;
            for (int i = 0; i < p.n_items && ok; ++i) {
                const Item& it = p.item[i];
                for (int T = first_tile(it, cta, n_ctas); T < it.n_tiles && ok; T += n_ctas) {
                    const uint8_t* src = it.packed + unit_offset(T, 0, it.k_blocks, p.unit_bytes);
                    for (int u0 = 0; u0 < it.k_blocks; u0 += kStageUnits) {
                        if (round > 0 && !mbar_wait_bounded(&empty_bar[slot], (round - 1) & 1, &abort_flag)) { ok = false; break; }
                        const int units = min(kStageUnits, it.k_blocks - u0);
                        const uint32_t bytes = (uint32_t)units * p.unit_bytes;
                        mbar_arrive_expect_tx(&full_bar[slot], bytes);
                        bulk_copy_g2s(ring + (size_t)slot * stage_bytes, src + (size_t)u0 * p.unit_bytes, bytes, &full_bar[slot]);
                        if (++slot == p.n_stages) { slot = 0; ++round; }
                        ++issued;
                    }
                }
            }
            if (!ok || abort_flag) drain_issued_stages(full_bar, issued, p.n_stages);
        }
        return;
    }

    // ---------------- consumers ----------------
    for (int i = tid; i < 64 * kLutCopies; i += kConsumerWarps * 32) {
        const uint32_t* e = c_exchange_lut.v[i / kLutCopies];
        *reinterpret_cast<uint4*>(lut + (size_t)i * 16) =
            I8 ? make_uint4(e[0], e[1], flip_ones(e[2]), flip_ones(e[3])) : make_uint4(e[0], e[1], e[2], e[3]);
    }
    const int g = lane >> 2, t = lane & 3;
    const uint32_t lut_lane = smem_u32(lut) + (lane & (kLutCopies - 1)) * 16;
    int slot = 0, phase = 0;   // position in the stage ring
    int n_tile_local = 0;      // tiles this CTA has finished (indexes the reduction slots)
    uint32_t x_phase = 0;

    for (int i = 0; i <= p.n_items; ++i) {
        // ---- boundary between linear i-1 and linear i ----
        GOQ_ST(i, 0);
        consumer_bar_sync();   // every warp has finished linear i-1: outputs stored, activation buffer free
        GOQ_ST(i, 1);
        if (i == p.n_items) {
            if (tid == 0 && i > 0) {
                // the CTA that completes the last linear last leaves the counters zero for the next call
                const int prev = atomic_add_acq_rel_gpu(&p.done[i - 1], 1);
                if (prev == n_ctas - 1) for (int j = 0; j < p.n_items; ++j) p.done[j] = 0;
            }
            break;
        }
        const Item& it = p.item[i];
        const int k_pad = it.k_blocks * kBlockK;
        const int T0 = first_tile(it, cta, n_ctas);
        const bool have_work = T0 < it.n_tiles;
        if (tid == 0) {
            if (i > 0) atomic_add_acq_rel_gpu(&p.done[i - 1], 1);   // releases this CTA's outputs (ordered by the barrier above)
            if (have_work && abort_flag == 0) {
                bool ok = true;
                if (it.depends && i > 0) {   // the activations may be outputs of earlier linears: all CTAs must be done with them
                    int spins = 0;
                    while (ld_acquire_gpu(&p.done[i - 1]) < n_ctas) {
                        if (abort_flag || ++spins > kGlobalSpin) { abort_flag = 1; ok = false; break; }
                        __nanosleep(64);
                    }
                }
                GOQ_ST(i, 2);
                if (ok && !I8) {
                    const uint32_t row_bytes = (uint32_t)it.k_in * 2;
                    mbar_arrive_expect_tx(x_bar, row_bytes * it.m_total);
                    for (int r = 0; r < it.m_total; ++r) bulk_copy_g2s(xs + (size_t)r * k_pad, it.x + (size_t)r * it.k_in, row_bytes, x_bar);
                }
            }
            if (I8 && have_work) mbar_arrive(x_bar);   // the activations may be read now (or the CTA has given up)
        }
        if (!have_work) continue;
        bool x_ok;
        if constexpr (I8) {
            // ---- fetch the activations and make them integers (see above): 16-byte chunks of 8 bf16, 16 chunks = one k-block ----
            x_ok = mbar_wait_bounded(x_bar, x_phase, &abort_flag) && abort_flag == 0;
            unsigned char* xb = reinterpret_cast<unsigned char*>(xs);
            const int cpt = k_pad / 8, total = cpt * it.m_total;
            for (int c0 = warp * 32; c0 < total; c0 += kConsumerWarps * 32) {
                const int c = c0 + lane;
                const bool in = c < total;
                const int r = in ? c / cpt : 0, k0 = in ? (c - r * cpt) * 8 : 0;
                uint4 v = make_uint4(0u, 0u, 0u, 0u);
                if (in && x_ok && k0 < it.k_in) v = __ldcg(reinterpret_cast<const uint4*>(it.x + (size_t)r * it.k_in + k0));   // L2: written by other SMs
                const uint32_t in32[4] = {v.x, v.y, v.z, v.w};
                uint32_t amax = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) amax = max(amax, max(in32[j] & 0x7FFFu, (in32[j] >> 16) & 0x7FFFu));
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
                int sfield = 268 - (int)(amax >> 7);   // 2^s: the block's largest magnitude lands in [2^14, 2^15)
                sfield = sfield < 1 ? 1 : (sfield > 253 ? 253 : sfield);
                const float mult = __uint_as_float((uint32_t)sfield << 23);
                uint32_t q0[2] = {0u, 0u}, q1[2] = {0u, 0u};
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t bits = (j & 1) ? (in32[j >> 1] & 0xFFFF0000u) : (in32[j >> 1] << 16);
                    // rne to an integer without the quarter-rate convert: adding 1.5 * 2^23 leaves it in the low mantissa bits
                    int Q = __float_as_int(fmaf(__uint_as_float(bits), mult, 12582912.0f)) - 0x4B400000;
                    Q = max(-32639, min(32639, Q));
                    const int lo = ((Q + 128) & 255) - 128, hi = (Q - lo) >> 8;   // Q = 256 hi + lo, both int8
                    q0[j >> 2] |= (uint32_t)(hi & 255) << (8 * (j & 3));
                    q1[j >> 2] |= (uint32_t)(lo & 255) << (8 * (j & 3));
                }
                if (in) {
                    *reinterpret_cast<uint2*>(xb + (size_t)(2 * r) * k_pad + k0) = make_uint2(q0[0], q0[1]);
                    *reinterpret_cast<uint2*>(xb + (size_t)(2 * r + 1) * k_pad + k0) = make_uint2(q1[0], q1[1]);
                    // 2^-s, and 2^-emax for the integer weights
                    if ((lane & 15) == 0) xscale[(k0 >> 7) * 4 + r] = __uint_as_float((uint32_t)(254 - sfield) << 23) * (1.0f / (float)(1 << ((1 << (WB - 1)) - 1)));
                }
            }
            consumer_bar_sync();
        } else {
            {   // zero the padding [k_in, k_pad) of every staged activation row (the copies do not touch it)
                const int tail = k_pad - it.k_in;
                for (int j = tid; j < tail * it.m_total; j += kConsumerWarps * 32) xs[(size_t)(j / tail) * k_pad + it.k_in + (j % tail)] = 0;
            }
            consumer_bar_sync();
            x_ok = mbar_wait_bounded(x_bar, x_phase, &abort_flag);
        }
        GOQ_ST(i, 3);
        x_phase ^= 1u;
        // lanes whose token does not exist read the last token's row: an MMA output column depends only on its own
        // B column, and columns of missing tokens are never stored
        const uint32_t xrow_s = I8 ? order_after_wait(smem_u32(xs) + (uint32_t)(min(g, 2 * it.m_total - 1) * k_pad + t * 8))
                                   : order_after_wait(smem_u32(xs) + (uint32_t)(min(g, it.m_total - 1) * k_pad + t * 8) * 2);

        for (int T = T0; T < it.n_tiles; T += n_ctas) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int u0 = 0; u0 < it.k_blocks; u0 += kStageUnits) {
                const int units = min(kStageUnits, it.k_blocks - u0);
                if (mbar_wait_bounded(&full_bar[slot], phase, &abort_flag) && x_ok && warp < units) {
                    const uint32_t unit = order_after_wait(smem_u32(ring) + slot * stage_bytes + warp * p.unit_bytes + lane * 16);
                    const int kb0 = (u0 + warp) * kBlockK;
                    const uint4 wv0 = lds128(unit), wv1 = lds128(unit + 512);
                    const uint32_t coef_addr = unit - lane * 16 + kCodeBytesPerUnit + g * 4;
                    const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
                    if constexpr (I8) {
                        int s1[4] = {0, 0, 0, 0}, s2[4] = {0, 0, 0, 0}, s3[4] = {0, 0, 0, 0};
                        float rec0 = 0.f, rec2 = 0.f;   // this record's sums for token t: row g, row g+8
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const uint2 xb = lds64(xrow_s + kb0 + c * 32);
                            uint32_t pa0, pb0, ra0, rb0, za0, zb0, pa1, pb1, ra1, rb1, za1, zb1;
                            decode_i8<WB>(p, w0[c], lut_lane, pa0, pb0, ra0, rb0, za0, zb0);
                            decode_i8<WB>(p, w1[c], lut_lane, pa1, pb1, ra1, rb1, za1, zb1);
                            // A fragment: a0/a1 = bytes k 0..3 of the micro-block for rows g / g+8, a2/a3 = bytes 4..7
                            mma_s8(s1, pa0, pa1, pb0, pb1, xb.x, xb.y);
                            mma_s8(s2, ra0, ra1, rb0, rb1, xb.x, xb.y);
                            mma_s8(s3, za0, za1, zb0, zb1, xb.x, xb.y);
                            if (((c + 1) % CPG) == 0) {   // end of a macro-block: the coefficient multiply, outside the inner product
                                const int jj = c / CPG;
                                const uint32_t cfa = lds32(coef_addr + jj * 64), cfb = lds32(coef_addr + jj * 64 + 32);
                                const float c1a = __half2float(__ushort_as_half((unsigned short)(cfa & 0xFFFFu)));
                                const float c2a = __half2float(__ushort_as_half((unsigned short)(cfa >> 16)));
                                const float c1b = __half2float(__ushort_as_half((unsigned short)(cfb & 0xFFFFu)));
                                const float c2b = __half2float(__ushort_as_half((unsigned short)(cfb >> 16)));
                                // columns 2t, 2t+1 hold the high and low activation slices of token t: S = 256 S_hi + S_lo, exact in int32
                                rec0 += c1a * (float)(s1[0] * 256 + s1[1]) + c2a * (float)((s2[0] + s3[0]) * 256 + s2[1] + s3[1]);
                                rec2 += c1b * (float)(s1[2] * 256 + s1[3]) + c2b * (float)((s2[2] + s3[2]) * 256 + s2[3] + s3[3]);
#pragma unroll
                                for (int r = 0; r < 4; ++r) s1[r] = s2[r] = s3[r] = 0;
                            }
                        }
                        const float sv = xscale[(u0 + warp) * 4 + (t < it.m_total ? t : 0)];   // undo the activation scale of this k-block
                        acc[0] = fmaf(sv, rec0, acc[0]);
                        acc[2] = fmaf(sv, rec2, acc[2]);
                    } else {
                        float d1[4] = {0.f, 0.f, 0.f, 0.f}, d2[4] = {0.f, 0.f, 0.f, 0.f};
    #pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            const uint4 xa = lds128(xrow_s + (kb0 + c * 32) * 2);
                            uint32_t R0[4], Q0[4], R1[4], Q1[4];
                            expand_word<WB>(w0[c], lut_lane, R0, Q0);
                            expand_word<WB>(w1[c], lut_lane, R1, Q1);
                            mma_bf16(d1, R0[0], R1[0], R0[1], R1[1], xa.x, xa.y);
                            mma_bf16(d2, Q0[0], Q1[0], Q0[1], Q1[1], xa.x, xa.y);
                            mma_bf16(d1, R0[2], R1[2], R0[3], R1[3], xa.z, xa.w);
                            mma_bf16(d2, Q0[2], Q1[2], Q0[3], Q1[3], xa.z, xa.w);
                            if (((c + 1) % CPG) == 0) {   // end of a macro-block: the coefficient multiply, outside the inner product
                                const int jj = c / CPG;
                                const uint32_t cfa = lds32(coef_addr + jj * 64), cfb = lds32(coef_addr + jj * 64 + 32);
                                const float c1a = __half2float(__ushort_as_half((unsigned short)(cfa & 0xFFFFu)));
                                const float c2a = __half2float(__ushort_as_half((unsigned short)(cfa >> 16)));
                                const float c1b = __half2float(__ushort_as_half((unsigned short)(cfb & 0xFFFFu)));
                                const float c2b = __half2float(__ushort_as_half((unsigned short)(cfb >> 16)));
                                acc[0] += c1a * d1[0] + c2a * d2[0];
                                acc[1] += c1a * d1[1] + c2a * d2[1];
                                acc[2] += c1b * d1[2] + c2b * d2[2];
                                acc[3] += c1b * d1[3] + c2b * d2[3];
    #pragma unroll
                                for (int r = 0; r < 4; ++r) d1[r] = d2[r] = 0.f;
                            }
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty_bar[slot]);
                if (++slot == p.n_stages) { slot = 0; phase ^= 1; }
            }
            GOQ_ST(i, 4 + min(3, (T - T0) / n_ctas));
            // ---- park this warp's sums; the last warp of the tile adds them in warp order and stores ----
            const int rs = n_tile_local % kRedSlots;
            const int contributors = min(kConsumerWarps, it.k_blocks);
            if (warp < contributors) {
                bool ok = abort_flag == 0;
                if (ok && n_tile_local >= kRedSlots) {   // the slot's previous tile must be fully reduced
                    volatile int* dg = &done_gen[rs];
                    int spins = 0;
                    while (*dg != n_tile_local - kRedSlots + 1) {
                        if (abort_flag || ++spins > kSpinLimit) { abort_flag = 1; ok = false; break; }
                        __nanosleep(40);
                    }
                }
                if (ok) {
                    float* rb = red + (size_t)rs * kConsumerWarps * 32 * 4;
                    reinterpret_cast<float4*>(rb)[warp * 32 + lane] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                    __threadfence_block();
                    __syncwarp();
                    int old = 0;
                    if (lane == 0) old = atomicAdd(&arrive_cnt[rs], 1);
                    old = __shfl_sync(0xFFFFFFFFu, old, 0);
                    if (old == contributors - 1) {
                        __threadfence_block();
                        float out[4] = {0.f, 0.f, 0.f, 0.f};
                        for (int w = 0; w < contributors; ++w) {   // warp order: the sum does not depend on which warp came last
                            const float4 f = reinterpret_cast<const float4*>(rb)[w * 32 + lane];
                            out[0] += f.x; out[1] += f.y; out[2] += f.z; out[3] += f.w;
                        }
                        if (abort_flag == 0) {
#pragma unroll
                            for (int r = 0; r < 4; ++r) {
                                const int row = T * 16 + g + ((r & 2) ? 8 : 0);
                                const int tok = I8 ? t : t * 2 + (r & 1);   // (I8) one token per lane, in elements 0 and 2
                                if (row < it.n_out && tok < it.m_total && !(I8 && (r & 1))) {
                                    if (it.y_dtype == GOQ_F32) reinterpret_cast<float*>(it.y)[(size_t)tok * it.n_out + row] = out[r];
                                    else reinterpret_cast<uint16_t*>(it.y)[(size_t)tok * it.n_out + row] = f32_to_bf16_rne(out[r]);
                                }
                            }
                        }
                        __syncwarp();
                        if (lane == 0) {
                            arrive_cnt[rs] = 0;
                            __threadfence_block();
                            done_gen[rs] = n_tile_local + 1;
                        }
                    }
                }
            }
            ++n_tile_local;
        }
    }
    if (tid == 0 && abort_flag) atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
}

}  // namespace seq
}  // namespace goq

// ---- host side -------------------------------------------------------------------------------------
namespace goq {

bool g_seq_int8 = true;   // integer operands for sequences whose items all have batch <= 4 (tests force both forms)

static int seq_sm_count() {
    int dev = 0, n = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    return n > 0 ? n : 148;
}

bool gemv_seq_supported(const Geometry& g, int m) {
    return g.group >= 32 && g.wbits <= 3 && m >= 1 && m <= 8 && (size_t)m * g.k_pad * 2 <= (size_t)seq::kXBufBytesMax &&
           g.k_blocks * 4 <= seq::kScaleFloats;
}
size_t gemv_seq_workspace(int n_items) { return 256 + (size_t)(n_items > 0 ? n_items : 0) * sizeof(int); }

template <int WB, int CPG, bool I8>
static cudaError_t launch_seq_cfg(seq::Params& p, cudaStream_t st) {
    auto kernel = seq::gemv_seq_kernel<WB, CPG, I8>;
    const int stage_bytes = seq::kStageUnits * p.unit_bytes;
    p.n_stages = 3;
    // The activations of the widest linear decide the buffer: the usual size leaves room for two CTAs per SM; a
    // larger batch or width gets what it needs and one CTA per SM (the grid follows from the occupancy query).
    size_t x_need = 0;
    for (int i = 0; i < p.n_items; ++i) {
        const size_t b = (size_t)p.item[i].m_total * p.item[i].k_blocks * kBlockK * 2;
        if (b > x_need) x_need = b;
    }
    const int xbuf_bytes = x_need <= (size_t)seq::kXBufBytes ? seq::kXBufBytes : (int)((x_need + 1023) & ~(size_t)1023);
    const size_t smem = (size_t)2 * kLutBytes + (size_t)p.n_stages * stage_bytes + (size_t)seq::kRedSlots * seq::kConsumerWarps * 32 * 4 * sizeof(float) +
                        (size_t)(2 * p.n_stages + 2) * sizeof(uint64_t) + (size_t)xbuf_bytes + (size_t)seq::kScaleFloats * sizeof(float);
    static size_t occ_smem[2] = {0, 0};   // occupancy cache: [0] the two-per-SM size, [1] the last larger size
    static int occ_per_sm[2] = {0, 0};
    static SmemAttrCache smem_attr;
    if (cudaError_t e = ensure_dynamic_smem(kernel, smem, smem_attr)) return e;
    const int slot = xbuf_bytes == seq::kXBufBytes ? 0 : 1;
    if (occ_smem[slot] != smem) {
        cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ_per_sm[slot], kernel, seq::kThreads, smem);
        if (e != cudaSuccess) return e;
        occ_smem[slot] = smem;
    }
    const int per_sm = occ_per_sm[slot];
    if (per_sm < 1) return cudaErrorLaunchOutOfResources;
    long long total_tiles = 0;
    for (int i = 0; i < p.n_items; ++i) total_tiles += p.item[i].n_tiles;
    int grid = seq_sm_count() * (per_sm > 2 ? 2 : per_sm);   // every CTA must be resident: the completion counters are waited on
    if ((long long)grid > total_tiles) grid = (int)total_tiles;
    int base = 0;
    for (int i = 0; i < p.n_items; ++i) {   // tiles are numbered across linears; tile number mod grid = owning CTA
        p.item[i].tile_base = base;
        base = (base + p.item[i].n_tiles) % grid;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(seq::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

cudaError_t launch_gemv_seq(const SeqCall* calls, int n, int wbits, int group, int unit_bytes, void* ws, cudaStream_t st) {
    static thread_local seq::Params p;   // ~14 KB: kept off the stack
    auto* wsb = (uint8_t*)ws;
    p.n_items = n;
    p.unit_bytes = unit_bytes;
    p.status = (int*)wsb;
    p.done = (int*)(wsb + 256);
    p.mul_255 = 255u;
    for (int i = 0; i < n; ++i) {
        seq::Item& it = p.item[i];
        it.packed = (const uint8_t*)calls[i].packed;
        it.x = (const uint16_t*)calls[i].x;
        it.y = calls[i].y;
        it.n_tiles = calls[i].g.n_tiles;
        it.k_blocks = calls[i].g.k_blocks;
        it.k_in = calls[i].g.k_in;
        it.n_out = calls[i].g.n_out;
        it.m_total = calls[i].m;
        it.y_dtype = calls[i].y_dtype;
        it.depends = calls[i].depends;
        it.tile_base = 0;
    }
    const int cpg = group / 32;
    bool i8 = g_seq_int8;   // the integer form serves batch <= 4; one kernel per launch, so every item must qualify
    for (int i = 0; i < n; ++i) i8 = i8 && calls[i].m <= 4;
    if (i8) {
        if (wbits == 3) return cpg == 1 ? launch_seq_cfg<3, 1, true>(p, st) : cpg == 2 ? launch_seq_cfg<3, 2, true>(p, st) : launch_seq_cfg<3, 4, true>(p, st);
        return cpg == 1 ? launch_seq_cfg<2, 1, true>(p, st) : cpg == 2 ? launch_seq_cfg<2, 2, true>(p, st) : launch_seq_cfg<2, 4, true>(p, st);
    }
    if (wbits == 3) return cpg == 1 ? launch_seq_cfg<3, 1, false>(p, st) : cpg == 2 ? launch_seq_cfg<3, 2, false>(p, st) : launch_seq_cfg<3, 4, false>(p, st);
    return cpg == 1 ? launch_seq_cfg<2, 1, false>(p, st) : cpg == 2 ? launch_seq_cfg<2, 2, false>(p, st) : launch_seq_cfg<2, 4, false>(p, st);
}

}  // namespace goq
