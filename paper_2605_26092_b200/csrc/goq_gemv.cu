// Float-activation layer (Eq. 4 of the paper read per macro-block):
//   y[m,n] = sum_j ( c1[n,j] * S1 + c2[n,j] * S2 ),  S1 = sum_{k in j} b1[n,k] x[m,k],  S2 likewise with b2.
// Two kernels over the tile16 packed layout:
//   gemv_scalar_kernel  every PoT term is applied to the fp32 activation as an exponent-field
//                       subtraction plus a sign XOR and added in fp32 (any group size, batch <= 16);
//   linear_mma_kernel   the same products and fp32 sums taken by the bf16 tensor-core MMA with the PoT
//                       value as one operand (a PoT operand only shifts the other operand's exponent, so
//                       every product is exact); b1 and b2 are separate exact operands and the
//                       coefficients multiply the per-group sums outside the MMA, as Eq. 4 has it.
// In both, lane (g,t) of a warp owns whole micro-blocks of rows g and g+8, so the Strided Dual-Exchange
// of Section 3.3 (partner i XOR s, pair signs) never leaves the thread.
#include <cuda_fp16.h>
#include "goq_common.cuh"
#include "goq_internal.h"

namespace goq {

// ------------------------------------------------------------------------------------------------
// scalar exponent-add kernel
// ------------------------------------------------------------------------------------------------
// x * (+-2^-e) by subtracting e from the exponent field and XOR-ing the sign; falls back to a
// multiply when the result would leave the normal range (zero, subnormal, inf, nan inputs).
__device__ __forceinline__ float pot_apply(float x, uint32_t e, uint32_t sign) {
    uint32_t u = __float_as_uint(x);
    uint32_t ex = (u >> 23) & 0xFFu;
    if (ex > e && ex != 0xFFu) return __uint_as_float((u - (e << 23)) ^ (sign << 31));
    return x * __uint_as_float(((127u - e) << 23) | (sign << 31));
}

template <int WB, int MB>
__global__ void __launch_bounds__(128)
gemv_scalar_kernel(const uint8_t* __restrict__ packed, int unit_bytes, int meta_off,
                   const uint16_t* __restrict__ x, void* __restrict__ y,
                   int y_dtype, int n_out, int k_in, int n_tiles, int k_blocks, int group, int batch) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int T = blockIdx.x * 4 + warp;
    if (T >= n_tiles) return;
    const int g = lane >> 2, t = lane & 3;
    constexpr uint32_t EMAX = (1u << (WB - 1)) - 1u;
    constexpr uint32_t CMASK = (WB <= 3) ? 0x77777777u : 0xFFFFFFFFu;

    float acc[2][MB], s1[2][MB], s2[2][MB];
#pragma unroll
    for (int v = 0; v < 2; ++v)
#pragma unroll
        for (int m = 0; m < MB; ++m) acc[v][m] = s1[v][m] = s2[v][m] = 0.f;

    for (int bk = 0; bk < k_blocks; ++bk) {
        const uint8_t* unit = packed + unit_offset(T, bk, k_blocks, unit_bytes);
        const uint4* blk = reinterpret_cast<const uint4*>(unit);
        const uint32_t* coefp = reinterpret_cast<const uint32_t*>(unit + kCodeBytesPerUnit);
        uint4 wv[2] = {blk[lane], blk[32 + lane]};
        uint32_t mv[2] = {0, 0};
        if (WB == 4) {
            mv[0] = *reinterpret_cast<const uint32_t*>(unit + meta_off + lane * 4);
            mv[1] = *reinterpret_cast<const uint32_t*>(unit + meta_off + 128 + lane * 4);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int k0 = bk * kBlockK + c * 32 + t * 8;
            uint32_t cw[2], src[2], flips[2];
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                uint32_t w = (c == 0) ? wv[v].x : (c == 1) ? wv[v].y : (c == 2) ? wv[v].z : wv[v].w;
                uint32_t meta = (WB <= 3) ? gather_meta(w) : ((mv[v] >> (8 * c)) & 63u);
                cw[v] = w & CMASK;
                src[v] = xor_permute_nibbles(cw[v], (int)(meta & 3u) + 1);
                flips[v] = flip_mask(meta);
            }
#pragma unroll
            for (int m = 0; m < MB; ++m) {
                if (m < batch && k0 < k_in) {
                    uint4 xv = *reinterpret_cast<const uint4*>(x + (size_t)m * k_in + k0);
                    uint32_t xr[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        float xi = __uint_as_float((i & 1) ? (xr[i >> 1] & 0xFFFF0000u) : (xr[i >> 1] << 16));
#pragma unroll
                        for (int v = 0; v < 2; ++v) {
                            uint32_t c1 = (cw[v] >> (4 * i)) & 15u;
                            uint32_t sg = c1 >> (WB - 1), e = c1 & EMAX;
                            if (!(sg == 0 && e == EMAX)) s1[v][m] += pot_apply(xi, e, sg);
                            uint32_t c2 = (src[v] >> (4 * i)) & 15u;
                            sg = c2 >> (WB - 1);
                            e = c2 & EMAX;
                            if (!(sg == 0 && e == EMAX)) s2[v][m] += pot_apply(xi, e, sg ^ ((flips[v] >> i) & 1u));
                        }
                    }
                }
            }
            if (group < 32 || ((c + 1) * 32) % group == 0) {
                const int jj = (c * 32 + t * 8) / group;  // macro-block inside this k-block
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    uint32_t cf = coefp[jj * 16 + v * 8 + g];
                    float c1 = __half2float(__ushort_as_half((unsigned short)(cf & 0xFFFFu)));
                    float c2 = __half2float(__ushort_as_half((unsigned short)(cf >> 16)));
#pragma unroll
                    for (int m = 0; m < MB; ++m) {
                        acc[v][m] += c1 * s1[v][m] + c2 * s2[v][m];
                        s1[v][m] = s2[v][m] = 0.f;
                    }
                }
            }
        }
    }
#pragma unroll
    for (int v = 0; v < 2; ++v)
#pragma unroll
        for (int m = 0; m < MB; ++m) {
            float a = acc[v][m];
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 1);
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 2);
            const int row = T * 16 + v * 8 + g;
            if (t == 0 && m < batch && row < n_out) {
                if (y_dtype == GOQ_F32) reinterpret_cast<float*>(y)[(size_t)m * n_out + row] = a;
                else reinterpret_cast<uint16_t*>(y)[(size_t)m * n_out + row] = f32_to_bf16_rne(a);
            }
        }
}

template <int WB>
static cudaError_t launch_scalar_wb(const Geometry& g, const void* packed, const void* x, int batch, void* y,
                                    int y_dtype, cudaStream_t st) {
    auto* base = (const uint8_t*)packed;
    dim3 grid((g.n_tiles + 3) / 4), block(128);
#define GOQ_LAUNCH_SC(MB)                                                                                      \
    gemv_scalar_kernel<WB, MB><<<grid, block, 0, st>>>(base, g.unit_bytes, g.meta_off, (const uint16_t*)x, y,  \
                                                       y_dtype, g.n_out, g.k_in, g.n_tiles, g.k_blocks,        \
                                                       g.group, batch)
    if (batch <= 1) GOQ_LAUNCH_SC(1);
    else if (batch <= 2) GOQ_LAUNCH_SC(2);
    else if (batch <= 4) GOQ_LAUNCH_SC(4);
    else if (batch <= 8) GOQ_LAUNCH_SC(8);
    else GOQ_LAUNCH_SC(16);
#undef GOQ_LAUNCH_SC
    return cudaGetLastError();
}

cudaError_t launch_gemv_scalar(const Geometry& g, const void* packed, const void* x, int batch, void* y,
                               int y_dtype, cudaStream_t st) {
    switch (g.wbits) {
        case 2: return launch_scalar_wb<2>(g, packed, x, batch, y, y_dtype, st);
        case 3: return launch_scalar_wb<3>(g, packed, x, batch, y, y_dtype, st);
        default: return launch_scalar_wb<4>(g, packed, x, batch, y, y_dtype, st);
    }
}

// ------------------------------------------------------------------------------------------------
// tensor-core fragment kernel
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// bf16 bit pattern of a PoT code: high byte / low byte tables indexed by the code (wbits 2 and 3).
template <int WB> struct PotTables;
template <> struct PotTables<3> {  // +1 +.5 +.25 0 -1 -.5 -.25 -.125
    static constexpr uint32_t H0 = 0x003E3F3Fu, H1 = 0xBEBEBFBFu, L0 = 0x00800080u, L1 = 0x00800080u;
};
template <> struct PotTables<2> {  // +1 0 -1 -.5
    static constexpr uint32_t H0 = 0xBFBF003Fu, H1 = 0u, L0 = 0x00800080u, L1 = 0u;
};

// One exchange-record lookup entry: byte selectors that route the 8 high (or low) bytes of b1 to
// b2's positions 0..3 and 4..7, and the sign flips of those positions (bit 7 of each byte).
__device__ inline uint4 make_exchange_entry(uint32_t meta) {
    const int s = (int)(meta & 3u) + 1;
    const uint32_t flips = flip_mask(meta);
    uint32_t sel_a = 0, sel_b = 0, f_a = 0, f_b = 0;
    for (int i = 0; i < 4; ++i) {
        sel_a |= (uint32_t)(i ^ s) << (4 * i);
        sel_b |= (uint32_t)((4 + i) ^ s) << (4 * i);
        f_a |= ((flips >> i) & 1u) << (8 * i + 7);
        f_b |= ((flips >> (4 + i)) & 1u) << (8 * i + 7);
    }
    return make_uint4(sel_a, sel_b, f_a, f_b);
}

// Expand one micro-block word into bf16x2 operand registers: R = b1 (elements 2q, 2q+1 in R[q]),
// Q = b2.
template <int WB>
__device__ __forceinline__ void expand_word(uint32_t w, uint32_t meta4, const uint4* __restrict__ lut,
                                            uint32_t (&R)[4], uint32_t (&Q)[4]) {
    uint32_t ha, hb, la, lb, meta;
    if constexpr (WB <= 3) {
        const uint32_t m = w & 0x77777777u, mh = m >> 16;
        ha = prmt(PotTables<WB>::H0, PotTables<WB>::H1, m);
        hb = prmt(PotTables<WB>::H0, PotTables<WB>::H1, mh);
        la = prmt(PotTables<WB>::L0, PotTables<WB>::L1, m);
        lb = prmt(PotTables<WB>::L0, PotTables<WB>::L1, mh);
        meta = gather_meta(w);
    } else {
        // W4: code = sign << 3 | e, value (-1)^sign 2^-e, except sign 0, e 7 = zero. bf16(2^-e) = (127 - e) << 7: the low
        // byte (0x80 for even e) does not depend on the sign, the high byte comes from a table per sign (the positive
        // one holds 0 at e = 7), chosen per byte by a mask made of the sign bits: prmt's sign-replicate mode turns the
        // top bit of each byte of w (odd weights) and of w << 4 (even weights) into 0x00 / 0xFF.
        constexpr uint32_t PH0 = 0x3E3E3F3Fu, PH1 = 0x003C3D3Du, NH0 = 0xBEBEBFBFu, NH1 = 0xBCBCBDBDu, LL = 0x00800080u;
        const uint32_t m = w & 0x77777777u, mh = m >> 16;
        const uint32_t s_odd = prmt(w, 0u, 0xBA98u), s_even = prmt(w << 4, 0u, 0xBA98u);
        const uint32_t ma = prmt(s_even, s_odd, 0x5140u), mb = prmt(s_even, s_odd, 0x7362u);   // weights 0..3, 4..7
        ha = (prmt(PH0, PH1, m) & ~ma) | (prmt(NH0, NH1, m) & ma);
        hb = (prmt(PH0, PH1, mh) & ~mb) | (prmt(NH0, NH1, mh) & mb);
        la = prmt(LL, LL, m);
        lb = prmt(LL, LL, mh);
        meta = meta4;
    }
    R[0] = prmt(la, ha, 0x5140u);
    R[1] = prmt(la, ha, 0x7362u);
    R[2] = prmt(lb, hb, 0x5140u);
    R[3] = prmt(lb, hb, 0x7362u);
    const uint4 e = lut[meta];
    const uint32_t qha = prmt(ha, hb, e.x) ^ e.z, qhb = prmt(ha, hb, e.y) ^ e.w;
    const uint32_t qla = prmt(la, lb, e.x), qlb = prmt(la, lb, e.y);
    Q[0] = prmt(qla, qha, 0x5140u);
    Q[1] = prmt(qla, qha, 0x7362u);
    Q[2] = prmt(qlb, qhb, 0x5140u);
    Q[3] = prmt(qlb, qhb, 0x7362u);
}

constexpr int kMmaWarps = 8;

template <int WB, int NT>
__global__ void __launch_bounds__(kMmaWarps * 32)
linear_mma_kernel(const uint8_t* __restrict__ packed, int unit_bytes, int meta_off,
                  const uint16_t* __restrict__ x, void* __restrict__ y,
                  int y_dtype, int n_out, int k_in, int k_blocks, int group, int m_total) {
    __shared__ uint4 lut[64];
    extern __shared__ float red[];  // [kMmaWarps][32][NT*4]
    if (threadIdx.x < 64) lut[threadIdx.x] = make_exchange_entry(threadIdx.x);
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int T = blockIdx.x;
    const int tok0 = blockIdx.y * (8 * NT);
    const int cpg = group >> 5;  // 32-wide chunks per group: 1, 2 or 4

    float acc[NT][4], d1[NT][4], d2[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc[nt][r] = d1[nt][r] = d2[nt][r] = 0.f;

    for (int bk = warp; bk < k_blocks; bk += kMmaWarps) {
        const uint8_t* unit = packed + unit_offset(T, bk, k_blocks, unit_bytes);
        const uint4* blk = reinterpret_cast<const uint4*>(unit);
        const uint32_t* coefp = reinterpret_cast<const uint32_t*>(unit + kCodeBytesPerUnit);
        const uint4 wv0 = blk[lane], wv1 = blk[32 + lane];
        const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
        uint32_t mv0 = 0, mv1 = 0;
        if (WB == 4) {
            mv0 = *reinterpret_cast<const uint32_t*>(unit + meta_off + lane * 4);
            mv1 = *reinterpret_cast<const uint32_t*>(unit + meta_off + 128 + lane * 4);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int k0 = bk * kBlockK + c * 32 + t * 8;
            uint4 xa[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const int tok = tok0 + nt * 8 + g;
                xa[nt] = make_uint4(0, 0, 0, 0);
                if (tok < m_total && k0 < k_in) xa[nt] = *reinterpret_cast<const uint4*>(x + (size_t)tok * k_in + k0);
            }
            uint32_t R0[4], Q0[4], R1[4], Q1[4];
            expand_word<WB>(w0[c], (mv0 >> (8 * c)) & 63u, lut, R0, Q0);
            expand_word<WB>(w1[c], (mv1 >> (8 * c)) & 63u, lut, R1, Q1);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                mma_bf16_16816(d1[nt], R0[0], R1[0], R0[1], R1[1], xa[nt].x, xa[nt].y);
                mma_bf16_16816(d1[nt], R0[2], R1[2], R0[3], R1[3], xa[nt].z, xa[nt].w);
                mma_bf16_16816(d2[nt], Q0[0], Q1[0], Q0[1], Q1[1], xa[nt].x, xa[nt].y);
                mma_bf16_16816(d2[nt], Q0[2], Q1[2], Q0[3], Q1[3], xa[nt].z, xa[nt].w);
            }
            if (((c + 1) % cpg) == 0) {
                const uint32_t* cf = coefp + ((c * 32) / group) * 16;
                const uint32_t cfa = cf[g], cfb = cf[8 + g];
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

    // fixed-order sum of the warps' partial results
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) red[(warp * 32 + lane) * (NT * 4) + nt * 4 + r] = acc[nt][r];
    __syncthreads();
    for (int o = threadIdx.x; o < 32 * NT * 4; o += kMmaWarps * 32) {
        const int ln = o / (NT * 4), q = o % (NT * 4), nt = q >> 2, r = q & 3;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kMmaWarps; ++w) s += red[(w * 32 + ln) * (NT * 4) + q];
        const int row = T * 16 + (ln >> 2) + ((r & 2) ? 8 : 0);
        const int tok = tok0 + nt * 8 + (ln & 3) * 2 + (r & 1);
        if (row < n_out && tok < m_total) {
            if (y_dtype == GOQ_F32) reinterpret_cast<float*>(y)[(size_t)tok * n_out + row] = s;
            else reinterpret_cast<uint16_t*>(y)[(size_t)tok * n_out + row] = f32_to_bf16_rne(s);
        }
    }
}

bool linear_mma_supported(const Geometry& g) { return g.group >= 32; }

template <int WB, int NT>
static cudaError_t launch_mma_nt(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype,
                                 cudaStream_t st) {
    auto* base = (const uint8_t*)packed;
    dim3 grid(g.n_tiles, (m + 8 * NT - 1) / (8 * NT)), block(kMmaWarps * 32);
    size_t smem = (size_t)kMmaWarps * 32 * NT * 4 * sizeof(float);
    linear_mma_kernel<WB, NT><<<grid, block, smem, st>>>(base, g.unit_bytes, g.meta_off, (const uint16_t*)x, y,
                                                         y_dtype, g.n_out, g.k_in, g.k_blocks, g.group, m);
    return cudaGetLastError();
}

template <int WB>
static cudaError_t launch_mma_wb(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype,
                                 cudaStream_t st) {
    if (m <= 8) return launch_mma_nt<WB, 1>(g, packed, x, m, y, y_dtype, st);
    if (m <= 16) return launch_mma_nt<WB, 2>(g, packed, x, m, y, y_dtype, st);
    if (m <= 32) return launch_mma_nt<WB, 4>(g, packed, x, m, y, y_dtype, st);
    return launch_mma_nt<WB, 8>(g, packed, x, m, y, y_dtype, st);
}

cudaError_t launch_linear_mma(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype,
                              cudaStream_t st) {
    switch (g.wbits) {
        case 2: return launch_mma_wb<2>(g, packed, x, m, y, y_dtype, st);
        case 3: return launch_mma_wb<3>(g, packed, x, m, y, y_dtype, st);
        default: return launch_mma_wb<4>(g, packed, x, m, y, y_dtype, st);
    }
}

}  // namespace goq
