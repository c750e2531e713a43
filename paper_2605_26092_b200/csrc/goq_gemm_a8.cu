// Integer-activation layer (Eq. 4 of the paper with integer X~ and c~), exact in int32:
//   S_b[m,j,n]  = sum_{k in j} x~[m,k] * Bint_b[n,k],   Bint_b = 2^emax * b_b in {0, +-2^(emax-e)}
//   ACC_b[m,n]  = sum_j c~_b[n,j] * S_b[m,j,n]
//   y[m,n]      = s_x[m] * 2^-emax * ( s_c1[n] * ACC_1 + s_c2[n] * ACC_2 )
// Multiplying an integer by +-2^(emax-e) is the left shift x~ << (emax-e) with a sign; the kernel
// takes four such shift-adds per instruction with the packed 8-bit integer dot product, whose
// int32 result is the same bits in any summation order.
// First version: one CTA = one 16-row tile x 128 tokens; a thread owns one token (its 128
// activations of the current k-block stay in registers) and reads the expanded int8 weights from
// shared memory as broadcasts.
#include "goq_common.cuh"
#include "goq_internal.h"

namespace goq {

template <int WB>
__device__ __forceinline__ int pot_int(uint32_t code) {
    constexpr uint32_t EMAX = (1u << (WB - 1)) - 1u;
    const uint32_t sg = code >> (WB - 1), e = code & EMAX;
    if (sg == 0 && e == EMAX) return 0;
    const int mag = 1 << (EMAX - e);
    return sg ? -mag : mag;
}

constexpr int kA8Tokens = 128;

template <int WB>
__global__ void __launch_bounds__(kA8Tokens)
gemm_a8_dp4a_kernel(const uint8_t* __restrict__ packed, int unit_bytes, const int8_t* __restrict__ x,
                    const float* __restrict__ sx,
                    const int8_t* __restrict__ cq, const float* __restrict__ sc, void* __restrict__ y, int y_dtype,
                    int32_t* __restrict__ acc_out, int n_out, int k_in, int k_blocks, int group, int m_total) {
    __shared__ __align__(16) int8_t b1s[16][kBlockK];
    __shared__ __align__(16) int8_t b2s[16][kBlockK];
    __shared__ int8_t cqs[16][16][2];  // [row][group inside the k-block][basis]

    const int T = blockIdx.x;
    const int tok = blockIdx.y * kA8Tokens + threadIdx.x;
    const bool tok_ok = tok < m_total;
    const int gpb = kBlockK / group;  // groups per k-block
    const int groups_in = k_in / group;

    int acc1[16], acc2[16];
#pragma unroll
    for (int r = 0; r < 16; ++r) acc1[r] = acc2[r] = 0;

    for (int bk = 0; bk < k_blocks; ++bk) {
        __syncthreads();
        // expand this block's 256 micro-block words to int8 operands
        for (int wi = threadIdx.x; wi < kWordsPerBlock; wi += kA8Tokens) {
            const uint32_t w =
                reinterpret_cast<const uint32_t*>(packed + unit_offset(T, bk, k_blocks, unit_bytes))[wi];
            const int v = wi >> 7, ln = (wi >> 2) & 31, c = wi & 3;
            const int row = v * 8 + (ln >> 2), kk = c * 32 + (ln & 3) * 8;
            const uint32_t meta = gather_meta(w);
            const uint32_t cw = w & 0x77777777u;
            const uint32_t src = xor_permute_nibbles(cw, (int)(meta & 3u) + 1);
            const uint32_t flips = flip_mask(meta);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                b1s[row][kk + i] = (int8_t)pot_int<WB>((cw >> (4 * i)) & 15u);
                const int v2 = pot_int<WB>((src >> (4 * i)) & 15u);
                b2s[row][kk + i] = (int8_t)(((flips >> i) & 1u) ? -v2 : v2);
            }
        }
        for (int i = threadIdx.x; i < 16 * gpb * 2; i += kA8Tokens) {
            const int b = i & 1, jj = (i >> 1) % gpb, row = (i >> 1) / gpb;
            const int n = T * 16 + row, j = bk * gpb + jj;
            cqs[row][jj][b] = (n < n_out && j < groups_in) ? cq[((size_t)n * groups_in + j) * 2 + b] : (int8_t)0;
        }
        // this token's 128 activations of the block
        uint4 xr[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int k0 = bk * kBlockK + q * 16;
            xr[q] = make_uint4(0, 0, 0, 0);
            if (tok_ok && k0 < k_in) xr[q] = *reinterpret_cast<const uint4*>(x + (size_t)tok * k_in + k0);
        }
        __syncthreads();
#pragma unroll 1
        for (int row = 0; row < 16; ++row) {
            for (int jj = 0; jj < gpb; ++jj) {
                int s1 = 0, s2 = 0;
                const int q0 = jj * group / 16, q1 = (jj + 1) * group / 16;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (q >= q0 && q < q1) {
                        const uint4 a = *reinterpret_cast<const uint4*>(&b1s[row][q * 16]);
                        const uint4 b = *reinterpret_cast<const uint4*>(&b2s[row][q * 16]);
                        s1 = __dp4a((int)xr[q].x, (int)a.x, s1);
                        s1 = __dp4a((int)xr[q].y, (int)a.y, s1);
                        s1 = __dp4a((int)xr[q].z, (int)a.z, s1);
                        s1 = __dp4a((int)xr[q].w, (int)a.w, s1);
                        s2 = __dp4a((int)xr[q].x, (int)b.x, s2);
                        s2 = __dp4a((int)xr[q].y, (int)b.y, s2);
                        s2 = __dp4a((int)xr[q].z, (int)b.z, s2);
                        s2 = __dp4a((int)xr[q].w, (int)b.w, s2);
                    }
                }
                // acc[row] with a compile-time index
#pragma unroll
                for (int r = 0; r < 16; ++r)
                    if (r == row) {
                        acc1[r] += (int)cqs[row][jj][0] * s1;
                        acc2[r] += (int)cqs[row][jj][1] * s2;
                    }
            }
        }
    }
    if (!tok_ok) return;
    constexpr float kInvScale = 1.0f / (float)(1u << ((1u << (WB - 1)) - 1u));
    const float sxm = sx ? sx[tok] : 1.f;
#pragma unroll
    for (int r = 0; r < 16; ++r) {
        const int n = T * 16 + r;
        if (n >= n_out) continue;
        if (acc_out) {
            acc_out[(size_t)tok * n_out + n] = acc1[r];
            acc_out[(size_t)m_total * n_out + (size_t)tok * n_out + n] = acc2[r];
        }
        if (y) {
            const float v = sxm * kInvScale * (sc[n * 2] * (float)acc1[r] + sc[n * 2 + 1] * (float)acc2[r]);
            if (y_dtype == GOQ_F32) reinterpret_cast<float*>(y)[(size_t)tok * n_out + n] = v;
            else reinterpret_cast<uint16_t*>(y)[(size_t)tok * n_out + n] = f32_to_bf16_rne(v);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Tensor-core version (macro-blocks of 32 or more): int8 x int8 -> int32 MMA, m16n8k32.
// The weight operand is the PoT integer 2^emax * b (a byte table lookup per four codes); b2 is b1's
// bytes routed by the exchange record, with the pair signs applied by choosing between the table and
// its negation. Lane (g,t) owns the micro-blocks of rows g and g+8, so one 8-byte activation load per
// token and lane feeds both 16-wide halves of the MMA's k dimension. Group sums S1, S2 stay in
// registers; after each macro-block ACC += c~ * S in int32. Every step is integer arithmetic whose
// result does not depend on evaluation order, so the accumulators equal the shift-and-add definition
// bit for bit.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prmt8(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
template <int WB> struct IntTables;
template <> struct IntTables<3> {  // codes 0..7 -> 8 4 2 0 -8 -4 -2 -1 and the negated table
    static constexpr uint32_t P0 = 0x00020408u, P1 = 0xFFFEFCF8u, N0 = 0x00FEFCF8u, N1 = 0x01020408u;
};
template <> struct IntTables<2> {  // codes 0..3 -> 2 0 -2 -1
    static constexpr uint32_t P0 = 0xFFFE0002u, P1 = 0u, N0 = 0x010200FEu, N1 = 0u;
};

constexpr int kA8Warps = 8;
constexpr int kA8NT = 8;  // 8-token column tiles per warp: 64 tokens

template <int WB>
__global__ void __launch_bounds__(kA8Warps * 32, 1)
gemm_a8_mma_kernel(const uint8_t* __restrict__ packed, int unit_bytes, const int8_t* __restrict__ x,
                   const float* __restrict__ sx, const int8_t* __restrict__ cq, const float* __restrict__ sc,
                   void* __restrict__ y, int y_dtype, int32_t* __restrict__ acc_out, int n_out, int n_tiles, int k_in,
                   int k_blocks, int group, int m_total) {
    __shared__ uint4 lut[64];  // per record: byte selectors for positions 0..3 / 4..7, byte masks of flipped positions
    if (threadIdx.x < 64) {
        const uint32_t meta = threadIdx.x;
        const int s = (int)(meta & 3u) + 1;
        const uint32_t flips = flip_mask(meta);
        uint32_t sel_a = 0, sel_b = 0, m_a = 0, m_b = 0;
        for (int i = 0; i < 4; ++i) {
            sel_a |= (uint32_t)(i ^ s) << (4 * i);
            sel_b |= (uint32_t)((4 + i) ^ s) << (4 * i);
            if ((flips >> i) & 1u) m_a |= 0xFFu << (8 * i);
            if ((flips >> (4 + i)) & 1u) m_b |= 0xFFu << (8 * i);
        }
        lut[meta] = make_uint4(sel_a, sel_b, m_a, m_b);
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int T = blockIdx.x * kA8Warps + warp;
    if (T >= n_tiles) return;
    const int tok0 = blockIdx.y * (8 * kA8NT);
    const int groups_in = k_in / group, cpg = group >> 5;
    const int row_a = T * 16 + g, row_b = row_a + 8;

    int acc1[kA8NT][4], acc2[kA8NT][4], s1[kA8NT][4], s2[kA8NT][4];
#pragma unroll
    for (int nt = 0; nt < kA8NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc1[nt][r] = acc2[nt][r] = s1[nt][r] = s2[nt][r] = 0;
    const int8_t* xrow[kA8NT];
#pragma unroll
    for (int nt = 0; nt < kA8NT; ++nt) xrow[nt] = x + (size_t)min(tok0 + nt * 8 + g, m_total - 1) * k_in + t * 8;

    for (int bk = 0; bk < k_blocks; ++bk) {
        const uint8_t* unit = packed + unit_offset(T, bk, k_blocks, unit_bytes);
        const uint4 wv0 = reinterpret_cast<const uint4*>(unit)[lane], wv1 = reinterpret_cast<const uint4*>(unit)[32 + lane];
        const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int k0 = bk * kBlockK + c * 32;
            uint32_t a[4], q[4];
#pragma unroll
            for (int v = 0; v < 2; ++v) {
                const uint32_t w = v ? w1[c] : w0[c];
                const uint32_t m = w & 0x77777777u, mh = m >> 16;
                const uint32_t p_lo = prmt8(IntTables<WB>::P0, IntTables<WB>::P1, m), p_hi = prmt8(IntTables<WB>::P0, IntTables<WB>::P1, mh);
                const uint32_t n_lo = prmt8(IntTables<WB>::N0, IntTables<WB>::N1, m), n_hi = prmt8(IntTables<WB>::N0, IntTables<WB>::N1, mh);
                const uint4 e = lut[gather_meta(w)];
                a[v] = p_lo;          // m16n8k32 A fragment: a0/a1 = k 4t..4t+3 of rows g / g+8, a2/a3 = k 16+4t..
                a[2 + v] = p_hi;
                const uint32_t qp_lo = prmt8(p_lo, p_hi, e.x), qn_lo = prmt8(n_lo, n_hi, e.x);
                const uint32_t qp_hi = prmt8(p_lo, p_hi, e.y), qn_hi = prmt8(n_lo, n_hi, e.y);
                q[v] = (qp_lo & ~e.z) | (qn_lo & e.z);
                q[2 + v] = (qp_hi & ~e.w) | (qn_hi & e.w);
            }
            const bool in_k = (k0 + t * 8) < k_in;
#pragma unroll
            for (int nt = 0; nt < kA8NT; ++nt) {
                uint2 b = make_uint2(0, 0);
                if (in_k) b = *reinterpret_cast<const uint2*>(xrow[nt] + k0);
                mma_s8(s1[nt], a[0], a[1], a[2], a[3], b.x, b.y);
                mma_s8(s2[nt], q[0], q[1], q[2], q[3], b.x, b.y);
            }
            if (((c + 1) % cpg) == 0) {
                const int j = k0 / group;
                int c1a = 0, c2a = 0, c1b = 0, c2b = 0;
                if (j < groups_in) {
                    if (row_a < n_out) { c1a = cq[((size_t)row_a * groups_in + j) * 2]; c2a = cq[((size_t)row_a * groups_in + j) * 2 + 1]; }
                    if (row_b < n_out) { c1b = cq[((size_t)row_b * groups_in + j) * 2]; c2b = cq[((size_t)row_b * groups_in + j) * 2 + 1]; }
                }
#pragma unroll
                for (int nt = 0; nt < kA8NT; ++nt) {
                    acc1[nt][0] += c1a * s1[nt][0]; acc1[nt][1] += c1a * s1[nt][1];
                    acc1[nt][2] += c1b * s1[nt][2]; acc1[nt][3] += c1b * s1[nt][3];
                    acc2[nt][0] += c2a * s2[nt][0]; acc2[nt][1] += c2a * s2[nt][1];
                    acc2[nt][2] += c2b * s2[nt][2]; acc2[nt][3] += c2b * s2[nt][3];
#pragma unroll
                    for (int r = 0; r < 4; ++r) s1[nt][r] = s2[nt][r] = 0;
                }
            }
        }
    }
    constexpr float kInvScale = 1.0f / (float)(1u << ((1u << (WB - 1)) - 1u));
#pragma unroll
    for (int nt = 0; nt < kA8NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int row = (r & 2) ? row_b : row_a;
            const int tok = tok0 + nt * 8 + t * 2 + (r & 1);
            if (row < n_out && tok < m_total) {
                if (acc_out) {
                    acc_out[(size_t)tok * n_out + row] = acc1[nt][r];
                    acc_out[(size_t)m_total * n_out + (size_t)tok * n_out + row] = acc2[nt][r];
                }
                if (y) {
                    const float v = sx[tok] * kInvScale * (sc[row * 2] * (float)acc1[nt][r] + sc[row * 2 + 1] * (float)acc2[nt][r]);
                    if (y_dtype == GOQ_F32) reinterpret_cast<float*>(y)[(size_t)tok * n_out + row] = v;
                    else reinterpret_cast<uint16_t*>(y)[(size_t)tok * n_out + row] = f32_to_bf16_rne(v);
                }
            }
        }
}

cudaError_t launch_gemm_a8(const Geometry& g, const void* packed, const int8_t* x, int m, const float* sx,
                           const int8_t* cq, const float* sc, void* y, int y_dtype, int32_t* acc, cudaStream_t st) {
    auto* words = (const uint8_t*)packed;
    if (g.group >= 32) {
        dim3 grid2((g.n_tiles + kA8Warps - 1) / kA8Warps, (m + 8 * kA8NT - 1) / (8 * kA8NT)), block2(kA8Warps * 32);
        if (g.wbits == 3)
            gemm_a8_mma_kernel<3><<<grid2, block2, 0, st>>>(words, g.unit_bytes, x, sx, cq, sc, y, y_dtype, acc, g.n_out,
                                                            g.n_tiles, g.k_in, g.k_blocks, g.group, m);
        else
            gemm_a8_mma_kernel<2><<<grid2, block2, 0, st>>>(words, g.unit_bytes, x, sx, cq, sc, y, y_dtype, acc, g.n_out,
                                                            g.n_tiles, g.k_in, g.k_blocks, g.group, m);
        return cudaGetLastError();
    }
    dim3 grid(g.n_tiles, (m + kA8Tokens - 1) / kA8Tokens), block(kA8Tokens);
    if (g.wbits == 3)
        gemm_a8_dp4a_kernel<3><<<grid, block, 0, st>>>(words, g.unit_bytes, x, sx, cq, sc, y, y_dtype, acc, g.n_out, g.k_in,
                                                       g.k_blocks, g.group, m);
    else
        gemm_a8_dp4a_kernel<2><<<grid, block, 0, st>>>(words, g.unit_bytes, x, sx, cq, sc, y, y_dtype, acc, g.n_out, g.k_in,
                                                       g.k_blocks, g.group, m);
    return cudaGetLastError();
}

}  // namespace goq
