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
                    int32_t* __restrict__ acc_out, float* __restrict__ amax, int n_out, int k_in, int k_blocks, int group, int m_total,
                    int meta_off) {
    __shared__ __align__(16) int8_t b1s[16][kBlockK];
    __shared__ __align__(16) int8_t b2s[16][kBlockK];
    // W4: 2^emax = 128 does not fit a signed byte, so an integer weight v = +-2^(7-e) is held as v = 2 h + l with
    // h = v / 2 for e <= 6 (|h| <= 64) and l = +-1 for e = 7: S = 2 (x . h) + (x . l), still exact integer arithmetic
    __shared__ __align__(16) int8_t b1l[WB == 4 ? 16 : 1][kBlockK];
    __shared__ __align__(16) int8_t b2l[WB == 4 ? 16 : 1][kBlockK];
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
            const uint32_t meta = WB == 4 ? (uint32_t)(packed + unit_offset(T, bk, k_blocks, unit_bytes))[meta_off + wi] : gather_meta(w);
            const uint32_t cw = WB == 4 ? w : (w & 0x77777777u);
            const uint32_t src = xor_permute_nibbles(cw, (int)(meta & 3u) + 1);
            const uint32_t flips = flip_mask(meta);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int v1 = pot_int<WB>((cw >> (4 * i)) & 15u);
                const int u2 = pot_int<WB>((src >> (4 * i)) & 15u);
                const int v2 = ((flips >> i) & 1u) ? -u2 : u2;
                if constexpr (WB == 4) {
                    b1s[row][kk + i] = (int8_t)(v1 / 2); b1l[row][kk + i] = (int8_t)(v1 % 2);
                    b2s[row][kk + i] = (int8_t)(v2 / 2); b2l[row][kk + i] = (int8_t)(v2 % 2);
                } else {
                    b1s[row][kk + i] = (int8_t)v1;
                    b2s[row][kk + i] = (int8_t)v2;
                }
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
                if constexpr (WB == 4) {
                    int l1 = 0, l2 = 0;
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (q >= q0 && q < q1) {
                            const uint4 a = *reinterpret_cast<const uint4*>(&b1l[row][q * 16]);
                            const uint4 b = *reinterpret_cast<const uint4*>(&b2l[row][q * 16]);
                            l1 = __dp4a((int)xr[q].x, (int)a.x, l1); l1 = __dp4a((int)xr[q].y, (int)a.y, l1);
                            l1 = __dp4a((int)xr[q].z, (int)a.z, l1); l1 = __dp4a((int)xr[q].w, (int)a.w, l1);
                            l2 = __dp4a((int)xr[q].x, (int)b.x, l2); l2 = __dp4a((int)xr[q].y, (int)b.y, l2);
                            l2 = __dp4a((int)xr[q].z, (int)b.z, l2); l2 = __dp4a((int)xr[q].w, (int)b.w, l2);
                        }
                    }
                    s1 = 2 * s1 + l1;
                    s2 = 2 * s2 + l2;
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
    float vmax = 0.f;
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
            vmax = fmaxf(vmax, fabsf(v));
        }
    }
    // requantising epilogue (Section 3.5): the token's largest output magnitude, which the next layer's activation
    // quantizer needs before it can write a single integer; non-negative floats order like their bit patterns
    if (amax && y) atomicMax(reinterpret_cast<int*>(amax) + tok, __float_as_int(vmax));
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
constexpr int kA8NT = 8;          // 8-token column tiles per warp: 64 tokens per CTA
constexpr int kA8Tok = 8 * kA8NT;
constexpr int kA8XStride = 160;   // bytes per token row of the staged activation tile: 128 + 32, so that the 16 lanes of a
                                  // half-warp (4 token rows x 4 eight-byte pieces) hit 32 different banks
constexpr uint32_t kA8HashMul = 0x01008420u;   // (record bits in place) * this >> 26 is a bijection onto 0..63

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ uint2 a8_lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint4 a8_lds128(uint32_t addr) {
    uint4 v;
    asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// CTA = 8 warps: warp w owns the 16-row tile 8*blockIdx.x + w, all warps share the same 64 tokens. Per 128-wide
// k-block the activation tile (64 tokens x 128 int8) is staged in shared memory with cp.async, double-buffered; each
// warp reads its unit record straight from global memory one k-block ahead. Row sums S1, S2 per macro-block on the
// int8 tensor cores, then ACC += c~ * S in int32: every order of these integer operations gives the same bits.
// A macro-block (CPG 32-wide slices) is decoded whole before its MMAs, so that the row sums of one token tile live
// only from its first MMA to its coefficient multiply: the 64 registers a full set of S1, S2 would hold buy a
// second CTA per SM instead.
template <int WB, int CPG>
__global__ void __launch_bounds__(kA8Warps * 32, 2)
gemm_a8_mma_kernel(const uint8_t* __restrict__ packed, int unit_bytes, const int8_t* __restrict__ x,
                   const float* __restrict__ sx, const int8_t* __restrict__ cq, const float* __restrict__ sc,
                   void* __restrict__ y, int y_dtype, int32_t* __restrict__ acc_out, float* __restrict__ amax, int n_out,
                   int n_tiles, int k_in, int k_blocks, int group, int m_total) {
    // record table: byte selectors for positions 0..3 / 4..7 and byte masks of the flipped positions, indexed by the
    // hash of the record bits, eight bank-disjoint copies (entry e, copy c at e*128 + c*16)
    __shared__ __align__(16) unsigned char lut[64 * 8 * 16];
    __shared__ __align__(16) unsigned char xs[2][kA8Tok * kA8XStride];
    for (int i = threadIdx.x; i < 512; i += kA8Warps * 32) {
        const uint32_t meta = i >> 3;
        const int s = (int)(meta & 3u) + 1;
        const uint32_t flips = flip_mask(meta);
        uint32_t sel_a = 0, sel_b = 0, m_a = 0, m_b = 0;
        for (int j = 0; j < 4; ++j) {
            sel_a |= (uint32_t)(j ^ s) << (4 * j);
            sel_b |= (uint32_t)((4 + j) ^ s) << (4 * j);
            if ((flips >> j) & 1u) m_a |= 0xFFu << (8 * j);
            if ((flips >> (4 + j)) & 1u) m_b |= 0xFFu << (8 * j);
        }
        const uint32_t slot = (scatter_meta(meta) * kA8HashMul) >> 26;
        *reinterpret_cast<uint4*>(lut + slot * 128 + (i & 7) * 16) = make_uint4(sel_a, sel_b, m_a, m_b);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int T = blockIdx.x * kA8Warps + warp;
    const bool have_tile = T < n_tiles;
    const int tok0 = blockIdx.y * kA8Tok;
    const int groups_in = k_in / group;
    constexpr int cpg = CPG;
    const int row_a = T * 16 + g, row_b = row_a + 8;
    const uint32_t lut_lane = (uint32_t)__cvta_generic_to_shared(lut) + (uint32_t)(lane & 7) * 16u;
    const uint32_t xs_base = (uint32_t)__cvta_generic_to_shared(&xs[0][0]);

    // the whole CTA copies the activation tile of k-block bk into buffer bk & 1: 512 chunks of 16 bytes, two per thread
    auto stage_x = [&](int bk) {
        const uint32_t dst0 = xs_base + (uint32_t)(bk & 1) * (kA8Tok * kA8XStride);
#pragma unroll
        for (int j = 0; j < (kA8Tok * 8) / (kA8Warps * 32); ++j) {
            const int q = threadIdx.x + j * kA8Warps * 32, tok = q >> 3, part = q & 7;
            const int k0 = bk * kBlockK + part * 16;
            const uint32_t dst = dst0 + (uint32_t)(tok * kA8XStride + part * 16);
            if (k0 < k_in) cp_async16(dst, x + (size_t)min(tok0 + tok, m_total - 1) * k_in + k0);   // k_in % 16 == 0: a chunk is all in or all out
            else asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(dst), "r"(0u) : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    int acc1[kA8NT][4], acc2[kA8NT][4];
#pragma unroll
    for (int nt = 0; nt < kA8NT; ++nt)
#pragma unroll
        for (int r = 0; r < 4; ++r) acc1[nt][r] = acc2[nt][r] = 0;

    // integer coefficient pairs (c1, c2) of rows g and g+8 for the up to four macro-blocks of k-block bk, fetched one
    // k-block ahead like the words: element jj = c1a | c2a << 8 | c1b << 16 | c2b << 24 (as unsigned bytes)
    const int gpb = 4 / cpg;
    auto fetch_coef = [&](int bk, uint32_t (&cf)[4]) {
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            cf[jj] = 0u;
            const int j = bk * gpb + jj;
            if (jj < gpb && j < groups_in) {
                uint32_t lo = 0u, hi = 0u;
                if (row_a < n_out) lo = *reinterpret_cast<const uint16_t*>(cq + ((size_t)row_a * groups_in + j) * 2);
                if (row_b < n_out) hi = *reinterpret_cast<const uint16_t*>(cq + ((size_t)row_b * groups_in + j) * 2);
                cf[jj] = lo | (hi << 16);
            }
        }
    };
    stage_x(0);
    uint32_t ncf[4] = {0u, 0u, 0u, 0u};
    if (have_tile) fetch_coef(0, ncf);
    uint4 nw0 = make_uint4(0, 0, 0, 0), nw1 = nw0;   // the next k-block's words of this warp's record
    if (have_tile) {
        const uint4* unit = reinterpret_cast<const uint4*>(packed + unit_offset(T, 0, k_blocks, unit_bytes));
        nw0 = unit[lane]; nw1 = unit[32 + lane];
    }
    for (int bk = 0; bk < k_blocks; ++bk) {
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();   // tile bk has landed for everyone; everyone has finished reading tile bk - 1
        if (bk + 1 < k_blocks) stage_x(bk + 1);
        const uint32_t w0[4] = {nw0.x, nw0.y, nw0.z, nw0.w}, w1[4] = {nw1.x, nw1.y, nw1.z, nw1.w};
        const uint32_t cf[4] = {ncf[0], ncf[1], ncf[2], ncf[3]};
        if (have_tile && bk + 1 < k_blocks) {
            fetch_coef(bk + 1, ncf);
            const uint4* unit = reinterpret_cast<const uint4*>(packed + unit_offset(T, bk + 1, k_blocks, unit_bytes));
            nw0 = unit[lane]; nw1 = unit[32 + lane];
        }
        if (!have_tile) continue;
        const uint32_t xt = xs_base + (uint32_t)(bk & 1) * (kA8Tok * kA8XStride) + (uint32_t)(g * kA8XStride + t * 8);
#pragma unroll
        for (int mb = 0; mb < 4 / CPG; ++mb) {   // macro-blocks of this k-block
            uint32_t a[CPG][4], q[CPG][4];
#pragma unroll
            for (int cc = 0; cc < CPG; ++cc) {
                const int c = mb * CPG + cc;
#pragma unroll
                for (int v = 0; v < 2; ++v) {
                    const uint32_t w = v ? w1[c] : w0[c];
                    const uint32_t m = w & 0x77777777u, mh = m >> 16;
                    const uint32_t p_lo = prmt8(IntTables<WB>::P0, IntTables<WB>::P1, m), p_hi = prmt8(IntTables<WB>::P0, IntTables<WB>::P1, mh);
                    const uint32_t n_lo = prmt8(IntTables<WB>::N0, IntTables<WB>::N1, m), n_hi = prmt8(IntTables<WB>::N0, IntTables<WB>::N1, mh);
                    const uint32_t h = (w - m) * kA8HashMul;
                    const uint4 e = a8_lds128((((h >> 26) * 128u)) + lut_lane);
                    a[cc][v] = p_lo;          // m16n8k32 A fragment: a0/a1 = k 4t..4t+3 of rows g / g+8, a2/a3 = k 16+4t..
                    a[cc][2 + v] = p_hi;
                    const uint32_t qp_lo = prmt8(p_lo, p_hi, e.x), qn_lo = prmt8(n_lo, n_hi, e.x);
                    const uint32_t qp_hi = prmt8(p_lo, p_hi, e.y), qn_hi = prmt8(n_lo, n_hi, e.y);
                    q[cc][v] = (qp_lo & ~e.z) | (qn_lo & e.z);
                    q[cc][2 + v] = (qp_hi & ~e.w) | (qn_hi & e.w);
                }
            }
            const uint32_t cw = cf[mb];
            const int c1a = (int)(int8_t)(cw & 255u), c2a = (int)(int8_t)((cw >> 8) & 255u);
            const int c1b = (int)(int8_t)((cw >> 16) & 255u), c2b = (int)(int8_t)(cw >> 24);
#pragma unroll
            for (int nt = 0; nt < kA8NT; ++nt) {
                int s1[4] = {0, 0, 0, 0}, s2[4] = {0, 0, 0, 0};
#pragma unroll
                for (int cc = 0; cc < CPG; ++cc) {
                    const uint2 b = a8_lds64(xt + (uint32_t)(nt * 8 * kA8XStride + (mb * CPG + cc) * 32));
                    mma_s8(s1, a[cc][0], a[cc][1], a[cc][2], a[cc][3], b.x, b.y);
                    mma_s8(s2, q[cc][0], q[cc][1], q[cc][2], q[cc][3], b.x, b.y);
                }
                acc1[nt][0] += c1a * s1[0]; acc1[nt][1] += c1a * s1[1];
                acc1[nt][2] += c1b * s1[2]; acc1[nt][3] += c1b * s1[3];
                acc2[nt][0] += c2a * s2[0]; acc2[nt][1] += c2a * s2[1];
                acc2[nt][2] += c2b * s2[2]; acc2[nt][3] += c2b * s2[3];
            }
        }
    }
    if (!have_tile) return;
    constexpr float kInvScale = 1.0f / (float)(1u << ((1u << (WB - 1)) - 1u));
#pragma unroll
    for (int nt = 0; nt < kA8NT; ++nt) {
        float vmax[2] = {0.f, 0.f};   // largest output magnitude of tokens nt*8 + 2t, + 2t+1 over this lane's two rows
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
                    vmax[r & 1] = fmaxf(vmax[r & 1], fabsf(v));
                }
            }
        }
        if (amax && y) {   // requantising epilogue (Section 3.5): per-token largest magnitude for the next layer's quantizer
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {   // over the eight lanes that share these two tokens
                vmax[0] = fmaxf(vmax[0], __shfl_xor_sync(0xFFFFFFFFu, vmax[0], o));
                vmax[1] = fmaxf(vmax[1], __shfl_xor_sync(0xFFFFFFFFu, vmax[1], o));
            }
            if (g == 0) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int tok = tok0 + nt * 8 + t * 2 + e;
                    if (tok < m_total) atomicMax(reinterpret_cast<int*>(amax) + tok, __float_as_int(vmax[e]));
                }
            }
        }
    }
}

cudaError_t launch_gemm_a8(const Geometry& g, const void* packed, const int8_t* x, int m, const float* sx,
                           const int8_t* cq, const float* sc, void* y, int y_dtype, int32_t* acc, float* amax, cudaStream_t st) {
    auto* words = (const uint8_t*)packed;
    if (g.group >= 32 && g.wbits <= 3) {
        dim3 grid2((g.n_tiles + kA8Warps - 1) / kA8Warps, (m + kA8Tok - 1) / kA8Tok), block2(kA8Warps * 32);
#define GOQ_A8_LAUNCH(WB_, CPG_)                                                                                          \
    gemm_a8_mma_kernel<WB_, CPG_><<<grid2, block2, 0, st>>>(words, g.unit_bytes, x, sx, cq, sc, y, y_dtype, acc, amax, g.n_out, \
                                                           g.n_tiles, g.k_in, g.k_blocks, g.group, m)
        const int cpg = g.group >> 5;   // 1, 2 or 4
        if (g.wbits == 3) { if (cpg == 1) GOQ_A8_LAUNCH(3, 1); else if (cpg == 2) GOQ_A8_LAUNCH(3, 2); else GOQ_A8_LAUNCH(3, 4); }
        else { if (cpg == 1) GOQ_A8_LAUNCH(2, 1); else if (cpg == 2) GOQ_A8_LAUNCH(2, 2); else GOQ_A8_LAUNCH(2, 4); }
#undef GOQ_A8_LAUNCH
        return cudaGetLastError();
    }
    dim3 grid(g.n_tiles, (m + kA8Tokens - 1) / kA8Tokens), block(kA8Tokens);
#define GOQ_A8_DP4A(WB_)                                                                                                    \
    gemm_a8_dp4a_kernel<WB_><<<grid, block, 0, st>>>(words, g.unit_bytes, x, sx, cq, sc, y, y_dtype, acc, amax, g.n_out, g.k_in, \
                                                     g.k_blocks, g.group, m, g.meta_off)
    if (g.wbits == 4) GOQ_A8_DP4A(4);
    else if (g.wbits == 3) GOQ_A8_DP4A(3);
    else GOQ_A8_DP4A(2);
#undef GOQ_A8_DP4A
    return cudaGetLastError();
}

}  // namespace goq
