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

cudaError_t launch_gemm_a8(const Geometry& g, const void* packed, const int8_t* x, int m, const float* sx,
                           const int8_t* cq, const float* sc, void* y, int y_dtype, int32_t* acc, cudaStream_t st) {
    auto* words = (const uint8_t*)packed;
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
