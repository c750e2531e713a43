// goq_pack / goq_unpack kernels: quantizer output <-> the tile16 packed layout.
// The fields are those of Sections 3.2-3.4 of the paper (code per weight, 6-bit exchange record
// per 8 weights, fp16 coefficient pair per macro-block); unpack also derives b2 the way
// Section 3.3 (Theorem 1) defines it, so tests can compare it with an independent decode.
#include "goq_common.cuh"
#include "goq_internal.h"

namespace goq {

__global__ void pack_words_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ meta,
                                  uint8_t* __restrict__ packed, int n_out, int k_in, int n_pad, int k_pad,
                                  int wbits, int unit_bytes, int meta_off, int k1) {
    const int mbs = k_pad / 8;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n_pad * mbs) return;
    int row = (int)(idx / mbs), mb = (int)(idx % mbs);
    const uint32_t zero_code = (1u << (wbits - 1)) - 1u;
    uint32_t w = 0, m = 0;
    if (row < n_out && mb * 8 < k_in) {
        const uint8_t* c = codes + (size_t)row * k_in + (size_t)mb * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) w |= ((uint32_t)c[i] & ((1u << wbits) - 1u)) << (4 * i);
        m = k1 ? 0u : (meta[(size_t)row * (k_in / 8) + mb] & 63u);   // single-basis weights carry no exchange record
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) w |= zero_code << (4 * i);
    }
    uint8_t* unit = packed + unit_offset(row >> 4, mb >> 4, k_pad / kBlockK, unit_bytes);
    const int wi = word_in_unit(row, mb);
    if (wbits <= 3) {
        w |= scatter_meta(m);
    } else {
        unit[meta_off + wi] = (uint8_t)m;
    }
    reinterpret_cast<uint32_t*>(unit)[wi] = w;
}

__global__ void pack_coef_kernel(const uint16_t* __restrict__ coef, uint8_t* __restrict__ packed, int n_out,
                                 int n_pad, int groups_in, int groups_pad, int gpb, int k_blocks, int unit_bytes, int k1) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n_pad * groups_pad) return;
    int row = (int)(idx / groups_pad), j = (int)(idx % groups_pad);
    uint32_t v = 0;
    if (row < n_out && j < groups_in) {
        const uint16_t* c = coef + ((size_t)row * groups_in + j) * 2;
        v = (uint32_t)c[0] | (k1 ? 0u : ((uint32_t)c[1] << 16));   // single-basis weights: c2 = 0
    }
    uint8_t* unit = packed + unit_offset(row >> 4, j / gpb, k_blocks, unit_bytes);
    reinterpret_cast<uint32_t*>(unit + kCodeBytesPerUnit)[(j % gpb) * 16 + (row & 15)] = v;
}

__global__ void unpack_kernel(const uint8_t* __restrict__ packed, uint8_t* __restrict__ codes_b1,
                              uint8_t* __restrict__ codes_b2, int n_out, int k_in, int k_pad, int wbits,
                              int unit_bytes, int meta_off) {
    const int mbs = k_in / 8;
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n_out * mbs) return;
    int row = (int)(idx / mbs), mb = (int)(idx % mbs);
    const uint8_t* unit = packed + unit_offset(row >> 4, mb >> 4, k_pad / kBlockK, unit_bytes);
    const int wi = word_in_unit(row, mb);
    uint32_t w = reinterpret_cast<const uint32_t*>(unit)[wi];
    uint32_t m = (wbits <= 3) ? gather_meta(w) : (uint32_t)unit[meta_off + wi];
    const uint32_t cmask = (wbits <= 3) ? 0x77777777u : 0xFFFFFFFFu;
    uint32_t cw = w & cmask;
    const uint32_t emax = (1u << (wbits - 1)) - 1u;
    size_t o = (size_t)row * k_in + (size_t)mb * 8;
    if (codes_b1) {
#pragma unroll
        for (int i = 0; i < 8; ++i) codes_b1[o + i] = (uint8_t)((cw >> (4 * i)) & 15u);
    }
    if (codes_b2) {
        int s = (int)(m & 3u) + 1;
        uint32_t src = xor_permute_nibbles(cw, s);
        uint32_t flips = flip_mask(m);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t c = (src >> (4 * i)) & 15u;
            uint32_t sign = c >> (wbits - 1), e = c & emax;
            uint8_t out;
            if (sign == 0 && e == emax) out = 0x80;
            else out = (uint8_t)(((sign ^ ((flips >> i) & 1u)) << 3) | e);
            codes_b2[o + i] = out;
        }
    }
}

__global__ void unpack_coef_kernel(const uint8_t* __restrict__ packed, uint16_t* __restrict__ coef, int n_out,
                                   int groups_in, int gpb, int k_blocks, int unit_bytes) {
    size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (size_t)n_out * groups_in) return;
    int row = (int)(idx / groups_in), j = (int)(idx % groups_in);
    const uint8_t* unit = packed + unit_offset(row >> 4, j / gpb, k_blocks, unit_bytes);
    uint32_t v = reinterpret_cast<const uint32_t*>(unit + kCodeBytesPerUnit)[(j % gpb) * 16 + (row & 15)];
    coef[idx * 2] = (uint16_t)(v & 0xFFFFu);
    coef[idx * 2 + 1] = (uint16_t)(v >> 16);
}

cudaError_t launch_pack(const Geometry& g, const uint8_t* codes, const uint8_t* meta, const uint16_t* coef,
                        void* packed, cudaStream_t st) {
    auto* base = (uint8_t*)packed;
    size_t nw = (size_t)g.n_pad * (g.k_pad / 8);
    pack_words_kernel<<<(unsigned)((nw + 255) / 256), 256, 0, st>>>(codes, meta, base, g.n_out, g.k_in, g.n_pad,
                                                                   g.k_pad, g.wbits, g.unit_bytes, g.meta_off, g.k1);
    size_t nc = (size_t)g.n_pad * g.n_groups;
    pack_coef_kernel<<<(unsigned)((nc + 255) / 256), 256, 0, st>>>(coef, base, g.n_out, g.n_pad, g.k_in / g.group,
                                                                  g.n_groups, g.groups_per_block, g.k_blocks,
                                                                  g.unit_bytes, g.k1);
    return cudaGetLastError();
}

cudaError_t launch_unpack(const Geometry& g, const void* packed, uint8_t* b1, uint8_t* b2, uint16_t* coef,
                          cudaStream_t st) {
    auto* base = (const uint8_t*)packed;
    if (b1 || b2) {
        size_t n = (size_t)g.n_out * (g.k_in / 8);
        unpack_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(base, b1, b2, g.n_out, g.k_in, g.k_pad, g.wbits,
                                                                  g.unit_bytes, g.meta_off);
    }
    if (coef) {
        size_t n = (size_t)g.n_out * (g.k_in / g.group);
        unpack_coef_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(base, coef, g.n_out, g.k_in / g.group,
                                                                       g.groups_per_block, g.k_blocks, g.unit_bytes);
    }
    return cudaGetLastError();
}

}  // namespace goq
