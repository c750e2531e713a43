// Shared device/host helpers of libgoq: packed-layout index arithmetic and code decoding.
//
// Layout GOQ_LAYOUT_TILE16 ("tile16"). Rows are padded to a multiple of 16 (a row tile), k to a
// multiple of 128 (a k-block). The buffer is a sequence of unit records, one per (row tile T,
// k-block bk), in the order T*k_blocks + bk, so a run of consecutive records is one contiguous
// byte range (what a bulk copy wants). A unit record holds
//   [0, 1024)            256 micro-block words. One 32-bit word = one micro-block (8 weights,
//                        Section 3.3 of the paper): nibble i, bits [4i+2:4i], is the code of weight i;
//                        for wbits <= 3 the six bits of the exchange record sit in bit 3 of nibbles 0..5.
//                            word = v*128 + (g*4 + t)*4 + c
//                        for row = 16*T + 8*v + g (v in 0..1, g in 0..7) and micro-block 4*c + t of the
//                        k-block (c = 32-wide chunk 0..3, t = position 0..3 inside the chunk). A warp whose
//                        lane id is g*4+t reads 512 contiguous bytes with one 128-bit load per lane and
//                        every lane receives whole micro-blocks of its two rows, which keeps the exchange
//                        inside a thread.
//   [1024, 1024 + 64*G)  coefficient pairs of the unit's G = 128/group macro-blocks: word jj*16 + (row % 16),
//                        fp16 c1 in the low half, c2 in the high half.
//   then, wbits = 4 only: 256 record bytes, indexed like the words.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/goq.h"

namespace goq {

constexpr int kTileRows = 16;
constexpr int kBlockK = 128;
// Scratch buffer layout shared by every kernel, so that one buffer (sized for the largest call) can serve calls of
// different shapes and kernels: [status word, 256 B][counters, kWsCounterBytes: zero on entry, left zero by every
// kernel][everything else: contents carry nothing from one call to the next].
constexpr size_t kWsStatusBytes = 256;
constexpr size_t kWsCounterBytes = 64 * 1024;
constexpr size_t kWsScratchOff = kWsStatusBytes + kWsCounterBytes;
constexpr int kWordsPerBlock = 256;
constexpr int kCodeBytesPerUnit = kWordsPerBlock * 4;

struct Geometry {
    int n_out, k_in, group, wbits;
    int n_pad, k_pad;
    int n_tiles, k_blocks, n_groups;  // n_groups counts padded groups: k_pad / group
    int groups_per_block;             // 128 / group
    int unit_bytes;                   // bytes of one unit record
    int k1;                           // 1: single-basis weights (layout GOQ_LAYOUT_TILE16_K1): records and c2 are zero
    int meta_off;                     // offset of the record-byte plane inside a unit (wbits = 4 only)
    size_t n_units;
    size_t total_bytes;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ inline bool make_geometry(const goq_desc* d, Geometry* g) {
    if (!d) return false;
    if (d->layout != GOQ_LAYOUT_TILE16 && d->layout != GOQ_LAYOUT_TILE16_K1) return false;
    if (d->n_out <= 0 || d->k_in <= 0) return false;
    if (d->wbits < 2 || d->wbits > 4) return false;
    int gr = d->group;
    if (!(gr == 8 || gr == 16 || gr == 32 || gr == 64 || gr == 128)) return false;
    if (d->k_in % gr) return false;
    g->n_out = d->n_out; g->k_in = d->k_in; g->group = gr; g->wbits = d->wbits;
    g->k1 = d->layout == GOQ_LAYOUT_TILE16_K1 ? 1 : 0;
    g->n_pad = (d->n_out + kTileRows - 1) / kTileRows * kTileRows;
    g->k_pad = (d->k_in + kBlockK - 1) / kBlockK * kBlockK;
    g->n_tiles = g->n_pad / kTileRows;
    g->k_blocks = g->k_pad / kBlockK;
    g->n_groups = g->k_pad / gr;
    g->groups_per_block = kBlockK / gr;
    g->meta_off = kCodeBytesPerUnit + 64 * g->groups_per_block;
    g->unit_bytes = g->meta_off + (d->wbits == 4 ? kWordsPerBlock : 0);
    g->n_units = (size_t)g->n_tiles * g->k_blocks;
    g->total_bytes = g->n_units * (size_t)g->unit_bytes;
    return true;
}

// index of the word of (row, micro-block mb of the k-block) inside its unit record
__host__ __device__ inline int word_in_unit(int row, int mb) {
    int rr = row & 15, v = rr >> 3, g = rr & 7, c = (mb & 15) >> 2, t = mb & 3;
    return v * 128 + (g * 4 + t) * 4 + c;
}
__host__ __device__ inline size_t unit_offset(int tile, int bk, int k_blocks, int unit_bytes) {
    return ((size_t)tile * k_blocks + bk) * (size_t)unit_bytes;
}

// ---- scalar decode helpers (used by pack/unpack and the scalar kernels) --------------------
__device__ __forceinline__ uint32_t gather_meta(uint32_t w) {
    return ((w >> 3) & 1u) | ((w >> 6) & 2u) | ((w >> 9) & 4u) | ((w >> 12) & 8u) | ((w >> 15) & 16u) |
           ((w >> 18) & 32u);
}
__host__ __device__ inline uint32_t scatter_meta(uint32_t meta) {
    uint32_t r = 0;
    for (int i = 0; i < 6; ++i) r |= ((meta >> i) & 1u) << (4 * i + 3);
    return r;
}
// nibble i of the result = nibble (i XOR s) of m
__device__ __forceinline__ uint32_t xor_permute_nibbles(uint32_t m, int s) {
    uint32_t r = m;
    if (s & 1) r = ((r & 0x0F0F0F0Fu) << 4) | ((r >> 4) & 0x0F0F0F0Fu);
    if (s & 2) r = __byte_perm(r, 0, 0x2301);
    if (s & 4) r = __byte_perm(r, 0, 0x1032);
    return r;
}
// Bit i of the result is 1 iff element i of b2 carries the opposite sign of the b1 element it
// was routed from. For the pair (i, j = i^s), i < j, with flag f (1 iff eta = -1):
//   y_i = -eta x_j -> flipped iff eta = +1 -> f ^ 1 ;   y_j = eta x_i -> flipped iff eta = -1 -> f.
__host__ __device__ inline uint32_t flip_mask(uint32_t meta) {
    int s = (int)(meta & 3u) + 1;
    uint32_t flips = 0;
    int p = 0;
    for (int i = 0; i < 8; ++i) {
        int j = i ^ s;
        if (i < j) {
            uint32_t f = (meta >> (2 + p)) & 1u;
            flips |= (f ^ 1u) << i;
            flips |= f << j;
            ++p;
        }
    }
    return flips;
}

__device__ __forceinline__ float bf16_to_f32(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }
__device__ __forceinline__ uint16_t f32_to_bf16_rne(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x40);  // NaN stays NaN
    uint32_t lsb = (u >> 16) & 1u;
    return (uint16_t)((u + 0x7FFFu + lsb) >> 16);
}

}  // namespace goq
