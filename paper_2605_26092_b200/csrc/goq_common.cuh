// Shared device/host helpers of libgoq: packed-layout index arithmetic and code decoding.
//
// Layout GOQ_LAYOUT_TILE16 ("tile16"). Rows are padded to a multiple of 16 (a row tile), k to a
// multiple of 128 (a k-block). One 32-bit word holds one micro-block (8 weights, Section 3.3 of
// the paper): nibble i, bits [4i+2:4i], is the code of weight i. For wbits <= 3 the six bits of
// the exchange record sit in bit 3 of nibbles 0..5; for wbits = 4 the record is a byte in a side
// plane with the same indexing. A (row tile, k-block) pair owns 256 consecutive words (1 KiB):
//     word = v*128 + (g*4 + t)*4 + c
// for row = 16*T + 8*v + g (v in 0..1, g in 0..7) and micro-block 4*c + t of the k-block
// (c = 32-wide chunk 0..3, t = position 0..3 inside the chunk). A warp whose lane id is g*4+t
// therefore reads 512 contiguous bytes with one 128-bit load per lane and every lane receives
// whole micro-blocks of its two rows, which is what lets the exchange stay inside a thread.
// Coefficient pairs (fp16 c1 in the low half, c2 in the high half of a 32-bit word) live in a
// second plane: word (T*J + j)*16 + (row % 16) for group j of J = k_pad/group.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/goq.h"

namespace goq {

constexpr int kTileRows = 16;
constexpr int kBlockK = 128;
constexpr int kWordsPerBlock = 256;

struct Geometry {
    int n_out, k_in, group, wbits;
    int n_pad, k_pad;
    int n_tiles, k_blocks, n_groups;       // n_groups counts padded groups: k_pad / group
    size_t code_words;                     // n_pad * k_pad / 8
    size_t coef_off_bytes, meta_off_bytes; // plane offsets from the packed base (meta: wbits = 4 only)
    size_t total_bytes;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ inline bool make_geometry(const goq_desc* d, Geometry* g) {
    if (!d) return false;
    if (d->layout != GOQ_LAYOUT_TILE16) return false;
    if (d->n_out <= 0 || d->k_in <= 0) return false;
    if (d->wbits < 2 || d->wbits > 4) return false;
    int gr = d->group;
    if (!(gr == 8 || gr == 16 || gr == 32 || gr == 64 || gr == 128)) return false;
    if (d->k_in % gr) return false;
    g->n_out = d->n_out; g->k_in = d->k_in; g->group = gr; g->wbits = d->wbits;
    g->n_pad = (d->n_out + kTileRows - 1) / kTileRows * kTileRows;
    g->k_pad = (d->k_in + kBlockK - 1) / kBlockK * kBlockK;
    g->n_tiles = g->n_pad / kTileRows;
    g->k_blocks = g->k_pad / kBlockK;
    g->n_groups = g->k_pad / gr;
    g->code_words = (size_t)g->n_pad * (size_t)(g->k_pad / 8);
    size_t off = g->code_words * 4;
    off = align_up(off, 128);
    g->coef_off_bytes = off;
    off += (size_t)g->n_pad * (size_t)g->n_groups * 4;
    off = align_up(off, 128);
    g->meta_off_bytes = off;
    if (d->wbits == 4) { off += g->code_words; off = align_up(off, 128); }
    g->total_bytes = off;
    return true;
}

// index of the word of (row, micro-block mb = k/8) in the code plane
__host__ __device__ inline size_t word_index(int row, int mb, int k_blocks) {
    int T = row >> 4, rr = row & 15, v = rr >> 3, g = rr & 7;
    int bk = mb >> 4, m = mb & 15, c = m >> 2, t = m & 3;
    return ((size_t)T * k_blocks + bk) * kWordsPerBlock + v * 128 + (g * 4 + t) * 4 + c;
}
__host__ __device__ inline size_t coef_index(int row, int j, int n_groups) {
    return ((size_t)(row >> 4) * n_groups + j) * 16 + (row & 15);
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
