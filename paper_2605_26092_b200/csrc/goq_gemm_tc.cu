// Prefill GEMM (float activations, many tokens) on the 5th-generation tensor cores.
//
// Eq. 4 of the paper with the coefficients folded into the weight operand:
//   y[m,n] = sum_k x[m,k] * w_hat[n,k],   w_hat[n,k] = c1[n,j] b1[n,k] + c2[n,j] b2[n,k]   (Section 3.1)
// Each CTA computes a 128 (output channels) x 512 (tokens) tile. Per 64-wide k-chunk
//   - a producer thread bulk-copies the packed unit records of the 128 rows (cp.async.bulk, 8 records per
//     128 k) and loads the 512 x 64 bf16 activation tile with two 2-D TMA copies (128-byte swizzle);
//   - eight expander warps decode the records (same byte-table decode and record lookup as the GEMV:
//     b1 from the code bytes, b2 = byte-permuted b1 with pair signs, Section 3.3), form
//     w_hat = c1*b1 + c2*b2 with one half2 multiply and one half2 fma (a single rounding to fp16: the products
//     c*b are exact scalings of c) and store the 128 x 64 operand tile to shared
//     memory in the K-major, 128-byte-swizzled layout the tensor core reads;
//   - one thread issues tcgen05.mma (M=128, N=256, K=16, fp16 x fp16 -> fp32) into a 128 x 512 fp32
//     accumulator that fills the SM's tensor memory, and commits each stage back to the producers.
// After the last chunk the warps read the accumulator with tcgen05.ld and store y.
//
// Operand precision. One rounding of w_hat to bf16 (8 significant bits) costs about 2e-3 normwise on the
// output, the whole error budget; fp16 keeps 11 bits (about 2.5e-4) for the same tensor work, where a
// bf16 hi + lo pair needs twice the MMAs. Both MMA operands must then be fp16, so a pre-pass rewrites
// the bf16 activations as fp16, each token scaled by the power of two that puts its largest magnitude in
// [2^14, 2^15): bf16's 8 significant bits are kept exactly, and only elements more than 2^-28 below the
// token's largest lose bits to fp16's range (they vanish below 2^-39 of it). The epilogue undoes the scale.
// The coefficients of every output channel are first multiplied by a power of two chosen from the channel's largest
// coefficient (undone in the epilogue), so w_hat stays in fp16's normal range whatever the scale of the weights.
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, skips the remaining work,
// still frees its tensor memory and records GOQ_ERR_TIMEOUT in the status word.
#include <cuda.h>
#include <cuda_fp16.h>
#include "goq_common.cuh"
#include "goq_internal.h"

namespace goq {
namespace tc {

constexpr int kTileN = 128;     // output channels per CTA (MMA M)
constexpr int kTileM = 512;     // tokens per CTA (two MMA N = 256 halves)
constexpr int kChunkK = 64;     // k per pipeline stage: 128 bytes of bf16 = one swizzle row
constexpr int kStages = 2;
constexpr int kExpanders = 8;   // expander warps; each owns one 16-row unit record per k-block
constexpr int kThreads = (2 + kExpanders) * 32;
constexpr int kATileBytes = kTileN * kChunkK * 2;   // 16 KiB, the weight operand tile of a stage
constexpr int kBTileBytes = kTileM * kChunkK * 2;   // 64 KiB
constexpr int kLutCopies = 8;   // record table, one copy per lane & 7: lookups are bank-conflict free (shared-memory
                                // bandwidth, shared with the tensor core's operand reads, bounds this kernel)
constexpr int kLutBytes = 64 * kLutCopies * 16;
constexpr int kSpin = 1 << 22;

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t n) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* b) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(s32(b)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
    for (int it = 0; it < kSpin; ++it) {
        if (mbar_try(b, parity)) return true;
        if ((it & 63) == 63 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(s32(dst)),
                 "l"(src), "r"(bytes), "r"(s32(bar)) : "memory");
}
// 2-D tiled TMA load (no multicast): coordinates {c0 = k element, c1 = token row}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int c0, int c1, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(s32(dst)), "l"(map), "r"(c0), "r"(c1), "r"(s32(bar)) : "memory");
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
    uint32_t v;
    asm("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint32_t after_wait(uint32_t addr) {
    uint32_t r;
    asm volatile("mov.u32 %0, %1;" : "=r"(r) : "r"(addr) : "memory");
    return r;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// ---- tensor memory and MMA ---------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc_512(uint32_t* smem_slot) {  // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s32(smem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_512(uint32_t taddr) {  // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(taddr) : "memory");
}
// K-major operand tile with 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address
    d |= (uint64_t)1 << 16;                          // leading byte offset (unused for this layout)
    d |= (uint64_t)(1024 >> 4) << 32;                // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                          // descriptor version for sm_100
    d |= (uint64_t)2 << 61;                          // SWIZZLE_128B
    return d;
}
// kind::f16 instruction descriptor: fp32 accumulate, fp16 x fp16 (format fields 0), both K-major, M = 128, N = 256
constexpr uint32_t kIdesc = (1u << 4) | ((256u >> 3) << 17) | ((128u >> 4) << 24);
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(kIdesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}


// ---- record decode (same tables as the decode GEMV) --------------------------------------------
// High byte of the fp16 number of every PoT state, by code (the low byte of a power of two is zero).
template <int WB> struct PotBytes;
template <> struct PotBytes<3> {  // +1 +.5 +.25 0 -1 -.5 -.25 -.125
    static constexpr uint32_t H0 = 0x0034383Cu, H1 = 0xB0B4B8BCu;
};
template <> struct PotBytes<2> {  // +1 0 -1 -.5
    static constexpr uint32_t H0 = 0xB8BC003Cu, H1 = 0u;
};
// W4: code = sign << 3 | e, value (-1)^sign 2^-e (fp16 high byte (15 - e) << 2), sign 0 with e = 7 is the zero state
struct PotBytes4 {
    static constexpr uint32_t PH0 = 0x3034383Cu, PH1 = 0x0024282Cu, NH0 = 0xB0B4B8BCu, NH1 = 0xA0A4A8ACu;
};
constexpr uint32_t kHashMul = 0x01008420u;  // (record bits in place) * kHashMul >> 26 is a bijection onto 0..63

struct ExchangeLut { uint32_t v[64][4]; };
constexpr ExchangeLut make_exchange_lut() {
    ExchangeLut t{};
    for (uint32_t meta = 0; meta < 64; ++meta) {
        const int s = (int)(meta & 3u) + 1;
        // flips: bit i = 1 iff b2 element i has the opposite sign of the b1 element routed to it
        uint32_t flips = 0;
        int p = 0;
        for (int i = 0; i < 8; ++i) {
            const int j = i ^ s;
            if (i < j) {
                const uint32_t f = (meta >> (2 + p)) & 1u;  // 1 iff eta = -1
                flips |= (f ^ 1u) << i;                     // y_i = -eta x_j
                flips |= f << j;                            // y_j =  eta x_i
                ++p;
            }
        }
        uint32_t sel_a = 0, sel_b = 0, f_a = 0, f_b = 0, spread = 0;
        for (int i = 0; i < 4; ++i) {
            sel_a |= (uint32_t)(i ^ s) << (4 * i);
            sel_b |= (uint32_t)((4 + i) ^ s) << (4 * i);
            f_a |= ((flips >> i) & 1u) << (8 * i + 7);
            f_b |= ((flips >> (4 + i)) & 1u) << (8 * i + 7);
        }
        for (int i = 0; i < 6; ++i) spread |= ((meta >> i) & 1u) << (4 * i + 3);
        const uint32_t slot = (uint32_t)(spread * kHashMul) >> 26;
        t.v[slot][0] = sel_a; t.v[slot][1] = sel_b; t.v[slot][2] = f_a; t.v[slot][3] = f_b;
    }
    return t;
}
__constant__ ExchangeLut c_lut = make_exchange_lut();

__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint32_t hfma2(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t r;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
// Eight weights of one micro-block -> w_hat = c1*b1 + c2*b2 in fp16, four f16x2 words. c1, c2: the coefficient in both
// halves of a register. b1 and b2 are built as fp16 directly (table high byte over a zero low byte), c1*b1 is a
// power-of-two scaling (exact) and the fused multiply-add rounds once: the same value as fp32 arithmetic rounded
// to fp16, for a quarter of the instructions.
// W <= 3: the exchange record sits in the spare bit of the word's nibbles and is hashed into the table slot. W = 4: the
// nibbles are full (the sign is bit 3), the record comes from the unit's byte plane (`record`) and the table is filled
// in record order; the high byte is taken from a positive or a negative table per weight, chosen by a byte mask that
// prmt's sign-replicate mode makes of the sign bits (top bit of each byte of w: odd weights; of w << 4: even weights).
template <int WB>
__device__ __forceinline__ void expand_what(uint32_t w, uint32_t record, uint32_t lut_lane, uint32_t c1, uint32_t c2, uint32_t (&out)[4]) {
    const uint32_t m = w & 0x77777777u, mh = m >> 16;
    uint32_t ha, hb, slot_off;
    if constexpr (WB <= 3) {
        ha = prmt(PotBytes<WB>::H0, PotBytes<WB>::H1, m);
        hb = prmt(PotBytes<WB>::H0, PotBytes<WB>::H1, mh);
        slot_off = (((w - m) * kHashMul) >> 19) & 0x1F80u;
    } else {
        const uint32_t s_odd = prmt(w, 0u, 0xBA98u), s_even = prmt(w << 4, 0u, 0xBA98u);
        const uint32_t ma = prmt(s_even, s_odd, 0x5140u), mb = prmt(s_even, s_odd, 0x7362u);   // weights 0..3, 4..7
        ha = (prmt(PotBytes4::PH0, PotBytes4::PH1, m) & ~ma) | (prmt(PotBytes4::NH0, PotBytes4::NH1, m) & ma);
        hb = (prmt(PotBytes4::PH0, PotBytes4::PH1, mh) & ~mb) | (prmt(PotBytes4::NH0, PotBytes4::NH1, mh) & mb);
        slot_off = (record & 63u) << 7;
    }
    const uint4 e = lds128(slot_off | lut_lane);  // table is 8 KiB aligned, lut_lane selects the copy
    const uint32_t qa = prmt(ha, hb, e.x) ^ e.z, qb = prmt(ha, hb, e.y) ^ e.w;   // b2: permuted, pair signs applied
    // bytes {0, h[2q], 0, h[2q+1]}: weights 2q, 2q+1 as one f16x2 word
    const uint32_t R[4] = {prmt(ha, 0u, 0x1404u), prmt(ha, 0u, 0x3424u), prmt(hb, 0u, 0x1404u), prmt(hb, 0u, 0x3424u)};
    const uint32_t Q[4] = {prmt(qa, 0u, 0x1404u), prmt(qa, 0u, 0x3424u), prmt(qb, 0u, 0x1404u), prmt(qb, 0u, 0x3424u)};
#pragma unroll
    for (int q = 0; q < 4; ++q) out[q] = hfma2(c2, Q[q], hmul2(c1, R[q]));
}

struct GemmParams {
    const uint8_t* packed;
    void* y;
    const float* inv_scale;   // [m_total] 2^-s of each token (the activations the tensor map covers are x * 2^s in fp16)
    const uint32_t* row_scale;   // [n_pad] per-channel power of two for the coefficients, fp16 in both halves
    const float* row_inv;        // [n_pad] its inverse
    int* status;
    int unit_bytes, meta_off, k_blocks, n_tiles, n_out, m_total, y_dtype, group_log2;
    // Tile schedule (1-D grid). CTAs [0, n_full) take 128 x 512 tiles, numbered channel-tile fastest; the remaining
    // CTAs take the last tiles as halves of 256 tokens each, so that a last wave that would fill less than half of
    // the SMs runs for half as long on twice as many.
    // With at most 256 tokens in all, every tile is one half (halves_per_tile = 1).
    int n_full, n_tiles_x, halves_per_tile;
    // Split-K (only with at most 256 tokens, where the tiles alone would leave most SMs idle): n_split CTAs share a
    // tile, each takes kb_per_split k-blocks and parks its fp32 partial tile in `partial`; the CTA that arrives last
    // at the tile's counter adds the partials in split order (the result does not depend on timing), scales and
    // stores, and leaves the counter zero.
    int n_split, kb_per_split;
    float* partial;      // [tile][split][256 tokens][128 channels]
    int* tile_counter;   // [tile], zero on entry, left zero
};

template <int WB>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const GemmParams p, const __grid_constant__ CUtensorMap x_map) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* base = smem_raw + ((8192u - (s32(smem_raw) & 8191u)) & 8191u);  // 8 KiB boundary: table offsets are OR-ed in
    unsigned char* lut = base;
    unsigned char* a_tiles = lut + kLutBytes;
    unsigned char* b_tiles = a_tiles + kStages * kATileBytes;
    unsigned char* pk_ring = b_tiles + kStages * kBTileBytes;
    const int pk_slot_bytes = kExpanders * p.unit_bytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(pk_ring + 2 * pk_slot_bytes);
    uint64_t* full_b = bars;            // [kStages] activation tile landed (tx bytes)
    uint64_t* full_a = bars + 2;        // [kStages] weight tile written by the 8 expander warps
    uint64_t* empty = bars + 4;         // [kStages] tensor core finished reading the stage
    uint64_t* pk_full = bars + 6;       // [2] packed records landed
    uint64_t* pk_empty = bars + 8;      // [2] expanders finished with the records
    uint64_t* tmem_full = bars + 10;    // accumulator complete
    uint64_t* epi_bar = bars + 11;      // [2] epilogue rendezvous of the four warps of a token half
    __shared__ uint32_t tmem_base_slot;
    __shared__ __align__(16) float inv_s[kTileM];   // 2^-s of this CTA's tokens (1 for tokens past the end)
    __shared__ uint32_t row_s[kTileN];              // per-channel coefficient scale (fp16 x 2) of this CTA's 128 channels
    __shared__ float row_i[kTileN];                 // ... and its inverse
    __shared__ volatile int abort_flag;
    __shared__ volatile int split_last;   // (split-K) this CTA completed its tile's counter

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bid = blockIdx.x;
    const int unit_id = bid / p.n_split, split = bid - unit_id * p.n_split;   // n_split > 1 only when every tile is one half
    const int tile = unit_id < p.n_full ? unit_id : p.n_full + (unit_id - p.n_full) / p.halves_per_tile;
    const int n_half = unit_id < p.n_full ? 2 : 1;   // token halves (of 256) this CTA computes
    const int kb0 = split * p.kb_per_split;            // this CTA's k-blocks: [kb0, kb0 + nkb)
    const int nkb = min(p.kb_per_split, p.k_blocks - kb0);
    const int tile_x = tile % p.n_tiles_x;
    const int T0 = tile_x * (kTileN / kTileRows);  // first 16-row tile of this CTA
    const int tok0 = (tile / p.n_tiles_x) * kTileM + (unit_id < p.n_full ? 0 : ((unit_id - p.n_full) % p.halves_per_tile) * 256);
    const int n_chunks = 2 * nkb;

    if (tid == 0) {
        abort_flag = 0;
        for (int i = 0; i < kStages; ++i) { mbar_init(&full_b[i], 1); mbar_init(&full_a[i], kExpanders); mbar_init(&empty[i], 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(&pk_full[i], 1); mbar_init(&pk_empty[i], kExpanders); }
        mbar_init(tmem_full, 1);
        mbar_init(&epi_bar[0], 4);
        mbar_init(&epi_bar[1], 4);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < 64 * kLutCopies; i += kThreads) {
        uint32_t slot = (uint32_t)(i / kLutCopies);
        if constexpr (WB == 4) {   // table in record order: entry `record` is the hashed table's entry of that record
            uint32_t spread = 0;
            for (int b = 0; b < 6; ++b) spread |= ((slot >> b) & 1u) << (4 * b + 3);
            slot = (spread * kHashMul) >> 26;
        }
        const uint32_t* e = c_lut.v[slot];
        *reinterpret_cast<uint4*>(lut + (size_t)i * 16) = make_uint4(e[0], e[1], e[2], e[3]);
    }
    if (warp == 1) tmem_alloc_512(&tmem_base_slot);
    // Everything above needs nothing from the activation pre-pass, which may still be running (programmatic dependent
    // launch: this grid is scheduled as soon as the pre-pass lets it); what follows reads what the pre-pass wrote.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    for (int i = tid; i < kTileM; i += kThreads) inv_s[i] = (tok0 + i < p.m_total) ? __ldcg(&p.inv_scale[tok0 + i]) : 1.0f;
    for (int i = tid; i < kTileN; i += kThreads) {
        const bool in = T0 * kTileRows + i < p.n_tiles * kTileRows;
        row_s[i] = in ? __ldcg(&p.row_scale[T0 * kTileRows + i]) : 0x3C003C00u;   // 1.0
        row_i[i] = in ? __ldcg(&p.row_inv[T0 * kTileRows + i]) : 1.0f;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_slot;

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            int n_rec = p.n_tiles - T0;
            if (n_rec > kExpanders) n_rec = kExpanders;
            bool ok = true;
            int pk_issued = 0, b_issued = 0;   // record blocks / activation chunks whose copies have been issued
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int ps = kb & 1;
                if (kb >= 2) ok = mbar_wait(&pk_empty[ps], ((kb >> 1) - 1) & 1, &abort_flag);
                if (!ok) break;
                pk_issued = kb + 1;
                mbar_expect_tx(&pk_full[ps], (uint32_t)n_rec * p.unit_bytes);
                for (int r = 0; r < n_rec; ++r)
                    bulk_g2s(pk_ring + ps * pk_slot_bytes + r * p.unit_bytes,
                             p.packed + unit_offset(T0 + r, kb0 + kb, p.k_blocks, p.unit_bytes), p.unit_bytes, &pk_full[ps]);
                for (int half = 0; half < 2 && ok; ++half) {
                    const int chunk = 2 * kb + half, s = chunk % kStages;
                    if (chunk >= kStages) ok = mbar_wait(&empty[s], ((chunk / kStages) - 1) & 1, &abort_flag);
                    if (!ok) break;
                    b_issued = chunk + 1;
                    mbar_expect_tx(&full_b[s], (uint32_t)n_half * (kBTileBytes / 2));
                    tma_load_2d(b_tiles + s * kBTileBytes, &x_map, (2 * kb0 + chunk) * kChunkK, tok0, &full_b[s]);
                    if (n_half == 2)
                        tma_load_2d(b_tiles + s * kBTileBytes + kBTileBytes / 2, &x_map, (2 * kb0 + chunk) * kChunkK, tok0 + 256, &full_b[s]);
                }
            }
            if (!ok || abort_flag) {
                // after a give-up: copies already issued must land before the CTA's shared memory goes away (bounded waits)
                for (int i = pk_issued > 2 ? pk_issued - 2 : 0; i < pk_issued; ++i)
                    for (int it = 0; it < kSpin && !mbar_try(&pk_full[i & 1], (uint32_t)(i >> 1) & 1u); ++it) { }
                for (int i = b_issued > kStages ? b_issued - kStages : 0; i < b_issued; ++i)
                    for (int it = 0; it < kSpin && !mbar_try(&full_b[i % kStages], (uint32_t)(i / kStages) & 1u); ++it) { }
            }
        }
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            bool ok = true;
            for (int chunk = 0; chunk < n_chunks; ++chunk) {
                const int s = chunk % kStages;
                const uint32_t par = (chunk / kStages) & 1;
                ok = mbar_wait(&full_b[s], par, &abort_flag) && mbar_wait(&full_a[s], par, &abort_flag);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint64_t adesc = smem_desc_sw128(s32(a_tiles + s * kATileBytes));
                const uint64_t bdesc0 = smem_desc_sw128(s32(b_tiles + s * kBTileBytes));
                const uint64_t bdesc1 = smem_desc_sw128(s32(b_tiles + s * kBTileBytes + kBTileBytes / 2));
#pragma unroll
                for (int ks = 0; ks < kChunkK / 16; ++ks) {
                    const uint32_t acc = (chunk > 0 || ks > 0) ? 1u : 0u;
                    umma_f16(tmem_base, adesc + 2 * ks, bdesc0 + 2 * ks, acc);         // tokens   0..255
                    if (n_half == 2) umma_f16(tmem_base + 256, adesc + 2 * ks, bdesc1 + 2 * ks, acc);   // tokens 256..511
                }
                umma_commit(&empty[s]);
            }
            if (ok) umma_commit(tmem_full);
        }
    } else {
        // ------------------------------ expanders, then epilogue ------------------------------
        const int e = warp - 2, g = lane >> 2, t = lane & 3;
        const uint32_t lut_lane = s32(lut) + (uint32_t)(lane & (kLutCopies - 1)) * 16;
        const bool valid = (T0 + e) < p.n_tiles;
        const uint32_t rs_a = row_s[e * 16 + g], rs_b = row_s[e * 16 + 8 + g];   // scales of this lane's two channels
        constexpr uint32_t kZeroWord = (WB == 4) ? 0x77777777u : (WB == 3) ? 0x33333333u : 0x11111111u;  // every code = the zero state
        bool ok = true;
        for (int kb = 0; kb < nkb && ok; ++kb) {
            const int ps = kb & 1;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&pk_full[ps], (kb >> 1) & 1, &abort_flag));
            if (!ok) break;
            const uint32_t unit = after_wait(s32(pk_ring) + ps * pk_slot_bytes + e * p.unit_bytes);
            uint4 wv0 = make_uint4(kZeroWord, kZeroWord, kZeroWord, kZeroWord), wv1 = wv0;
            uint32_t mv0 = 0u, mv1 = 0u;   // (W4) the exchange records of this lane's eight words, one byte each
            if (valid) {
                wv0 = lds128(unit + lane * 16); wv1 = lds128(unit + 512 + lane * 16);
                if constexpr (WB == 4) { mv0 = lds32(unit + p.meta_off + lane * 4); mv1 = lds32(unit + p.meta_off + 128 + lane * 4); }
            }
            const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                const int chunk = 2 * kb + half, s = chunk % kStages;
                if (chunk >= kStages) ok = __all_sync(0xFFFFFFFFu, mbar_wait(&empty[s], ((chunk / kStages) - 1) & 1, &abort_flag));
                if (!ok) break;
                const uint32_t a_tile = s32(a_tiles + s * kATileBytes);
#pragma unroll
                for (int cci = 0; cci < 2; ++cci) {
                    // odd rows take the chunk's two 32-wide slices in the other order: the eight lanes of a quarter warp
                    // (two rows) then store to all eight 16-byte columns of the swizzled rows instead of four, twice
                    const int cc = cci ^ (g & 1);
                    const int c = half * 2 + cc;
                    const uint32_t wa = (g & 1) ? w0[half * 2 + (cci ^ 1)] : w0[half * 2 + cci];
                    const uint32_t wb = (g & 1) ? w1[half * 2 + (cci ^ 1)] : w1[half * 2 + cci];
                    const int jj = (c * 32 + t * 8) >> p.group_log2;  // macro-block of this micro-block inside the k-block
                    uint32_t cfa = 0u, cfb = 0u;   // {c1, c2} as stored: fp16 pairs
                    if (valid) {
                        cfa = hmul2(lds32(unit + kCodeBytesPerUnit + (jj * 16 + g) * 4), rs_a);        // exact: a power of two
                        cfb = hmul2(lds32(unit + kCodeBytesPerUnit + (jj * 16 + 8 + g) * 4), rs_b);
                    }
                    const uint32_t c1a = prmt(cfa, cfa, 0x1010u), c2a = prmt(cfa, cfa, 0x3232u);
                    const uint32_t c1b = prmt(cfb, cfb, 0x1010u), c2b = prmt(cfb, cfb, 0x3232u);
                    uint32_t oa[4], ob[4];
                    expand_what<WB>(wa, mv0 >> (8 * c), lut_lane, c1a, c2a, oa);
                    expand_what<WB>(wb, mv1 >> (8 * c), lut_lane, c1b, c2b, ob);
                    // K-major tile, 128-byte rows, 16-byte chunk j of row r stored at chunk j ^ (r & 7)
                    const int j = cc * 4 + t;
                    const int ra = e * 16 + g, rb = ra + 8;  // (ra & 7) == (rb & 7) == g
                    const uint32_t off = (uint32_t)((j ^ g) << 4);
                    sts128(a_tile + ra * 128 + off, oa[0], oa[1], oa[2], oa[3]);
                    sts128(a_tile + rb * 128 + off, ob[0], ob[1], ob[2], ob[3]);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> tensor-core reads
                __syncwarp();
                if (lane == 0) mbar_arrive(&full_a[s]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&pk_empty[ps]);
        }
        // ---- epilogue: tensor memory -> registers -> y ----
        if (ok) ok = mbar_wait(tmem_full, 0, &abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (ok && (e < 4 || n_half == 2)) {
            // Each thread holds one output channel (a TMEM lane) for 32 tokens; stored directly that is one 4-byte store
            // per token and thread, 2048 128-byte requests per CTA, and the request rate of that burst, not its bytes,
            // set the epilogue's time. So the four warps of a token half transpose 32 tokens x 128 channels through
            // shared memory (the activation ring is idle by now) and store 16 bytes per thread: a quarter of the requests.
            const int q = warp & 3, col_half = (e >= 4) ? 1 : 0;
            const int row4 = tile_x * kTileN + 4 * lane;
            const bool f32 = p.y_dtype == GOQ_F32;
            const bool vec = (tile_x + 1) * kTileN <= p.n_out && (p.n_out & 3) == 0 &&
                             (reinterpret_cast<uintptr_t>(p.y) & (f32 ? 15u : 7u)) == 0;
            auto store4 = [&](int tok, float4 f) {   // four channels of one token
                const size_t o = (size_t)tok * p.n_out + row4;
                if (f32) {
                    float* y = reinterpret_cast<float*>(p.y);
                    if (vec) *reinterpret_cast<float4*>(y + o) = f;
                    else {
                        if (row4 + 0 < p.n_out) y[o + 0] = f.x;
                        if (row4 + 1 < p.n_out) y[o + 1] = f.y;
                        if (row4 + 2 < p.n_out) y[o + 2] = f.z;
                        if (row4 + 3 < p.n_out) y[o + 3] = f.w;
                    }
                } else {
                    uint16_t* y = reinterpret_cast<uint16_t*>(p.y);
                    const uint32_t h01 = pack_bf16x2(f.x, f.y), h23 = pack_bf16x2(f.z, f.w);   // round to nearest even, in hardware
                    if (vec) *reinterpret_cast<uint2*>(y + o) = make_uint2(h01, h23);
                    else {
                        if (row4 + 0 < p.n_out) y[o + 0] = (uint16_t)(h01 & 0xFFFFu);
                        if (row4 + 1 < p.n_out) y[o + 1] = (uint16_t)(h01 >> 16);
                        if (row4 + 2 < p.n_out) y[o + 2] = (uint16_t)(h23 & 0xFFFFu);
                        if (row4 + 3 < p.n_out) y[o + 3] = (uint16_t)(h23 >> 16);
                    }
                }
            };
#pragma unroll 1
            for (int cb = 0; cb < 8 && ok; ++cb) {
                uint32_t v[32];
                const int col0 = col_half * 256 + cb * 32;
                tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)col0, v);
                float* st = reinterpret_cast<float*>(b_tiles) + (col_half * 2 + (cb & 1)) * (32 * kTileN);
                const float irs = row_i[q * 32 + lane];   // this lane's channel: undo the coefficient scale (a power of two)
#pragma unroll
                for (int j4 = 0; j4 < 8; ++j4) {   // the 32 tokens' inverse scales: eight broadcast 16-byte loads
                    const float4 f = *reinterpret_cast<const float4*>(&inv_s[col0 + 4 * j4]);
                    st[(4 * j4 + 0) * kTileN + q * 32 + lane] = __uint_as_float(v[4 * j4 + 0]) * (f.x * irs);
                    st[(4 * j4 + 1) * kTileN + q * 32 + lane] = __uint_as_float(v[4 * j4 + 1]) * (f.y * irs);
                    st[(4 * j4 + 2) * kTileN + q * 32 + lane] = __uint_as_float(v[4 * j4 + 2]) * (f.z * irs);
                    st[(4 * j4 + 3) * kTileN + q * 32 + lane] = __uint_as_float(v[4 * j4 + 3]) * (f.w * irs);
                }
                // bounded rendezvous of the half's four warps (a named barrier could not give up)
                __syncwarp();
                if (lane == 0) mbar_arrive(&epi_bar[col_half]);
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(&epi_bar[col_half], cb & 1, &abort_flag));
                if (!ok) break;
                if (p.n_split > 1) {   // park the (already scaled) partial rows: [token][128 channels], 512 bytes per warp store
                    float* part = p.partial + ((size_t)tile * p.n_split + split) * (256 * kTileN);
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int jt = q * 8 + i;
                        __stcg(reinterpret_cast<float4*>(part + (size_t)(cb * 32 + jt) * kTileN + 4 * lane),
                               *reinterpret_cast<const float4*>(&st[jt * kTileN + 4 * lane]));
                    }
                    continue;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int jt = q * 8 + i, tok = tok0 + col0 + jt;
                    if (tok < p.m_total) store4(tok, *reinterpret_cast<const float4*>(&st[jt * kTileN + 4 * lane]));
                }
            }
            if (p.n_split > 1 && ok) {
                // Every warp's partial rows are on their way: make them visible, meet, and let one thread count this CTA
                // in. The epilogue barrier has been through eight phases, so the next two have parities 0 and 1.
                __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(&epi_bar[0]);
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(&epi_bar[0], 0, &abort_flag));
                if (ok) {
                    if (lane == 0) {
                        if (q == 0) {
                            split_last = (atomicAdd(&p.tile_counter[tile], 1) == p.n_split - 1) ? 1 : 0;
                            __threadfence();
                        }
                        mbar_arrive(&epi_bar[0]);
                    }
                    ok = __all_sync(0xFFFFFFFFu, mbar_wait(&epi_bar[0], 1, &abort_flag));
                }
                if (ok && split_last) {
                    const float* part = p.partial + (size_t)tile * p.n_split * (256 * kTileN);
                    for (int jt = q * 64; jt < q * 64 + 64; ++jt) {
                        const int tok = tok0 + jt;
                        if (tok >= p.m_total) break;
                        float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
                        for (int sp = 0; sp < p.n_split; ++sp) {   // split order: the sum does not depend on which CTA came last
                            const float4 a = __ldcg(reinterpret_cast<const float4*>(part + ((size_t)sp * 256 + jt) * kTileN + 4 * lane));
                            f.x += a.x; f.y += a.y; f.z += a.z; f.w += a.w;
                        }
                        store4(tok, f);
                    }
                    if (q == 0 && lane == 0) p.tile_counter[tile] = 0;
                }
            }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    }
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        tmem_dealloc_512(tmem_base);
    }
    if (tid == 0 && abort_flag) atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
}


// ---- activation pre-pass: bf16 -> scaled fp16, one CTA per token ------------------------------------
// xh[tok][k] = fp16(x[tok][k] * 2^s), inv_scale[tok] = 2^-s, s chosen from the exponent field of the token's largest
// magnitude (an all-zero token gets the largest scale, harmlessly; inf / nan stay inf / nan).
constexpr int kPrepThreads = 256;
// Blocks beyond the tokens compute the per-channel scales of the weight operand, one 16-row tile each: w_hat is
// formed in fp16, whose normal range ends at 2^-14, so every channel's coefficients are multiplied by the power of two
// that puts the channel's largest |c1|, |c2| in [2^6, 2^7) (exact in fp16) and the epilogue divides it out again.
// Coefficients down to 2^-13 of their channel's largest then keep full precision even times the smallest PoT state.
__global__ void __launch_bounds__(kPrepThreads) x_to_f16_kernel(const uint16_t* __restrict__ x, int k_in, uint16_t* __restrict__ xh,
                                                                float* __restrict__ inv_scale, int m_total,
                                                                const uint8_t* __restrict__ packed, int unit_bytes, int k_blocks,
                                                                int groups_per_block, uint32_t* __restrict__ row_scale,
                                                                float* __restrict__ row_inv) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the GEMM's CTAs may set themselves up meanwhile
    if ((int)blockIdx.x >= m_total) {
        __shared__ uint32_t part_max[kPrepThreads / 16][16];
        const int T = (int)blockIdx.x - m_total, r = threadIdx.x & 15, part = threadIdx.x >> 4;
        uint32_t mx = 0;
        for (int bk = part; bk < k_blocks; bk += kPrepThreads / 16) {
            const uint32_t* cw = reinterpret_cast<const uint32_t*>(packed + ((size_t)T * k_blocks + bk) * unit_bytes + kCodeBytesPerUnit);
            for (int jj = 0; jj < groups_per_block; ++jj) {
                const uint32_t w = __ldg(&cw[jj * 16 + r]);
                mx = max(mx, max(w & 0x7FFFu, (w >> 16) & 0x7FFFu));   // fp16 magnitudes order like their bit patterns
            }
        }
        part_max[part][r] = mx;
        __syncthreads();
        if (threadIdx.x < 16) {
            for (int q = 1; q < kPrepThreads / 16; ++q) mx = max(mx, part_max[q][r]);
            int e = (int)(mx >> 10);                 // biased exponent of the largest coefficient (0: zero or subnormal)
            if (e > 30) e = 30;                      // inf / nan coefficients: leave them alone
            int shift = (mx == 0u) ? 0 : 21 - max(e, 1);   // 2^shift brings it to [2^6, 2^7)
            shift = shift < -14 ? -14 : (shift > 15 ? 15 : shift);
            const uint32_t h = (uint32_t)(15 + shift) << 10;
            row_scale[T * 16 + r] = h | (h << 16);
            row_inv[T * 16 + r] = __uint_as_float((uint32_t)(127 - shift) << 23);
        }
        return;
    }
    const int tok = blockIdx.x, tid = threadIdx.x;
    const uint4* row = reinterpret_cast<const uint4*>(x + (size_t)tok * k_in);
    uint4* out = reinterpret_cast<uint4*>(xh + (size_t)tok * k_in);
    const int n_vec = k_in / 8;   // k_in is a multiple of 8 (checked by the launcher)
    __shared__ uint32_t warp_max[kPrepThreads / 32];
    uint32_t amax = 0;
    for (int i = tid; i < n_vec; i += kPrepThreads) {
        const uint4 v = __ldg(&row[i]);
        const uint32_t in32[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) amax = max(amax, max(in32[j] & 0x7FFFu, (in32[j] >> 16) & 0x7FFFu));
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
    if ((tid & 31) == 0) warp_max[tid >> 5] = amax;
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kPrepThreads / 32; ++w) amax = max(amax, warp_max[w]);
    int sfield = 268 - (int)(amax >> 7);   // exponent field of 2^s: the largest magnitude lands in [2^14, 2^15)
    sfield = sfield < 1 ? 1 : (sfield > 253 ? 253 : sfield);
    const float mult = __uint_as_float((uint32_t)sfield << 23);
    for (int i = tid; i < n_vec; i += kPrepThreads) {
        const uint4 v = __ldg(&row[i]);
        const uint32_t in32[4] = {v.x, v.y, v.z, v.w};
        uint32_t o32[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
            o32[j] = pack_f16x2(__uint_as_float(in32[j] << 16) * mult, __uint_as_float(in32[j] & 0xFFFF0000u) * mult);
        out[i] = make_uint4(o32[0], o32[1], o32[2], o32[3]);
    }
    if (tid == 0) inv_scale[tok] = __uint_as_float((uint32_t)(254 - sfield) << 23);
}

// ---- host side ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

static int sm_count_cached() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}
// Split-K factor for a call (1 = none): only with at most 256 tokens, when the channel tiles alone would leave at
// least half of the SMs idle, and never below four k-blocks per CTA.
static int split_factor(const Geometry& g, int m) {
    if (m > 256) return 1;
    const int tiles_x = (g.n_pad + kTileN - 1) / kTileN;
    int s = sm_count_cached() / tiles_x;
    if (s > 4) s = 4;
    if (s > g.k_blocks / 4) s = g.k_blocks / 4;
    if (s < 2) return 1;
    const int per = (g.k_blocks + s - 1) / s;
    return (g.k_blocks + per - 1) / per;   // no empty split
}

static size_t smem_bytes(const Geometry& g) {
    return 8192 /* alignment slack */ + kLutBytes + (size_t)kStages * (kATileBytes + kBTileBytes) +
           (size_t)2 * kExpanders * g.unit_bytes + 16 * sizeof(uint64_t);
}

template <int WB>
static cudaError_t launch_wb(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype, int* status,
                             float* inv_scale, uint32_t* row_scale, float* row_inv, uint16_t* xh, int* tile_counter, float* partial,
                             cudaStream_t st) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return cudaErrorNotSupported;
    if (g.k_in % 8 != 0) return cudaErrorInvalidValue;
    x_to_f16_kernel<<<m + g.n_tiles, kPrepThreads, 0, st>>>((const uint16_t*)x, g.k_in, xh, inv_scale, m, (const uint8_t*)packed,
                                                           g.unit_bytes, g.k_blocks, g.groups_per_block, row_scale, row_inv);
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)g.k_in, (cuuint64_t)m};
    const cuuint64_t strides[1] = {(cuuint64_t)g.k_in * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kChunkK, 256};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(&map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, xh, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidTexture;  // distinct code: the tensor map could not be encoded
    const size_t smem = smem_bytes(g);
    static SmemAttrCache smem_attr;
    if (cudaError_t e = ensure_dynamic_smem(gemm_tc_kernel<WB>, smem, smem_attr)) return e;
    GemmParams p;
    p.packed = (const uint8_t*)packed;
    p.y = y;
    p.inv_scale = inv_scale;
    p.row_scale = row_scale;
    p.row_inv = row_inv;
    p.status = status;
    p.unit_bytes = g.unit_bytes;
    p.meta_off = g.meta_off;
    p.k_blocks = g.k_blocks;
    p.n_tiles = g.n_tiles;
    p.n_out = g.n_out;
    p.m_total = m;
    p.y_dtype = y_dtype;
    int lg = 3;
    while ((1 << lg) < g.group) ++lg;
    p.group_log2 = lg;
    const int tiles_x = (g.n_pad + kTileN - 1) / kTileN, tiles = tiles_x * ((m + kTileM - 1) / kTileM);
    const int sm_count = sm_count_cached();
    const int tail = tiles % sm_count;   // tiles of the last, partial wave
    const int split = (tiles > sm_count && tail > 0 && 2 * tail <= sm_count) ? tail : 0;
    p.n_tiles_x = tiles_x;
    p.halves_per_tile = (m <= 256) ? 1 : 2;
    p.n_full = (m <= 256) ? 0 : tiles - split;
    p.n_split = split_factor(g, m);
    p.kb_per_split = (g.k_blocks + p.n_split - 1) / p.n_split;
    p.partial = partial;
    p.tile_counter = tile_counter;
    const int n_ctas = (m <= 256) ? tiles * p.n_split : p.n_full + 2 * split;
    // Programmatic dependent launch on the pre-pass just enqueued: the CTAs fill their tables, allocate tensor memory
    // and initialise their barriers while it runs, and wait (griddepcontrol.wait) before the first read of its outputs.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(n_ctas);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (m > 256) ? 1 : 0;   // measured: with at most 256 tokens (two waves of split-K CTAs) the early launch costs ~5 us
    return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<WB>, p, map);
}

}  // namespace tc
}  // namespace goq

namespace goq {
bool gemm_tc_supported(const Geometry& g) { return g.wbits <= 4 && g.k_in % 8 == 0 && tc::smem_bytes(g) + 2048 <= 227 * 1024; }
// Scratch: status word and tile counters in the common areas; behind them the per-token inverse scales, the fp16
// copy of the activations and (split-K) the partial tiles.
static size_t align256(size_t v) { return (v + 255) & ~(size_t)255; }
namespace {
struct TcScratch { size_t inv_off, rs_off, ri_off, xh_off, partial_off, total; };
TcScratch tc_scratch(const Geometry& g, int m) {
    TcScratch t;
    t.inv_off = kWsScratchOff;
    t.rs_off = t.inv_off + align256((size_t)m * sizeof(float));
    t.ri_off = t.rs_off + align256((size_t)g.n_pad * sizeof(uint32_t));
    t.xh_off = t.ri_off + align256((size_t)g.n_pad * sizeof(float));
    t.partial_off = align256(t.xh_off + (size_t)m * g.k_in * 2);
    const int split = tc::split_factor(g, m);
    const size_t tiles_x = (size_t)(g.n_pad + tc::kTileN - 1) / tc::kTileN;
    t.total = t.partial_off + (split > 1 ? tiles_x * split * 256 * tc::kTileN * sizeof(float) : 0);
    return t;
}
}  // namespace
size_t gemm_tc_workspace(const Geometry& g, int m) { return tc_scratch(g, m).total; }
cudaError_t launch_gemm_tc(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype, void* ws,
                           cudaStream_t st) {
    int* status = (int*)ws;
    const TcScratch t = tc_scratch(g, m);
    uint8_t* b = (uint8_t*)ws;
    float* inv_scale = (float*)(b + t.inv_off);
    uint32_t* rs = (uint32_t*)(b + t.rs_off);
    float* ri = (float*)(b + t.ri_off);
    uint16_t* xh = (uint16_t*)(b + t.xh_off);
    int* counters = (int*)(b + kWsStatusBytes);   // at most sm_count / 2 tiles when the split is on
    float* partial = (float*)(b + t.partial_off);
    if (g.wbits == 4) return tc::launch_wb<4>(g, packed, x, m, y, y_dtype, status, inv_scale, rs, ri, xh, counters, partial, st);
    return g.wbits == 3 ? tc::launch_wb<3>(g, packed, x, m, y, y_dtype, status, inv_scale, rs, ri, xh, counters, partial, st)
                        : tc::launch_wb<2>(g, packed, x, m, y, y_dtype, status, inv_scale, rs, ri, xh, counters, partial, st);
}
}  // namespace goq
