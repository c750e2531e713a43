// Device helpers shared by the decode-GEMV kernels that feed mma.sync with bf16 PoT operands:
// mbarrier / bulk-copy wrappers with bounded waits, and the in-register decode of a micro-block word
// (Section 3.3 of the paper: b2 is b1 routed by "partner i XOR s" with pair signs).
#pragma once
#include <cuda_fp16.h>
#include "goq_common.cuh"

namespace goq {

// ------------------------------------------------------------------------------------------------
// PTX helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t prmt_b32(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait. Returns false (and raises *abort_flag) if the phase does not complete in time or another
// thread has already given up.
constexpr int kSpinLimit = 1 << 22;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    // try_wait itself suspends the thread for a hardware-defined interval before it reports failure
    for (int it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63) == 63 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// After a give-up: the bulk copies this thread has already issued must land before the CTA (and its shared
// memory) goes away. `issued` stages were issued in ring order over `n_stages` slots; the last min(issued, n_stages)
// may still be in flight. Bounded, and deliberately blind to the abort flag.
__device__ __forceinline__ void drain_issued_stages(uint64_t* full_bar, int issued, int n_stages) {
    const int first = issued > n_stages ? issued - n_stages : 0;
    for (int s = first; s < issued; ++s) {
        const int slot = s % n_stages;
        const uint32_t parity = (uint32_t)(s / n_stages) & 1u;
        for (int it = 0; it < kSpinLimit && !mbar_try_wait(&full_bar[slot], parity); ++it) { }
    }
}
// Device-scope fetch-add that releases this warp's earlier writes (ordered before it by __syncwarp) and
// acquires the writes of the CTAs that incremented before.
__device__ __forceinline__ int atomic_add_acq_rel_gpu(int* addr, int v) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(addr), "r"(v) : "memory");
    return old;
}
// 1-D bulk async copy global -> shared, completion counted in bytes on an mbarrier.
// Source, destination and size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// ------------------------------------------------------------------------------------------------
// weights: code word -> bf16x2 operand registers
// ------------------------------------------------------------------------------------------------
// bf16 bit pattern of a PoT code, high byte / low byte tables indexed by the code
template <int WB> struct PotBytes;
template <> struct PotBytes<3> {  // +1 +.5 +.25 0 -1 -.5 -.25 -.125
    static constexpr uint32_t H0 = 0x003E3F3Fu, H1 = 0xBEBEBFBFu, L0 = 0x00800080u, L1 = 0x00800080u;
};
template <> struct PotBytes<2> {  // +1 0 -1 -.5
    static constexpr uint32_t H0 = 0xBFBF003Fu, H1 = 0u, L0 = 0x00800080u, L1 = 0u;
};

// The six record bits sit in bit 3 of nibbles 0..5 of a word. (spare bits * kHashMul) >> 26 is a
// bijection of the 64 records onto 0..63 (checked exhaustively on the host before the first launch),
// which replaces gathering the bits one by one.
constexpr uint32_t kHashMul = 0x01008420u;
__host__ __device__ inline uint32_t record_slot(uint32_t meta) { return (scatter_meta(meta) * kHashMul) >> 26; }

constexpr int kLutCopies = 8;  // one copy per lane of a quarter-warp: 128-bit lookups never share a bank
constexpr int kLutBytes = 64 * kLutCopies * 16;

// Lookup entry of one exchange record: byte selectors that route the eight high (or low) bytes of b1
// to b2's positions 0..3 (x) and 4..7 (y), and the sign flips of those positions (z, w: bit 7 of each byte).
// The table is built at compile time, indexed by record_slot(record).
struct ExchangeLut {
    uint32_t v[64][4];
};
constexpr uint32_t cx_scatter(uint32_t meta) {
    uint32_t r = 0;
    for (int i = 0; i < 6; ++i) r |= ((meta >> i) & 1u) << (4 * i + 3);
    return r;
}
constexpr uint32_t cx_flips(uint32_t meta) {
    // bit i = 1 iff b2 element i has the opposite sign of the b1 element routed to it:
    // pair (i, j = i^s), i < j, flag f (1 iff eta = -1): y_i = -eta x_j -> f^1 ; y_j = eta x_i -> f
    const int s = (int)(meta & 3u) + 1;
    uint32_t flips = 0;
    int p = 0;
    for (int i = 0; i < 8; ++i) {
        const int j = i ^ s;
        if (i < j) {
            const uint32_t f = (meta >> (2 + p)) & 1u;
            flips |= (f ^ 1u) << i;
            flips |= f << j;
            ++p;
        }
    }
    return flips;
}
constexpr ExchangeLut make_exchange_lut() {
    ExchangeLut t{};
    for (uint32_t meta = 0; meta < 64; ++meta) {
        const int s = (int)(meta & 3u) + 1;
        const uint32_t flips = cx_flips(meta);
        uint32_t sel_a = 0, sel_b = 0, f_a = 0, f_b = 0;
        for (int i = 0; i < 4; ++i) {
            sel_a |= (uint32_t)(i ^ s) << (4 * i);
            sel_b |= (uint32_t)((4 + i) ^ s) << (4 * i);
            f_a |= ((flips >> i) & 1u) << (8 * i + 7);
            f_b |= ((flips >> (4 + i)) & 1u) << (8 * i + 7);
        }
        const uint32_t slot = (uint32_t)(cx_scatter(meta) * kHashMul) >> 26;
        t.v[slot][0] = sel_a; t.v[slot][1] = sel_b; t.v[slot][2] = f_a; t.v[slot][3] = f_b;
    }
    return t;
}
static __constant__ ExchangeLut c_exchange_lut = make_exchange_lut();  // one copy per translation unit

// Shared-memory loads by 32-bit shared-window address. They carry no memory clobber so the compiler may
// schedule them freely; ordering after a barrier wait comes from the address, which is passed through
// order_after_wait() once the wait has returned.
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
__device__ __forceinline__ uint32_t order_after_wait(uint32_t addr) {
    uint32_t r;
    asm volatile("mov.u32 %0, %1;" : "=r"(r) : "r"(addr) : "memory");
    return r;
}

// R[q] = bf16x2 (b1 element 2q, 2q+1); Q[q] the same for b2 (Section 3.3: partner i XOR s routed by a
// byte permute, pair signs XOR-ed into the bf16 sign bit; a flipped zero is -0 and adds nothing).
// lut_lane: shared address of this lane's copy of the record table; the table is 8 KiB aligned, so the
// slot offset (bits 7..12) is OR-ed in.
template <int WB>
__device__ __forceinline__ void expand_word(uint32_t w, uint32_t lut_lane, uint32_t (&R)[4], uint32_t (&Q)[4]) {
    const uint32_t m = w & 0x77777777u, mh = m >> 16;
    const uint32_t ha = prmt_b32(PotBytes<WB>::H0, PotBytes<WB>::H1, m), hb = prmt_b32(PotBytes<WB>::H0, PotBytes<WB>::H1, mh);
    const uint32_t la = prmt_b32(PotBytes<WB>::L0, PotBytes<WB>::L1, m), lb = prmt_b32(PotBytes<WB>::L0, PotBytes<WB>::L1, mh);
    R[0] = prmt_b32(la, ha, 0x5140u);
    R[1] = prmt_b32(la, ha, 0x7362u);
    R[2] = prmt_b32(lb, hb, 0x5140u);
    R[3] = prmt_b32(lb, hb, 0x7362u);
    const uint32_t h = (w - m) * kHashMul;
    const uint4 e = lds128(((h >> 19) & 0x1F80u) | lut_lane);
    const uint32_t qha = prmt_b32(ha, hb, e.x) ^ e.z, qhb = prmt_b32(ha, hb, e.y) ^ e.w;
    const uint32_t qla = prmt_b32(la, lb, e.x), qlb = prmt_b32(la, lb, e.y);
    Q[0] = prmt_b32(qla, qha, 0x5140u);
    Q[1] = prmt_b32(qla, qha, 0x7362u);
    Q[2] = prmt_b32(qlb, qhb, 0x5140u);
    Q[3] = prmt_b32(qlb, qhb, 0x7362u);
}

}  // namespace goq
