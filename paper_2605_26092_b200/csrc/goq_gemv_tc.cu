// Decode GEMV (batch <= 16) on tcgen05 tensor cores with the weight operand in tensor memory.
//
// Eq. 4 of the paper read per macro-block:  y[m,n] = sum_j ( c1[n,j] S1 + c2[n,j] S2 ),
// S1 = sum_{k in j} b1[n,k] x[m,k], S2 likewise with b2 (Sections 3.1, 3.3, 3.5).
//
// Every PoT state of b1 and of b2 is one FP8 (e4m3) byte, so a 32-bit micro-block word decodes to the
// eight b1 bytes with two byte-table lookups (prmt) and to the eight b2 bytes with two more permutes of
// those bytes plus a sign XOR, driven by the 6-bit exchange record through a shared-memory table. The
// bytes never touch shared memory: the lane that owns micro-blocks of rows g and g+8 of a 16-row unit
// record writes them straight into tensor memory with the 16-lane x 256-bit store shape, whose
// thread-to-element map is exactly that ownership. Eight records (128 output channels x 128 k) form one
// MMA A operand, M = 128; b1 and b2 get separate A tiles and separate fp32 accumulators per macro-block,
// so the coefficient multiply stays outside the inner product as Eq. 4 has it.
//
// The activations are bf16 and an FP8 MMA wants FP8 on both sides: per token and per 128-wide k-block,
// x * 2^s is split into two e4m3 slices, hi = e4m3(x 2^s) and lo = e4m3(16 (x 2^s - hi)); the second is
// exact whenever it is in range, so x = 2^-s (hi + lo/16) to ~2^-17 of the block's largest element. hi and
// lo are two columns of the B operand; the epilogue recombines them with the block's scale.
//
// Roles in a CTA (one CTA per SM, contiguous range of 128x128 super-units, Stream-K style):
//   warp 0      producer: 1-D bulk async copies of unit records (one per lane) into a ring of stages
//   warp 1      MMA issuer (one thread), owns the tensor-memory allocation
//   warps 2-3   activation slicer: bf16 -> two e4m3 slices, written as the swizzled K-major B tile
//   warps 4-19  two teams of eight expander warps: words -> FP8 bytes -> tensor memory
//   warps 20-23 epilogue: accumulators out of tensor memory, coefficient and scale multiply, row sums,
//               output or parked partial sums (a 128-row tile that straddles CTAs is finished by the CTA
//               that arrives last, adding the parked sums in CTA order: results do not depend on timing).
// A CTA visits the tile it shares with the next CTA first, so the cross-CTA hand-off is off the tail.
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, every role leaves its loop,
// tensor memory is released and GOQ_ERR_TIMEOUT is written to the scratch status word.
#include <cuda_fp16.h>
#include "goq_common.cuh"
#include "goq_internal.h"

namespace goq {
namespace gtc {

constexpr int kRowTiles = 8;                 // unit records per super-unit (MMA M = 128)
constexpr int kTeams = 2;
constexpr int kWarpProducer = 0, kWarpMma = 1, kWarpX0 = 2, kXWarps = 2, kWarpExp0 = 4;
constexpr int kExpWarps = kRowTiles * kTeams;
constexpr int kWarpEpi0 = kWarpExp0 + kExpWarps, kEpiWarps = 4;
constexpr int kThreads = (kWarpEpi0 + kEpiWarps) * 32;   // 768
constexpr int kXSlots = 8;                   // ring of activation tiles
constexpr int kMaxStages = 16;
constexpr int kLutBytes = 8192;              // 64 records x 8 bank-disjoint copies x 16 bytes
constexpr int kSpin = 1 << 22;
constexpr int kMaxCtas = 160;
constexpr int kStatusBytes = 256;
constexpr int kSlotFloats = 128 * 16;        // parked partial sums of one segment: 128 rows x up to 16 tokens

struct Ws { size_t counters_off, partials_off, total; };
__host__ inline Ws ws_layout(const Geometry& g) {
    Ws w;
    w.counters_off = kStatusBytes;
    w.partials_off = kWsScratchOff;
    w.total = w.partials_off + (size_t)kMaxCtas * 2 * kSlotFloats * sizeof(float);
    return w;
}

// ---- PTX helpers -----------------------------------------------------------------------------------
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
// Whole-warp wait with one polling lane (a warp-wide poll is 32 shared-memory barrier operations per try).
__device__ __forceinline__ bool warp_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
    bool ok = true;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(b, parity, abort_flag);
    return __all_sync(0xFFFFFFFFu, ok);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(s32(bar)) : "memory");
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
__device__ __forceinline__ uint4 lds128_v(uint32_t addr) {  // ordered with respect to the barrier waits around it
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds32_v(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ int atomic_add_acq_rel_gpu(int* p, int v) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}

// ---- tensor memory ---------------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc_512(uint32_t* smem_slot) {  // whole warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s32(smem_slot)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_512(uint32_t taddr) {  // whole warp
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(taddr) : "memory");
}
// 16 lanes x 256 bits, four times along the columns (32 columns): lane (g,t) of the warp supplies, for column
// block c, registers {4c, 4c+1} -> tensor-memory lane g, columns 8c+2t, 8c+2t+1 and {4c+2, 4c+3} -> lane g+8.
__device__ __forceinline__ void tmem_st_16x256b_x4(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.16x256b.x4.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
          "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 32 lanes x 32 bits, 16 consecutive columns: thread i of the warp reads lane (32*(warp%4) + i)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand tile with 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// kind::f8f6f4 instruction descriptor: fp32 accumulate, e4m3 x e4m3, both K-major, M = 128
__host__ __device__ constexpr uint32_t idesc_e4m3(int n) { return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((128u >> 4) << 24); }
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void umma_f8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(bar)) : "memory");
}

// ---- record decode ---------------------------------------------------------------------------------
// e4m3 byte of every code of the lattice of Section 3.2 (code = sign << (b-1) | exponent, exponent emax = zero
// on the positive side): b = 3: +1 +.5 +.25 0 -1 -.5 -.25 -.125 ; b = 2: +1 0 -1 -.5
template <int WB> struct PotFp8;
template <> struct PotFp8<3> { static constexpr uint32_t F0 = 0x00283038u, F1 = 0xA0A8B0B8u; };
template <> struct PotFp8<2> { static constexpr uint32_t F0 = 0xB0B80038u, F1 = 0u; };
constexpr uint32_t kHashMul = 0x01008420u;  // (record bits in place) * kHashMul >> 26 is a bijection onto 0..63

// Table of the 64 exchange records (Section 3.3: partner i XOR s, y_i = -eta x_j, y_j = eta x_i), addressed by
// the hash of the record bits: two byte selectors that route the eight b1 bytes and two sign-flip masks.
struct ExchangeLut { uint32_t v[64][4]; };
constexpr ExchangeLut make_exchange_lut() {
    ExchangeLut t{};
    for (uint32_t meta = 0; meta < 64; ++meta) {
        const int s = (int)(meta & 3u) + 1;
        uint32_t flips = 0;  // bit i = 1 iff b2 element i has the opposite sign of the b1 element routed to it
        int p = 0;
        for (int i = 0; i < 8; ++i) {
            const int j = i ^ s;
            if (i < j) {
                const uint32_t f = (meta >> (2 + p)) & 1u;  // 1 iff eta = -1
                flips |= (f ^ 1u) << i;
                flips |= f << j;
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

// one micro-block word -> eight b1 bytes (a: weights 0..3, b: weights 4..7) and eight b2 bytes
template <int WB>
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t lut_lane, uint32_t& b1a, uint32_t& b1b, uint32_t& b2a,
                                            uint32_t& b2b) {
    const uint32_t m = w & 0x77777777u;
    b1a = prmt(PotFp8<WB>::F0, PotFp8<WB>::F1, m);
    // shifts written as high multiplies: they issue on the multiplier pipe, not on the half-rate logic pipe
    b1b = prmt(PotFp8<WB>::F0, PotFp8<WB>::F1, __umulhi(m, 1u << 16));
    const uint32_t h = (w - m) * kHashMul;
    const uint4 e = lds128((__umulhi(h, 1u << 13) & 0x1F80u) | lut_lane);  // entry (h >> 26) * 128 + copy * 16, table 8 KiB aligned
    b2a = prmt(b1a, b1b, e.x) ^ e.z;   // a flipped zero becomes -0: adds nothing
    b2b = prmt(b1a, b1b, e.y) ^ e.w;
}

struct Params {
    const uint8_t* packed;
    const uint16_t* x;
    void* y;
    int* status;
    int* counters;
    float* partials;
    int unit_bytes, k_blocks, n_tiles, n_super, k_in, n_out, m_total, y_dtype, n_stages;
};

// ---- work decomposition ----------------------------------------------------------------------------
// Super-unit index su = ST * k_blocks + bk (ST: 128-row tile, bk: k-block). CTA c owns [U*c/G, U*(c+1)/G).
// It visits the part of its last row tile first when that tile continues in the next CTA.
struct Range {
    int s0, s1, nq, n_tail, tail_start, st_first, st_last;
};
// 32-bit arithmetic: the launcher refuses shapes with n_su * (n_ctas + 1) >= 2^32
__host__ __device__ inline int range_begin(int c, int n_su, int n_ctas) { return (int)((uint32_t)n_su * (uint32_t)c / (uint32_t)n_ctas); }
__host__ __device__ inline int owner_of(int su, int n_su, int n_ctas) {
    return (int)((((uint32_t)su + 1u) * (uint32_t)n_ctas - 1u) / (uint32_t)n_su);
}
__host__ __device__ inline Range make_range(int c, int n_su, int n_ctas, int k_blocks) {
    Range r;
    r.s0 = range_begin(c, n_su, n_ctas);
    r.s1 = range_begin(c + 1, n_su, n_ctas);
    r.nq = r.s1 - r.s0;
    r.st_first = r.s0 / k_blocks;
    r.st_last = (r.s1 - 1) / k_blocks;
    r.tail_start = r.st_last * k_blocks;
    const bool tail_partial = (r.s1 % k_blocks) != 0 && r.st_first != r.st_last;
    r.n_tail = tail_partial ? r.s1 - r.tail_start : 0;
    return r;
}
__host__ __device__ inline int su_of(const Range& r, int q) { return q < r.n_tail ? r.tail_start + q : r.s0 + (q - r.n_tail); }
// which of the two parking slots of CTA c holds its part of row tile st
__host__ __device__ inline int slot_kind(int c, int st, int n_su, int n_ctas, int k_blocks) {
    const int s0 = range_begin(c, n_su, n_ctas), s1 = range_begin(c + 1, n_su, n_ctas);
    const int f = s0 / k_blocks, l = (s1 - 1) / k_blocks;
    return (st == l && f != l) ? 1 : 0;
}

// Position in a CTA's sequence of super-units, advanced without divisions (every warp of every role keeps one).
struct Cursor {
    int q, su, st, bk, s;
    uint32_t ph;   // parity of the pass over the stage ring
    __device__ __forceinline__ void init(const Range& r, int q0, int k_blocks, int n_stages) {
        q = q0; su = su_of(r, q0); st = su / k_blocks; bk = su - st * k_blocks; s = q0 % n_stages; ph = (uint32_t)(q0 / n_stages) & 1u;
    }
    __device__ __forceinline__ void next(const Range& r, int k_blocks, int n_stages) {
        ++q;
        if (++s == n_stages) { s = 0; ph ^= 1u; }
        if (q == r.n_tail) { su = r.s0; st = r.st_first; bk = r.s0 - r.st_first * k_blocks; }
        else { ++su; if (++bk == k_blocks) { bk = 0; ++st; } }
    }
    __device__ __forceinline__ void skip(int n, const Range& r, int k_blocks, int n_stages) {
        for (int i = 0; i < n; ++i) next(r, k_blocks, n_stages);
    }
};

// bf16 bits -> two e4m3 slices of x * scale; returns the packed hi bytes and lo bytes of four elements
__device__ __forceinline__ uint32_t cvt_e4m3x2(float hi_elem, float lo_elem) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi_elem), "f"(lo_elem));
    return r;
}
__device__ __forceinline__ void e4m3x2_to_f32(uint32_t v, float& lo_elem, float& hi_elem) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"((uint16_t)v));
    asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}"
        : "=f"(lo_elem), "=f"(hi_elem) : "r"(h2));
}
__device__ __forceinline__ void slice4(const uint32_t (&xb)[4], float scale, uint32_t& hi4, uint32_t& lo4) {
    float f[4], b[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) f[i] = __uint_as_float(xb[i] << 16) * scale;
    const uint32_t h01 = cvt_e4m3x2(f[1], f[0]), h23 = cvt_e4m3x2(f[3], f[2]);
    e4m3x2_to_f32(h01, b[0], b[1]);
    e4m3x2_to_f32(h23, b[2], b[3]);
    const uint32_t l01 = cvt_e4m3x2((f[1] - b[1]) * 16.f, (f[0] - b[0]) * 16.f);
    const uint32_t l23 = cvt_e4m3x2((f[3] - b[3]) * 16.f, (f[2] - b[2]) * 16.f);
    hi4 = h01 | (h23 << 16);
    lo4 = l01 | (l23 << 16);
}

#ifndef GOQ_TRQ0
#define GOQ_TRQ0 0   // first super-unit the optional timeline hooks record
#endif
#ifdef GOQ_TRACE
__device__ unsigned long long g_trace[kMaxCtas][kThreads / 32][16];
__device__ __forceinline__ unsigned long long gtime() { unsigned long long t; asm volatile("mov.u64 %0, %%clock64;" : "=l"(t)); return t; }
#define GOQ_TR(slot) do { if ((threadIdx.x & 31) == 0 && (slot) < 16) g_trace[blockIdx.x][threadIdx.x >> 5][slot] = gtime(); } while (0)
// timestamp taken only once `dep` has been computed
#define GOQ_TRD(slot, dep) do { unsigned long long t_; asm volatile("mov.u64 %0, %%clock64;" : "=l"(t_) : "r"(dep) : "memory"); \
    if ((threadIdx.x & 31) == 0 && (slot) < 16) g_trace[blockIdx.x][threadIdx.x >> 5][slot] = t_; } while (0)
#else
#define GOQ_TRD(slot, dep) do { } while (0)
#define GOQ_TR(slot) do { } while (0)
#endif

template <int WB, int GPB, int N>
__global__ void __launch_bounds__(kThreads, 1)
gemv_tc_kernel(const Params p) {
    // Four accumulators per buffer, index (h, beta): h = macro-block of the k-block when there are two, else the
    // parity of the 32-wide k slice. Consecutive MMAs then never accumulate into the same columns (an MMA
    // waits for the previous one on its accumulator), and the epilogue adds the two halves.
    constexpr int kBufCols = 64 + 4 * N;                       // A1 (32) + A2 (32) + accumulators
    constexpr int NB = (512 / kBufCols >= 4) ? 4 : 2;          // tensor-memory buffers in flight
    constexpr int kBTileBytes = N * 128;
    constexpr int MP = N / 2;                                  // tokens the B tile can hold
    static_assert(NB * kBufCols <= 512, "tensor memory budget");

    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const uint32_t raw = s32(smem_raw);
    const uint32_t base = raw + ((8192u - (raw & 8191u)) & 8191u);   // 8 KiB boundary for the OR-addressed table
    const uint32_t lut = base;
    const uint32_t b_tiles = lut + kLutBytes;                        // kXSlots x kBTileBytes, 1 KiB aligned
    const uint32_t stages = b_tiles + kXSlots * kBTileBytes;
    const int stage_bytes = kRowTiles * p.unit_bytes;
    const uint32_t coefbuf = stages + (uint32_t)p.n_stages * stage_bytes;   // [NB][GPB][128] words
    const uint32_t scales = coefbuf + NB * GPB * 128 * 4;                   // [kXSlots][16] floats
    unsigned char* gen = smem_raw + (scales + kXSlots * 16 * 4 - raw);
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen);
    uint64_t* full = bars;                          // [n_stages] records landed (tx bytes)
    uint64_t* empty = full + kMaxStages;            // [n_stages] expanders done with the stage
    uint64_t* a_ready = empty + kMaxStages;         // [NB] A tiles and coefficients written
    uint64_t* d_ready = a_ready + 4;                // [NB] MMAs of the buffer complete
    uint64_t* buf_free = d_ready + 4;               // [NB] epilogue has read the accumulators
    uint64_t* b_ready = buf_free + 4;               // [kXSlots] activation tile written
    uint64_t* b_free = b_ready + kXSlots;           // [kXSlots] tile and scales no longer needed
    uint64_t* epi_bar = b_free + kXSlots;           // rendezvous of the four epilogue warps (bounded, unlike bar.sync)
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile int abort_flag;
    __shared__ volatile int last_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    GOQ_TR(0);
    const int n_su = p.n_super * p.k_blocks, n_ctas = (int)gridDim.x, cta = (int)blockIdx.x;
    const Range R = make_range(cta, n_su, n_ctas, p.k_blocks);

    // The producer warp sets up the barriers and starts the weight stream at once (the first ring-full of
    // copies waits for nobody); the other warps fill the tables meanwhile.
    const int stage_fill = R.nq < p.n_stages ? R.nq : p.n_stages;
    auto issue = [&](const Cursor& c) {   // whole producer warp: lane r copies record r of the super-unit
        int n_rec = p.n_tiles - c.st * kRowTiles;
        if (n_rec > kRowTiles) n_rec = kRowTiles;
        if (lane == 0) mbar_expect_tx(&full[c.s], (uint32_t)n_rec * p.unit_bytes);
        __syncwarp();
        if (lane < n_rec)
            bulk_g2s(stages + c.s * stage_bytes + lane * p.unit_bytes,
                     p.packed + unit_offset(c.st * kRowTiles + lane, c.bk, p.k_blocks, p.unit_bytes), (uint32_t)p.unit_bytes, &full[c.s]);
    };
    Cursor pc;   // producer's position
    pc.init(R, 0, p.k_blocks, p.n_stages);
    if (warp == kWarpProducer) {
        if (lane == 0) abort_flag = 0;
        if (lane < p.n_stages) { mbar_init(&full[lane], 1); mbar_init(&empty[lane], kRowTiles); }
        if (lane < NB) { mbar_init(&a_ready[lane], kRowTiles); mbar_init(&d_ready[lane], 1); mbar_init(&buf_free[lane], kEpiWarps); }
        if (lane < kXSlots) { mbar_init(&b_ready[lane], 1); mbar_init(&b_free[lane], kEpiWarps); }
        if (lane == 0) mbar_init(epi_bar, kEpiWarps);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        __syncwarp();
        // the barriers exist: let the other warps go on without waiting for the first copies to be issued
        asm volatile("bar.arrive 2, %0;" ::"n"(kThreads) : "memory");
        GOQ_TR(2);
        for (int q = 0; q < stage_fill; ++q) { issue(pc); pc.next(R, p.k_blocks, p.n_stages); }
        GOQ_TR(3);
    } else {
        for (int i = tid - 32; i < 512; i += kThreads - 32) {  // entry i>>3, copy i&7 at byte (i>>3)*128 + (i&7)*16
            const uint32_t* e = c_lut.v[i >> 3];
            asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(lut + i * 16), "r"(e[0]), "r"(e[1]), "r"(e[2]), "r"(e[3]) : "memory");
        }
        for (int i = tid - 32; i < kXSlots * kBTileBytes / 4; i += kThreads - 32) sts32(b_tiles + i * 4, 0u);  // unused token rows stay 0
        GOQ_TR(2);
    }
    if (warp == kWarpMma) { tmem_alloc_512(&tmem_base_slot); GOQ_TR(3); }
    uint32_t tmem_base = 0;
    if (warp != kWarpProducer) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        tc_fence_before();
        asm volatile("bar.sync 2, %0;" ::"n"(kThreads) : "memory");
        tc_fence_after();
        tmem_base = tmem_base_slot;
    }
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    GOQ_TR(1);

    if (warp == kWarpProducer) {
        // ------------------------------------------------ producer ------------------------------------------------
        bool ok = true;
        int q = stage_fill;
        for (; q < R.nq; ++q) {
            if (lane == 0) ok = mbar_wait(&empty[pc.s], pc.ph ^ 1u, &abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            issue(pc);
            pc.next(R, p.k_blocks, p.n_stages);
            if (q >= GOQ_TRQ0 + 8 && q - GOQ_TRQ0 - 8 < 6) GOQ_TR(4 + q - GOQ_TRQ0 - 8);
        }
        GOQ_TR(14);
        if (lane == 0 && (!ok || abort_flag)) {
            // copies still in flight must land before the CTA's shared memory goes away
            const int first = q > p.n_stages ? q - p.n_stages : 0;
            for (int i = first; i < q; ++i) {
                const int s = i % p.n_stages;
                for (int it = 0; it < kSpin && !mbar_try(&full[s], (i / p.n_stages) & 1); ++it) { }
            }
        }
    } else if (warp == kWarpMma) {
        // ------------------------------------------------ MMA issuer ------------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_e4m3(N);
            for (int q = 0; q < R.nq; ++q) {
                const int buf = q % NB, xs = q % kXSlots;
                if (!mbar_wait(&a_ready[buf], (q / NB) & 1, &abort_flag)) break;
                if (!mbar_wait(&b_ready[xs], (q / kXSlots) & 1, &abort_flag)) break;
                if (q >= GOQ_TRQ0 && q - GOQ_TRQ0 < 5) GOQ_TR(4 + 2 * (q - GOQ_TRQ0));
                tc_fence_after();
                const uint64_t bdesc = smem_desc_sw128(b_tiles + xs * kBTileBytes);
                const uint32_t tb = tmem_base + buf * kBufCols;
#pragma unroll
                for (int jj = 0; jj < 2; ++jj)
#pragma unroll
                    for (int h = 0; h < 2; ++h)
#pragma unroll
                        for (int beta = 0; beta < 2; ++beta) {
                            const int j = (GPB == 2) ? h * 2 + jj : jj * 2 + h;   // 32-wide k slice of the k-block
                            umma_f8_ts(tb + 64 + (h * 2 + beta) * N, tb + beta * 32 + 8 * j, bdesc + 2 * j, idesc, jj > 0 ? 1u : 0u);
                        }
                umma_commit(&d_ready[buf]);
                if (q >= GOQ_TRQ0 && q - GOQ_TRQ0 < 5) GOQ_TR(5 + 2 * (q - GOQ_TRQ0));
            }
        }
    } else if (warp < kWarpExp0) {
        // ------------------------------------------------ activation slicer ------------------------------------------------
        const int xw = warp - kWarpX0;
        asm volatile("griddepcontrol.wait;" ::: "memory");
        const bool vec_ok = (p.k_in % 4) == 0;
        auto load_x = [&](int bk, int t) -> uint2 {   // four consecutive bf16 of token t in k-block bk
            const int k0 = bk * 128 + lane * 4;
            const uint16_t* xr = p.x + (size_t)t * p.k_in;
            uint2 v = make_uint2(0u, 0u);
            if (vec_ok && k0 + 3 < p.k_in) {
                v = *reinterpret_cast<const uint2*>(xr + k0);
            } else {
                uint32_t e[4] = {0u, 0u, 0u, 0u};
#pragma unroll
                for (int i = 0; i < 4; ++i) if (k0 + i < p.k_in) e[i] = xr[k0 + i];
                v = make_uint2(e[0] | (e[1] << 16), e[2] | (e[3] << 16));
            }
            return v;
        };
        auto put = [&](int xs, int t, uint2 v) {
            const uint32_t tile = b_tiles + xs * kBTileBytes;
            const uint32_t xb[4] = {v.x & 0xFFFFu, v.x >> 16, v.y & 0xFFFFu, v.y >> 16};
            uint32_t amax = max(max(xb[0] & 0x7FFFu, xb[1] & 0x7FFFu), max(xb[2] & 0x7FFFu, xb[3] & 0x7FFFu));
            amax = __reduce_max_sync(0xFFFFFFFFu, amax);
            // scale 2^s puts the block's largest magnitude in [2^7, 2^8): inside e4m3's range (max 448)
            int sfield = 261 - (int)(amax >> 7);
            sfield = sfield < 1 ? 1 : (sfield > 253 ? 253 : sfield);
            const float scale = __uint_as_float((uint32_t)sfield << 23);
            uint32_t hi4, lo4;
            slice4(xb, scale, hi4, lo4);
            // B tile row 2t = hi slice, row 2t+1 = lo slice; 16-byte chunk j of row r stored at chunk j ^ (r & 7)
            const int r_hi = 2 * t, r_lo = 2 * t + 1, ch = lane >> 2, wi = (lane & 3) * 4;
            sts32(tile + (r_hi >> 3) * 1024 + (r_hi & 7) * 128 + ((ch ^ (r_hi & 7)) << 4) + wi, hi4);
            sts32(tile + (r_lo >> 3) * 1024 + (r_lo & 7) * 128 + ((ch ^ (r_lo & 7)) << 4) + wi, lo4);
            if (lane == 0) sts32(scales + (xs * 16 + t) * 4, (uint32_t)(254 - sfield) << 23);   // 2^-s
        };
        // Each slicer warp takes super-units xw, xw + 2, ... two at a time (independent dependency chains), and for
        // small batches fetches the activations of the next pair while it converts the current one.
        constexpr int kPre = 4, kStep = 2 * kXWarps;
        const bool pre = p.m_total <= kPre;
        uint2 nxt[2][kPre];
        Cursor cx[2];   // the two super-units whose activations are fetched next
        cx[0].init(R, xw, p.k_blocks, p.n_stages);
        cx[1] = cx[0];
        cx[1].skip(kXWarps, R, p.k_blocks, p.n_stages);
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int t = 0; t < kPre; ++t)
                nxt[u][t] = (pre && t < p.m_total && cx[u].q < R.nq) ? load_x(cx[u].bk, t) : make_uint2(0u, 0u);
        for (int q = xw; q < R.nq; q += kStep) {
            uint2 cur[2][kPre];
            const int bkc[2] = {cx[0].bk, cx[1].bk};
#pragma unroll
            for (int u = 0; u < 2; ++u) {
#pragma unroll
                for (int t = 0; t < kPre; ++t) cur[u][t] = nxt[u][t];
                cx[u].skip(kStep, R, p.k_blocks, p.n_stages);
            }
            if (pre) {
#pragma unroll
                for (int u = 0; u < 2; ++u)
#pragma unroll
                    for (int t = 0; t < kPre; ++t)
                        if (t < p.m_total && cx[u].q < R.nq) nxt[u][t] = load_x(cx[u].bk, t);
            }
            bool ok = true;
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int qu = q + u * kXWarps;
                if (qu < R.nq && qu >= kXSlots) ok = ok && warp_wait(&b_free[qu % kXSlots], ((qu / kXSlots) - 1) & 1, &abort_flag);
            }
            if (!ok) break;
            if (q >= GOQ_TRQ0 && (q - GOQ_TRQ0) / kStep < 5) GOQ_TR(4 + 2 * ((q - GOQ_TRQ0) / kStep));
            const bool two = q + kXWarps < R.nq;
            const int xs0 = q % kXSlots, xs1 = (q + kXWarps) % kXSlots;
            if (pre) {
#pragma unroll
                for (int t = 0; t < kPre; ++t) {
                    if (t < p.m_total) {
                        put(xs0, t, cur[0][t]);
                        if (two) put(xs1, t, cur[1][t]);
                    }
                }
            } else {
                for (int t0 = 0; t0 < p.m_total; t0 += 4) {
                    uint2 v[2][4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        v[0][i] = (t0 + i < p.m_total) ? load_x(bkc[0], t0 + i) : make_uint2(0u, 0u);
                        v[1][i] = (two && t0 + i < p.m_total) ? load_x(bkc[1], t0 + i) : make_uint2(0u, 0u);
                    }
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (t0 + i < p.m_total) {
                            put(xs0, t0 + i, v[0][i]);
                            if (two) put(xs1, t0 + i, v[1][i]);
                        }
                    }
                }
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> tensor-core reads
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&b_ready[xs0]);
                if (two) mbar_arrive(&b_ready[xs1]);
            }
            if (q >= GOQ_TRQ0 && (q - GOQ_TRQ0) / kStep < 5) GOQ_TR(5 + 2 * ((q - GOQ_TRQ0) / kStep));
        }
    } else if (warp < kWarpEpi0) {
        // ------------------------------------------------ expanders ------------------------------------------------
        const int e = warp - kWarpExp0, team = e / kRowTiles, j = e % kRowTiles;   // j: record of the super-unit
        // (warp % 4) == (j % 4) selects the 32-lane quarter of tensor memory this warp may touch; j / 4 its half
        const uint32_t lane_base = (uint32_t)(32 * (j & 3) + 16 * (j >> 2));
        const uint32_t lut_lane = lut | ((uint32_t)(lane & 7) << 4);
        // The words of the next super-unit are fetched while this one's bytes go to tensor memory.
        uint4 wv0 = make_uint4(0u, 0u, 0u, 0u), wv1 = wv0;
        uint32_t cw[GPB];
        bool valid = false;
        // blocking = false: take the words only if they have already landed (returns whether they were taken)
        auto fetch = [&](const Cursor& c, bool blocking) -> bool {
            if (blocking) {
                if (!warp_wait(&full[c.s], c.ph, &abort_flag)) return false;
            } else {
                bool there = true;
                if (lane == 0) there = mbar_try(&full[c.s], c.ph);
                if (!__all_sync(0xFFFFFFFFu, there)) return false;
            }
            valid = c.st * kRowTiles + j < p.n_tiles;
            const uint32_t unit = stages + c.s * stage_bytes + j * p.unit_bytes;
            if (valid) {
                wv0 = lds128_v(unit + lane * 16);
                wv1 = lds128_v(unit + 512 + lane * 16);
                if (lane < 16) {
#pragma unroll
                    for (int gi = 0; gi < GPB; ++gi) cw[gi] = lds32_v(unit + kCodeBytesPerUnit + gi * 64 + lane * 4);
                }
            }
            return true;
        };
#pragma unroll
        for (int gi = 0; gi < GPB; ++gi) cw[gi] = 0u;
        bool ok = true, have = false;
        Cursor ec, en;   // this super-unit and the team's next one
        ec.init(R, team, p.k_blocks, p.n_stages);
        en = ec;
        en.skip(kTeams, R, p.k_blocks, p.n_stages);
        for (int q = team; q < R.nq; q += kTeams) {
            const int s = ec.s, buf = q % NB;
            if (!have) ok = fetch(ec, true);
            if (!ok) break;
            if (q >= GOQ_TRQ0 && (q - GOQ_TRQ0) / kTeams < 2) GOQ_TRD(4 + 5 * ((q - GOQ_TRQ0) / kTeams), wv0.x ^ wv1.w);
            uint32_t a1[16], a2[16], cwc[GPB];
#pragma unroll
            for (int gi = 0; gi < GPB; ++gi) cwc[gi] = valid ? cw[gi] : 0u;
            if (valid) {
                const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {   // micro-block 4c + (lane & 3): rows (lane >> 2) and (lane >> 2) + 8
                    decode_word<WB>(w0[c], lut_lane, a1[4 * c], a1[4 * c + 1], a2[4 * c], a2[4 * c + 1]);
                    decode_word<WB>(w1[c], lut_lane, a1[4 * c + 2], a1[4 * c + 3], a2[4 * c + 2], a2[4 * c + 3]);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) { a1[i] = 0u; a2[i] = 0u; }
            }
            if (q >= GOQ_TRQ0 && (q - GOQ_TRQ0) / kTeams < 2) GOQ_TRD(5 + 5 * ((q - GOQ_TRQ0) / kTeams), a2[0] ^ a2[15] ^ a2[7] ^ a1[9]);
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);   // the record is in registers
            have = (en.q < R.nq) ? fetch(en, false) : false;
            ec = en;
            en.skip(kTeams, R, p.k_blocks, p.n_stages);
            if (q >= GOQ_TRQ0 && (q - GOQ_TRQ0) / kTeams < 2) GOQ_TR(6 + 5 * ((q - GOQ_TRQ0) / kTeams));
            if (q >= NB) ok = warp_wait(&buf_free[buf], ((q / NB) - 1) & 1, &abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t ta = tmem_base + (lane_base << 16) + (uint32_t)(buf * kBufCols);
            tmem_st_16x256b_x4(ta, a1);
            tmem_st_16x256b_x4(ta + 32, a2);
            if (lane < 16) {
#pragma unroll
                for (int gi = 0; gi < GPB; ++gi) sts32(coefbuf + ((buf * GPB + gi) * 128 + j * 16 + lane) * 4, cwc[gi]);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&a_ready[buf]);
            if (q >= GOQ_TRQ0 && (q - GOQ_TRQ0) / kTeams < 2) GOQ_TR(7 + 5 * ((q - GOQ_TRQ0) / kTeams));
        }
    } else {
        // ------------------------------------------------ epilogue ------------------------------------------------
        const int ew = warp - kWarpEpi0;                                   // == warp % 4: tensor-memory quarter
        const int row_in_su = 16 * (ew + 4 * (lane >> 4)) + (lane & 15);   // record j = ew + 4*half, row lane%16 of it
        float acc[MP];
#pragma unroll
        for (int t = 0; t < MP; ++t) acc[t] = 0.f;
        int seg_first_bk = -1;
        bool waited = false;
        Cursor pe;
        pe.init(R, 0, p.k_blocks, p.n_stages);
        uint32_t epi_phase = 0;
        auto epi_sync = [&]() -> bool {
            __syncwarp();
            if (lane == 0) mbar_arrive(epi_bar);
            const bool ok = warp_wait(epi_bar, epi_phase & 1, &abort_flag);
            ++epi_phase;
            return ok;
        };
        for (int q = 0; q < R.nq; ++q) {
            const int buf = q % NB, xs = q % kXSlots;
            const int st = pe.st, bk = pe.bk;
            pe.next(R, p.k_blocks, p.n_stages);
            if (seg_first_bk < 0) seg_first_bk = bk;
            if (!warp_wait(&d_ready[buf], (q / NB) & 1, &abort_flag)) break;
            if (q >= GOQ_TRQ0 && q - GOQ_TRQ0 < 5) GOQ_TR(4 + 2 * (q - GOQ_TRQ0));
            tc_fence_after();
            const uint32_t td = tmem_base + ((uint32_t)(32 * ew) << 16) + (uint32_t)(buf * kBufCols + 64);
            float part[MP];
#pragma unroll
            for (int t = 0; t < MP; ++t) part[t] = 0.f;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int gi = (GPB == 2) ? h : 0;
                const uint32_t cfw = lds32_v(coefbuf + ((buf * GPB + gi) * 128 + row_in_su) * 4);
                const float c1 = __half2float(__ushort_as_half((unsigned short)(cfw & 0xFFFFu)));
                const float c2 = __half2float(__ushort_as_half((unsigned short)(cfw >> 16)));
#pragma unroll
                for (int beta = 0; beta < 2; ++beta) {
                    const float cb = beta ? c2 : c1;
#pragma unroll
                    for (int hh = 0; hh < N / 16; ++hh) {
                        uint32_t d[16];
                        tmem_ld16(td + (h * 2 + beta) * N + hh * 16, d);
                        tmem_wait_ld();
#pragma unroll
                        for (int tt = 0; tt < 8; ++tt)   // columns 2t (hi slice), 2t+1 (lo slice, scaled by 16)
                            part[hh * 8 + tt] = fmaf(cb, fmaf(__uint_as_float(d[2 * tt + 1]), 0.0625f, __uint_as_float(d[2 * tt])), part[hh * 8 + tt]);
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < MP; ++t)
                if (t < p.m_total) acc[t] = fmaf(__uint_as_float(lds32_v(scales + (xs * 16 + t) * 4)), part[t], acc[t]);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(&buf_free[buf]); mbar_arrive(&b_free[xs]); }
            if (q >= GOQ_TRQ0 && q - GOQ_TRQ0 < 5) GOQ_TR(5 + 2 * (q - GOQ_TRQ0));

            const bool seg_end = (q == R.nq - 1) || (q == R.n_tail - 1) || (bk == p.k_blocks - 1);
            if (!seg_end) continue;
            // ---- a segment of row tile st is complete: write it out, or park it for the CTA that arrives last ----
            if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
            const bool whole = (seg_first_bk == 0) && (bk == p.k_blocks - 1);
            const int row = st * 128 + row_in_su;
            bool store = whole;
            if (!whole) {
                const int kind = slot_kind(cta, st, n_su, n_ctas, p.k_blocks);
                float* mine = p.partials + (size_t)(cta * 2 + kind) * kSlotFloats;
#pragma unroll
                for (int t = 0; t < MP; ++t) if (t < p.m_total) mine[t * 128 + row_in_su] = acc[t];
                // the rendezvous orders every thread's stores before thread 0's device-scope release below
                if (!epi_sync()) break;
                const int c_first = owner_of(st * p.k_blocks, n_su, n_ctas);
                const int c_last = owner_of(st * p.k_blocks + p.k_blocks - 1, n_su, n_ctas);
                if (ew == 0 && lane == 0) {
                    const int prev = atomic_add_acq_rel_gpu(&p.counters[st], 1);
                    const int is_last = (prev == c_last - c_first) ? 1 : 0;
                    if (is_last) p.counters[st] = 0;   // left zero for the next call
                    last_flag = is_last;
                }
                if (!epi_sync()) break;   // ... and thread 0's acquire before everyone's loads
                store = last_flag != 0;
                if (store) {
#pragma unroll
                    for (int t = 0; t < MP; ++t) acc[t] = 0.f;
                    for (int c0 = c_first; c0 <= c_last; c0 += 8) {   // fixed order: the sum does not depend on who is last
                        const float* src[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const int c = (c0 + i <= c_last) ? c0 + i : c_last;
                            src[i] = p.partials + (size_t)(c * 2 + slot_kind(c, st, n_su, n_ctas, p.k_blocks)) * kSlotFloats + row_in_su;
                        }
#pragma unroll
                        for (int t = 0; t < MP; ++t) {
                            if (t < p.m_total) {
                                float v[8];
#pragma unroll
                                for (int i = 0; i < 8; ++i) v[i] = __ldcg(src[i] + t * 128);
#pragma unroll
                                for (int i = 0; i < 8; ++i) if (c0 + i <= c_last) acc[t] += v[i];
                            }
                        }
                    }
                }
                if (!epi_sync()) break;   // last_flag may be rewritten only after everyone has read it
            }
            if (store && row < p.n_out) {
#pragma unroll
                for (int t = 0; t < MP; ++t) {
                    if (t < p.m_total) {
                        if (p.y_dtype == GOQ_F32) reinterpret_cast<float*>(p.y)[(size_t)t * p.n_out + row] = acc[t];
                        else reinterpret_cast<uint16_t*>(p.y)[(size_t)t * p.n_out + row] = f32_to_bf16_rne(acc[t]);
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < MP; ++t) acc[t] = 0.f;
            seg_first_bk = -1;
        }
    }
    GOQ_TR(15);
    tc_fence_before();
    __syncthreads();
    if (warp == kWarpMma) {
        tc_fence_after();
        tmem_dealloc_512(tmem_base);
    }
    if (tid == 0 && abort_flag) atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
}

// ---- host side -------------------------------------------------------------------------------------
static int sm_count() {
    static int cached[64];
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64) dev = 0;
    if (cached[dev] == 0) {
        int n = 0;
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        cached[dev] = n > 0 ? n : 148;
    }
    return cached[dev];
}

static size_t smem_fixed(int gpb, int n) {
    const int buf_cols = 64 + 4 * n, nb = (512 / buf_cols >= 4) ? 4 : 2;
    return 8192 /* alignment slack */ + kLutBytes + (size_t)kXSlots * n * 128 + (size_t)nb * gpb * 128 * 4 + kXSlots * 16 * 4 + 512;
}

template <int WB, int GPB, int N>
static cudaError_t launch_cfg(const Geometry& g, Params p, cudaStream_t st) {
    const int n_su = p.n_super * p.k_blocks;
    if ((unsigned long long)n_su * (kMaxCtas + 1) >= (1ull << 32)) return cudaErrorInvalidValue;
    int grid = sm_count();
    if (grid > kMaxCtas) grid = kMaxCtas;
    if (grid > n_su) grid = n_su;
    const int stage_bytes = kRowTiles * g.unit_bytes;
    const size_t fixed = smem_fixed(GPB, N);
    int n_stages = (int)((200 * 1024 - fixed) / stage_bytes);
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    const int need = (n_su + grid - 1) / grid + 1;
    if (n_stages > need) n_stages = need;
    if (n_stages < 2) n_stages = 2;
    p.n_stages = n_stages;
    const size_t smem = fixed + (size_t)n_stages * stage_bytes;
    auto kernel = gemv_tc_kernel<WB, GPB, N>;
    static SmemAttrCache smem_attr;
    if (cudaError_t e = ensure_dynamic_smem(kernel, smem, smem_attr)) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

template <int WB>
static cudaError_t launch_wb(const Geometry& g, const Params& p, cudaStream_t st) {
    const bool wide = p.m_total > 8;
    if (g.group == 128) return wide ? launch_cfg<WB, 1, 32>(g, p, st) : launch_cfg<WB, 1, 16>(g, p, st);
    return wide ? launch_cfg<WB, 2, 32>(g, p, st) : launch_cfg<WB, 2, 16>(g, p, st);
}

}  // namespace gtc

bool gemv_tc_supported(const Geometry& g, int m) {
    return g.wbits <= 3 && (g.group == 128 || g.group == 64) && m >= 1 && m <= 16 && (size_t)g.n_tiles * 4 <= kWsCounterBytes;
}
size_t gemv_tc_workspace(const Geometry& g) { return gtc::ws_layout(g).total; }

cudaError_t launch_gemv_tc(const Geometry& g, const void* packed, const void* x, int m, void* y, int y_dtype, void* ws,
                           cudaStream_t st) {
    const gtc::Ws L = gtc::ws_layout(g);
    auto* wsb = (uint8_t*)ws;
    gtc::Params p;
    p.packed = (const uint8_t*)packed;
    p.x = (const uint16_t*)x;
    p.y = y;
    p.status = (int*)wsb;
    p.counters = (int*)(wsb + L.counters_off);
    p.partials = (float*)(wsb + L.partials_off);
    p.unit_bytes = g.unit_bytes;
    p.k_blocks = g.k_blocks;
    p.n_tiles = g.n_tiles;
    p.n_super = (g.n_tiles + gtc::kRowTiles - 1) / gtc::kRowTiles;
    p.k_in = g.k_in;
    p.n_out = g.n_out;
    p.m_total = m;
    p.y_dtype = y_dtype;
    p.n_stages = 0;
    return g.wbits == 3 ? gtc::launch_wb<3>(g, p, st) : gtc::launch_wb<2>(g, p, st);
}

}  // namespace goq
