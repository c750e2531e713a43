// A chain of decode GEMVs (batch <= 8) in ONE persistent kernel: one CTA per SM, resident for the whole chain.
//
// Work split. The unit records of a linear (16 rows x 128 k each, Section 3.1's macro-blocks tiled 16 rows high)
// are numbered tile by tile, k-block by k-block, which is also their order in the packed buffer. CTA c of G takes
// the contiguous range [U c / G, U (c+1) / G) of the U records of every linear: equal bytes per SM whatever the
// shape. A range is consumed 16 records at a time (one ring stage = one bulk copy), record w of a stage by
// consumer warp w; a last stage of n < 16 records is shared out so that 16 / n warps take a run of 32-wide k-chunks
// of the same record each (no warp visits more than one).
//
// Roles. 16 consumer warps do the arithmetic and touch global memory only to read activations. One producer
// thread keeps the weight stream going, across the boundaries between linears too (weights do not depend on
// results). One control warp does everything else that waits on global memory: per 16-row tile part it adds the
// 16 partial sums the consumer warps parked in shared memory (fixed pairing) and stores the outputs; a tile whose
// records fall into several CTAs is finished by the CTA that holds its end, the others post their part in scratch
// (each value in one 64-bit word together with a per-launch tag: no fence, no counter), and the finisher adds the
// parts in a fixed order - deterministic. A range that ends inside a tile is walked starting with that open tile, so
// the posted parts are early and a finisher waits only on lower-numbered CTAs.
//
// Order between linears. (a) Data flow: a linear whose activations lie inside an earlier linear's bf16 output reads
// them from a copy of that output in scratch, in which two values share a 64-bit word with the launch's tag. The
// finisher of a tile writes those words with plain relaxed stores; a reader polls exactly the words it converts until
// they carry the tag. That is the whole hand-over: no fence, no counter, and a reader waits for the tiles it needs, not
// for the linear. (b) Counter: the control warp reports every linear finished on a device-wide counter (release), and
// before a linear flagged `depends` (or whose buffers overlap earlier ones in a way (a) does not cover) waits until
// every CTA has. The host decides between the two from the address ranges of the items.
//
// A lone warp runs at instruction latency, and at the start and the end of a small linear every warp is alone on the
// critical path. So the kernel never divides (quotients and reciprocals come from the host), the control warp works
// out every address before it waits for a part and fetches the lower CTAs' parts ahead of its own.
//
// Math per record (Eq. 4 of the paper, integer operands): every PoT state times 2^emax is a small integer, so b1
// is one byte-table lookup per four weights; b2 = the same bytes routed by "partner i XOR s" (Section 3.3) with
// the pair signs applied as  sum_k q_k x_k - 2 sum_{k flipped} q_k x_k : the second operand is the first one
// masked, which costs one AND per register (a flipped zero contributes 0 - 0). The activations of a token and a
// 128-wide k-block are 16-bit fixed point Q = 256 q0 + q1 (two int8 columns of the MMA's B operand), the sums are
// exact in int32, and the coefficient multiply happens once per macro-block in fp32, outside the inner product.
//
// Every wait is bounded; on expiry an abort flag is raised, every role leaves its loops (all waits watch the flag),
// copies in flight are drained and GOQ_ERR_TIMEOUT is written to the status word.
#include "goq_stream_core.cuh"
#include "goq_internal.h"
#include <vector>

namespace goq {
namespace chain {

constexpr int kNW = 16;                      // consumer warps
constexpr int kCtrlWarp = kNW;               // polls the completion counters
constexpr int kProdWarp = kNW + 1;           // issues the bulk copies
constexpr int kThreads = (kNW + 2) * 32;
constexpr int kStageRecs = kNW;
constexpr int kTileSlots = 4;                // in-CTA reduction slots (tile parts in flight)
constexpr int kXPad = 32;                    // bytes between activation planes beyond k_pad: keeps the B-fragment loads conflict-free
constexpr int kMaxKBlocks = 96;              // activation scales kept per k-block: k_in <= 12288
constexpr int kGlobalSpin = 1 << 20;
constexpr int kMaxStages = 8;

struct Item {
    const uint8_t* packed;
    const uint16_t* x;
    void* y;
    unsigned long long kb_magic;             // ceil(2^32 / k_blocks): record number -> tile by multiply and shift (exact while units * k_blocks < 2^32)
    unsigned int units;                      // n_tiles * k_blocks
    int n_tiles, k_blocks, k_in, n_out, m, y_dtype, depends;
    int xsrc;                                // earlier item whose output this item's x lies in (read from that item's tagged copy), or -1
    unsigned int xoff;                       // first 64-bit word of x inside that copy
    int tag_out;                             // a later item reads this item's output: keep the tagged copy
    unsigned int uq, ur;                     // units / G and units % G for the launch's G CTAs (the kernel never divides)
};
struct Params {
    Item item[kSeqMaxItems];
    int n_items, unit_bytes, n_stages, x_double, xbuf_bytes, spin_limit;
    unsigned long long g_magic;   // ceil(2^32 / G): n / G for n < G^2 by multiply and shift
    int* status;
    int* done;       // [n_items] CTAs that have finished each linear; zero on entry, left zero
    unsigned* epoch; // launches this scratch buffer has seen: tags the posted parts (zero-filled scratch carries no valid tag)
    uint2* parts;    // [n_items][G][2][32 lanes x 2 NG] posted partial sums, each value in one 64-bit word with its tag
    uint2* tags;     // [n_items][kTagWords] tagged copies of bf16 outputs: [token][16 n_tiles / 2] words of (two values, tag)
};

// Split of a last stage of n < 16 records over the 16 consumer warps: 16 / n warps share a record, each a run of its four chunks.
struct TailShare { unsigned short v[16][16]; };
constexpr TailShare make_tail_share() {
    TailShare t{};
    for (int n = 1; n < 16; ++n) {
        const int wpr = 16 / n;
        for (int w = 0; w < 16; ++w) {
            const int rloc = w / wpr, sub = w - rloc * wpr;
            const int cb = 4 * sub / wpr, ce = 4 * (sub + 1) / wpr;
            t.v[n][w] = (unsigned short)(rloc < n ? (rloc | (cb << 4) | (ce << 7)) : 15);   // 15: no share (first chunk = end chunk = 0)
        }
    }
    return t;
}
__constant__ TailShare c_tail_share = make_tail_share();

constexpr int kPartWords = 128;              // 64-bit (value, tag) words of one posted part: 16 rows x 8 tokens
constexpr int kTagWords = 4 * (kMaxKBlocks * kBlockK / 2);   // per item: four tokens of the widest input a linear can take
constexpr int kXBatch = 3;                   // 16-byte activation chunks a lane holds while it polls their tags

// ---- small helpers ---------------------------------------------------------------------------------
template <int WB> struct IntTables;
template <> struct IntTables<3> { static constexpr uint32_t P0 = 0x00020408u, P1 = 0xFFFEFCF8u; };  // 8 4 2 0 -8 -4 -2 -1
template <> struct IntTables<2> { static constexpr uint32_t P0 = 0xFFFE0002u, P1 = 0u; };           // 2 0 -2 -1

// volatile: stays behind the waits (also volatile) that make the activation planes valid
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ void mma_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float ld_cg_f32(const float* p) {
    float v;
    asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
    return v;
}
// mbarrier operations by 32-bit shared-window address (no generic-to-shared conversion in the hot loop)
__device__ __forceinline__ bool try_wait_a(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void arrive_a(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// slow path of a wait whose first probe failed: bounded, gives up when another thread has
__device__ __noinline__ bool wait_slow_a(uint32_t bar, uint32_t parity, volatile int* abort_flag, int limit) {
    for (int it = 0; it < limit; ++it) {
        if (try_wait_a(bar, parity)) return true;
        if ((it & 63) == 63 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
// the same bounded wait, inlined (start-of-linear waits: a call would sit on the critical path)
__device__ __forceinline__ bool wait_a(uint32_t bar, uint32_t parity, volatile int* abort_flag, int limit) {
    for (int it = 0; it < limit; ++it) {
        if (try_wait_a(bar, parity)) return true;
        if ((it & 63) == 63 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ float lds_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ bool wait_bar(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int limit) {
    for (int it = 0; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63) == 63 && *abort_flag) return false;
    }
    *abort_flag = 1;
    return false;
}

// One micro-block word -> int8 operands (value * 2^emax): b1 (pa: weights 0..3, pb: 4..7), the routed bytes of
// b2 (qa, qb) and the same bytes at the sign-flipped positions only (fa, fb).
template <int WB, bool K1>
__device__ __forceinline__ void decode_word(uint32_t w, uint32_t lut_lane, uint32_t& pa, uint32_t& pb, uint32_t& qa,
                                            uint32_t& qb, uint32_t& fa, uint32_t& fb) {
    const uint32_t m = w & 0x77777777u, mh = m >> 16;
    pa = prmt_b32(IntTables<WB>::P0, IntTables<WB>::P1, m);
    pb = prmt_b32(IntTables<WB>::P0, IntTables<WB>::P1, mh);
    if constexpr (K1) {   // single-basis weights (Section 3.1, w_hat = c1 b1): no second operand
        qa = qb = fa = fb = 0u;
    } else {
        const uint32_t h = (w & 0x88888888u) * kHashMul;
        const uint4 e = lds128(((h >> 19) & 0x1F80u) | lut_lane);   // selectors x, y; 0xFF at the flipped bytes z, w
        qa = prmt_b32(pa, pb, e.x);
        qb = prmt_b32(pa, pb, e.y);
        fa = qa & e.z;
        fb = qb & e.w;
    }
}

// The range of CTA `cta` of `G` over `units` records, and the order it is walked in.
struct Walk {
    unsigned a, b, L;        // range [a, b), length
    unsigned L1, s1;         // the first L1 positions are records s1, s1+1, ... (the open tile at the end of the range); then a, a+1, ...
    int Ta, Tb, P;           // first and last tile touched, number of tile parts
    bool rot;
};
// No division anywhere: every warp works this out at the start of every linear, on the critical path of a chain of small ones.
__device__ __forceinline__ unsigned mul_shift32(unsigned n, unsigned long long magic) { return (unsigned)(((unsigned long long)n * magic) >> 32); }
__device__ __forceinline__ Walk make_walk(const Item& it, int cta, unsigned long long g_magic) {
    Walk w;
    // floor(units c / G) = c (units / G) + floor(c (units % G) / G)
    w.a = (unsigned)cta * it.uq + mul_shift32((unsigned)cta * it.ur, g_magic);
    w.b = (unsigned)(cta + 1) * it.uq + mul_shift32((unsigned)(cta + 1) * it.ur, g_magic);
    w.L = w.b - w.a;
    w.L1 = 0; w.s1 = 0; w.Ta = 0; w.Tb = 0; w.P = 0; w.rot = false;
    if (w.L) {
        const unsigned kb = (unsigned)it.k_blocks;
        w.Ta = (int)mul_shift32(w.a, it.kb_magic);
        w.Tb = (int)mul_shift32(w.b - 1, it.kb_magic);
        w.P = w.Tb - w.Ta + 1;
        w.rot = w.Tb > w.Ta && w.b != mul_shift32(w.b, it.kb_magic) * kb;
        if (w.rot) { w.s1 = (unsigned)w.Tb * kb; w.L1 = w.b - w.s1; }
    }
    return w;
}
__device__ __forceinline__ unsigned walk_record(const Walk& w, unsigned j) { return j < w.L1 ? w.s1 + j : w.a + (j - w.L1); }
__device__ __forceinline__ int walk_part_of_tile(const Walk& w, int T) { return w.rot ? (T == w.Tb ? 0 : 1 + T - w.Ta) : T - w.Ta; }
__device__ __forceinline__ int walk_tile_of_part(const Walk& w, int q) { return w.rot ? (q == 0 ? w.Tb : w.Ta + q - 1) : w.Ta + q; }

// ---- hand-over of one tile part (kept out of line) ------------------------------------------------------
// A consumer warp parks its sums of part number sq (counted per CTA over the whole chain) in reduction slot sq % kTileSlots
// and arrives on the slot's mbarrier; the control warp adds the 16 partials, stores or passes on the result and then
// frees the slot. Returns false after a give-up.
struct FlushCtx {
    uint32_t red_addr;        // shared-window addresses: no 64-bit pointers are kept alive across the record loop
    uint32_t part_bar_addr;
    volatile int* done_gen;
    volatile int* abort_flag;
    int spin;
};
struct Sums4 { float v[4]; };   // by value: the accumulators never have their address taken, so they stay in registers
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
template <int NG>
__device__ __forceinline__ bool flush_part(const FlushCtx& c, unsigned sq, Sums4 sums) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
    const int rs = (int)(sq % kTileSlots);
    if (*c.abort_flag) return false;
    if (sq >= (unsigned)kTileSlots) {   // the slot's previous part must have been taken over
        int spins = 0;
        while (c.done_gen[rs] != (int)(sq - kTileSlots + 1)) {
            if (*c.abort_flag || ++spins > c.spin) { *c.abort_flag = 1; return false; }
            __nanosleep(20);
        }
    }
    const uint32_t rb = c.red_addr + (uint32_t)(((rs * kNW + warp) * (NG * 64) + g * 4 + t) * 4);
#pragma unroll
    for (int cg = 0; cg < NG; ++cg) {
        sts_f32(rb + (cg * 64) * 4, sums.v[2 * cg]);
        sts_f32(rb + (cg * 64 + 32) * 4, sums.v[2 * cg + 1]);
    }
    __syncwarp();
    if (lane == 0) arrive_a(c.part_bar_addr + rs * 8);   // releases the warp's stores (ordered before it by the barrier above)
    return true;
}

// sums of one macro-block -> fp32, times the coefficients (outside the inner product, Eq. 4)
template <int NG, bool K1>
__device__ __forceinline__ void group_end(int (&s1)[NG][4], int (&s2)[NG][4], int (&s3)[NG][4], uint32_t cfa, uint32_t cfb, float (&rec)[NG][2]) {
    const float c1a = __half2float(__ushort_as_half((unsigned short)(cfa & 0xFFFFu)));
    const float c2a = __half2float(__ushort_as_half((unsigned short)(cfa >> 16)));
    const float c1b = __half2float(__ushort_as_half((unsigned short)(cfb & 0xFFFFu)));
    const float c2b = __half2float(__ushort_as_half((unsigned short)(cfb >> 16)));
#pragma unroll
    for (int cg = 0; cg < NG; ++cg) {
        // columns 2t, 2t+1 hold the high and low activation slices of one token: S = 256 S_hi + S_lo, exact in int32
        if constexpr (K1) {
            rec[cg][0] += c1a * (float)(s1[cg][0] * 256 + s1[cg][1]);
            rec[cg][1] += c1b * (float)(s1[cg][2] * 256 + s1[cg][3]);
        } else {
            rec[cg][0] += c1a * (float)(s1[cg][0] * 256 + s1[cg][1]) + c2a * (float)((s2[cg][0] - 2 * s3[cg][0]) * 256 + (s2[cg][1] - 2 * s3[cg][1]));
            rec[cg][1] += c1b * (float)(s1[cg][2] * 256 + s1[cg][3]) + c2b * (float)((s2[cg][2] - 2 * s3[cg][2]) * 256 + (s2[cg][3] - 2 * s3[cg][3]));
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) s1[cg][r] = s2[cg][r] = s3[cg][r] = 0;
    }
}

template <int WB, int CPG, int NG, bool K1>
__global__ void __launch_bounds__(kThreads, 1) gemv_chain_kernel(const __grid_constant__ Params p) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* lut = smem + ((8192u - (smem_u32(smem) & 8191u)) & 8191u);   // 8 KiB boundary: slot offsets are OR-ed in
    const int stage_bytes = kStageRecs * p.unit_bytes;
    unsigned char* ring = lut + kLutBytes;
    float* red = reinterpret_cast<float*>(ring + (size_t)p.n_stages * stage_bytes);     // [slot][warp][NG][64]
    float* xscale = red + kTileSlots * kNW * NG * 64;                                   // [2][k-block][4 NG tokens]
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(xscale + 2 * kMaxKBlocks * 4 * NG);
    uint64_t* empty_bar = full_bar + kMaxStages;
    uint64_t* dep_bar = empty_bar + kMaxStages;
    uint64_t* x_bar = dep_bar + 1;
    uint64_t* free_bar = x_bar + 1;
    uint64_t* part_bar = free_bar + 1;
    unsigned char* xq = reinterpret_cast<unsigned char*>(part_bar + kTileSlots);                 // [2][2 m][k_pad + kXPad] int8 planes
    __shared__ volatile int abort_flag;
    __shared__ volatile int done_gen[kTileSlots];
    __shared__ unsigned tag_s;   // the launch's tag, for the consumer warps (one register less across the record loop)

    // the broadcast tells the compiler that the warp index (and everything derived from it) is uniform across the warp
    const int tid = threadIdx.x, warp = __shfl_sync(0xFFFFFFFFu, tid >> 5, 0), lane = tid & 31;
    const int G = (int)gridDim.x, cta = (int)blockIdx.x;
    const int spin = p.spin_limit;

    if (tid == 0) {
        abort_flag = 0;
        tag_s = ((*p.epoch + 1u) * 0x9E3779B1u) | 1u;   // nobody changes the count before every CTA has finished the last linear
        for (int i = 0; i < kTileSlots; ++i) { done_gen[i] = 0; mbar_init(&part_bar[i], kNW); }
        for (int s = 0; s < p.n_stages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kNW); }
        mbar_init(dep_bar, 1);
        mbar_init(x_bar, kNW);
        mbar_init(free_bar, kNW);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < 64 * kLutCopies; i += kThreads) {
        const uint32_t* e = c_exchange_lut.v[i / kLutCopies];
        *reinterpret_cast<uint4*>(lut + (size_t)i * 16) = make_uint4(e[0], e[1], (e[2] >> 7) * 255u, (e[3] >> 7) * 255u);
    }
    __syncthreads();

    // ================= producer: the weight stream of this CTA's ranges, linear after linear =================
    if (warp == kProdWarp) {
        if (lane == 0) {
            int slot = 0, round = 0, issued = 0;
            bool ok = true;
            for (int i = 0; i < p.n_items && ok; ++i) {
                const Item& it = p.item[i];
                const Walk wk = make_walk(it, cta, p.g_magic);
                for (unsigned j0 = 0; j0 < wk.L; j0 += kStageRecs) {
                    if (round > 0 && !wait_bar(&empty_bar[slot], (round - 1) & 1, &abort_flag, spin)) { ok = false; break; }
                    const unsigned n = min((unsigned)kStageRecs, wk.L - j0);
                    unsigned char* dst = ring + (size_t)slot * stage_bytes;
                    mbar_arrive_expect_tx(&full_bar[slot], n * (unsigned)p.unit_bytes);
                    // positions j0 .. j0+n-1 of the walk: one run of records, or two if the stage straddles the turn of the walk
                    const unsigned n1 = (j0 < wk.L1) ? min(n, wk.L1 - j0) : 0u;
                    if (n1) bulk_copy_g2s(dst, it.packed + (size_t)walk_record(wk, j0) * p.unit_bytes, n1 * (unsigned)p.unit_bytes, &full_bar[slot]);
                    if (n > n1)
                        bulk_copy_g2s(dst + (size_t)n1 * p.unit_bytes, it.packed + (size_t)walk_record(wk, j0 + n1) * p.unit_bytes,
                                      (n - n1) * (unsigned)p.unit_bytes, &full_bar[slot]);
                    if (++slot == p.n_stages) { slot = 0; ++round; }
                    ++issued;
                }
            }
            // after a give-up the copies this thread issued must still land before the CTA (and its shared memory) goes away
            if (!ok || abort_flag) {
                const int first = issued > p.n_stages ? issued - p.n_stages : 0;
                for (int s = first; s < issued; ++s) {
                    const int sl = s % p.n_stages;
                    const uint32_t parity = (uint32_t)(s / p.n_stages) & 1u;
                    for (int t = 0; t < kSpinLimit && !mbar_try_wait(&full_bar[sl], parity); ++t) { }
                }
                atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
            }
        }
        return;
    }

    // ================= control: everything that touches global memory apart from the activations =================
    // Per linear and tile part of this CTA: add the 16 parked partials in warp order; a part that covers its whole tile is
    // stored, another one is parked in scratch, and the last CTA of the tile to arrive adds all parts in CTA order and
    // stores. Then report the CTA finished; before a dependent linear, wait until every CTA has reported.
    if (warp == kCtrlWarp) {
        unsigned seq = 0;
        bool ok = true;
        // nobody changes the count before every CTA has finished the last linear; the tag is the count scrambled (and odd,
        // hence non-zero), so that neither zero-filled scratch nor small integers left by other kernels pass for it
        const unsigned epoch = *p.epoch, tag = ((epoch + 1u) * 0x9E3779B1u) | 1u;
        for (int i = 0; i < p.n_items && ok; ++i) {
            const Item& it = p.item[i];
            const Walk wk = make_walk(it, cta, p.g_magic);
            if (wk.L) {
                if (it.depends && i > 0) {
                    if (lane == 0) {
                        int spins = 0;
                        while (abort_flag == 0 && ld_acquire_gpu(&p.done[i - 1]) < G)
                            if (++spins > kGlobalSpin || spins > spin) { abort_flag = 1; break; }
                        if (abort_flag == 0) mbar_arrive(dep_bar);
                    }
                    __syncwarp();
                    if (abort_flag) { ok = false; break; }
                }
                // The control warp is alone on the critical path between the last arithmetic of a tile and the SMs that wait
                // for its outputs, and a lone warp runs at instruction latency: whatever does not need the sums (which tile, who
                // finishes it, every address) is worked out BEFORE the wait for the part, and nothing on the far side divides.
                const unsigned kb = (unsigned)it.k_blocks;
                const unsigned uq = it.uq, ur = it.ur;   // range boundaries step by uq (+1) from CTA to CTA
                const unsigned rem_a = (unsigned)cta * ur - (unsigned)G * mul_shift32((unsigned)cta * ur, p.g_magic);
                const int tok0 = lane & 3;
                const size_t tstride4 = (size_t)4 * (it.n_tiles * 8), ystride4 = (size_t)4 * it.n_out;
                const bool y32 = it.y_dtype == GOQ_F32;
                bool tokv[NG];
#pragma unroll
                for (int cg = 0; cg < NG; ++cg) tokv[cg] = cg * 4 + tok0 < it.m;
                const bool tagw = it.tag_out && (lane & 4) == 0;
                for (int q = 0; q < wk.P; ++q) {
                    const unsigned sq = seq + (unsigned)q;
                    const int rs = (int)(sq % kTileSlots);
                    const int T = walk_tile_of_part(wk, q);
                    const unsigned r_lo = (unsigned)T * kb, r_hi = r_lo + kb;
                    const bool whole = r_lo >= wk.a && r_hi <= wk.b;   // every record of the tile is this CTA's
                    const bool finisher = r_hi <= wk.b;                  // this CTA holds the tile's end
                    uint2* post = p.parts + (((size_t)i * G + cta) * 2 + (T == wk.Ta ? 0 : 1)) * kPartWords + lane;
                    uint2* tgp = p.tags + (size_t)i * kTagWords + (size_t)tok0 * (it.n_tiles * 8) + T * 8 + (lane >> 3);
                    const size_t yoff = (size_t)tok0 * it.n_out + T * 16 + (lane >> 2);
                    bool rowv[2];
                    rowv[0] = T * 16 + (lane >> 2) < it.n_out;
                    rowv[1] = T * 16 + (lane >> 2) + 8 < it.n_out;
                    const float* rall = red + (size_t)rs * kNW * (NG * 64) + lane;
                    // A tile this CTA finishes for others: their parts were posted early (every CTA starts with the tile that is
                    // open at the end of its range), so they are fetched now, before this CTA's own sums are ready - nearest CTA
                    // first, down to the one that holds the tile's first record.
                    float below[NG][2];
#pragma unroll
                    for (int cg = 0; cg < NG; ++cg) below[cg][0] = below[cg][1] = 0.f;
                    if (!whole && finisher) {
                        bool good = true;
                        unsigned bc = wk.a, remc = rem_a;   // upper boundary of CTA cc's range (= lower boundary of CTA cc + 1)
                        for (int cc = cta - 1; cc >= 0 && bc > r_lo && good; --cc) {
                            const unsigned borrow = remc < ur ? 1u : 0u;
                            const unsigned ac = bc - uq - borrow;
                            remc = remc - ur + (borrow ? (unsigned)G : 0u);
                            if (ac != bc) {   // CTA cc has records of this tile; they are its first tile's if its range starts inside
                                const uint2* pc = p.parts + (((size_t)i * G + cc) * 2 + (ac >= r_lo ? 0 : 1)) * kPartWords + lane;
                                int spins = 0;
                                for (;;) {
                                    uint2 w[NG][2];
                                    bool all = true;
#pragma unroll
                                    for (int cg = 0; cg < NG; ++cg)
#pragma unroll
                                        for (int hh = 0; hh < 2; ++hh) {
                                            asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(w[cg][hh].x), "=r"(w[cg][hh].y)
                                                         : "l"(pc + (cg * 2 + hh) * 32) : "memory");
                                            all = all && w[cg][hh].y == tag;
                                        }
                                    if (__all_sync(0xFFFFFFFFu, all)) {
#pragma unroll
                                        for (int cg = 0; cg < NG; ++cg) { below[cg][0] += __uint_as_float(w[cg][0].x); below[cg][1] += __uint_as_float(w[cg][1].x); }
                                        break;
                                    }
                                    ++spins;
                                    if (__any_sync(0xFFFFFFFFu, abort_flag != 0) || spins > kGlobalSpin || spins > spin) { abort_flag = 1; good = false; break; }
                                }
                            }
                            bc = ac;
                        }
                        if (!good) { ok = false; break; }
                    }
                    if (!wait_bar(&part_bar[rs], (sq / kTileSlots) & 1u, &abort_flag, spin)) { ok = false; break; }
                    float out[NG][2];
#pragma unroll
                    for (int cg = 0; cg < NG; ++cg)
#pragma unroll
                        for (int hh = 0; hh < 2; ++hh) {
                            float v[kNW];
#pragma unroll
                            for (int w2 = 0; w2 < kNW; ++w2) v[w2] = rall[(size_t)w2 * (NG * 64) + cg * 64 + hh * 32];
#pragma unroll
                            for (int sft = kNW / 2; sft >= 1; sft >>= 1)   // fixed pairing: deterministic
#pragma unroll
                                for (int w2 = 0; w2 < sft; ++w2) v[w2] += v[w2 + sft];
                            out[cg][hh] = v[0] + below[cg][hh];
                        }
                    __syncwarp();
                    if (lane == 0) done_gen[rs] = (int)(sq + 1);   // every lane has read the slot: it may be parked in again
                    if (!whole && !finisher) {
                        // The CTA that holds the end of the tile finishes it; the others post their part and go on. A posted
                        // value travels in one 64-bit word with the launch's tag, so it needs no fence and no counter: the
                        // finisher reads the words until the tag is there, and it waits only on lower-numbered CTAs (no cycle).
#pragma unroll
                        for (int cg = 0; cg < NG; ++cg)
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh)
                                asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(post + (cg * 2 + hh) * 32),
                                             "r"(__float_as_uint(out[cg][hh])), "r"(tag) : "memory");
                    } else {
                        // A later item reads this output: first the copy it polls. Two neighbouring channels (bf16, as in y)
                        // and the launch's tag share one 64-bit word, so a reader that sees the tag has the values - no fence
                        // and no counter between the finisher of a tile and the SMs that wait for it.
                        uint32_t pair[NG][2];
#pragma unroll
                        for (int cg = 0; cg < NG; ++cg)
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh) {
                                const float next = __shfl_down_sync(0xFFFFFFFFu, out[cg][hh], 4);   // channel + 1 of the same token
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pair[cg][hh]) : "f"(next), "f"(out[cg][hh]));
                                if (tagw && tokv[cg])
                                    asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(tgp + cg * tstride4 + hh * 4), "r"(pair[cg][hh]), "r"(tag) : "memory");
                            }
#pragma unroll
                        for (int cg = 0; cg < NG; ++cg)
#pragma unroll
                            for (int hh = 0; hh < 2; ++hh)
                                if (rowv[hh] && tokv[cg]) {
                                    const size_t o = yoff + cg * ystride4 + hh * 8;
                                    if (y32) reinterpret_cast<float*>(it.y)[o] = out[cg][hh];
                                    else reinterpret_cast<uint16_t*>(it.y)[o] = (uint16_t)(pair[cg][hh] & 0xFFFFu);   // the bits the copy carries
                                }
                    }
                }
                if (!ok) break;
                seq += (unsigned)wk.P;
            }
            // this CTA has finished linear i: the warp's stores are ordered before lane 0's fetch-add, which releases them
            __syncwarp();
            if (lane == 0) {
                if (i < p.n_items - 1) {
                    asm volatile("red.release.gpu.global.add.s32 [%0], 1;" ::"l"(&p.done[i]) : "memory");
                } else {   // the CTA that completes the last linear last leaves the counters zero for the next call
                    const int prev = atomic_add_acq_rel_gpu(&p.done[i], 1);
                    if (prev == G - 1) {
                        for (int j = 0; j < p.n_items; ++j) p.done[j] = 0;
                        *p.epoch = epoch + 1u;
                    }
                }
            }
        }
        if (lane == 0 && abort_flag) atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
        return;
    }

    // ================= consumers =================
    const int g = lane >> 2, t = lane & 3;
    const uint32_t lut_lane = smem_u32(lut) + (lane & (kLutCopies - 1)) * 16;
    const uint32_t ring_addr = smem_u32(ring), unit_bytes = (uint32_t)p.unit_bytes;
    const uint32_t full_addr = smem_u32(full_bar), empty_addr = smem_u32(empty_bar);
    const uint32_t dep_addr = smem_u32(dep_bar), xbar_addr = smem_u32(x_bar), free_addr = smem_u32(free_bar);
    int slot = 0, phase = 0;          // position in the stage ring ...
    uint32_t stage_off = 0, bar_off = 0;   // ... and the same as byte offsets of the stage and of its barriers
    const uint32_t unit0 = ring_addr + (uint32_t)warp * unit_bytes + (uint32_t)lane * 16;
    uint32_t phases = 0;              // bit 0: dependency barrier, bit 1: activation barrier, bit 2: buffer hand-shake, bit 3: activation buffer in use
    unsigned seq = 0;                 // tile parts this CTA has opened so far (same in every warp): indexes the reduction slots
    bool alive = true;

    for (int i = 0; i < p.n_items && alive; ++i) {
        const Item& it = p.item[i];
        const Walk wk = make_walk(it, cta, p.g_magic);
        if (wk.L == 0) continue;   // nothing of this linear belongs to this CTA (the control warp reports it finished)
        const int kb = it.k_blocks, k_pad = kb * kBlockK, plane = k_pad + kXPad, m = it.m;
        if (p.x_double) phases ^= 8u;
        const int x_sel = (int)((phases >> 3) & 1u);
        unsigned char* xb = xq + (size_t)x_sel * p.xbuf_bytes;
        float* xsc = xscale + x_sel * (kMaxKBlocks * 4 * NG);

        const unsigned n_full = wk.L / kStageRecs, n_tail = wk.L - n_full * kStageRecs;

        // ---- start of the linear: wait for the dependency, then every warp converts its slice of the activations ----
        if (it.depends && i > 0) {
            if (!wait_a(dep_addr, phases & 1u, &abort_flag, spin)) { alive = false; break; }
            phases ^= 1u;
        } else if (!p.x_double) {   // one buffer: every warp must have left the previous linear
            __syncwarp();
            if (lane == 0) arrive_a(free_addr);
            if (!wait_a(free_addr, (phases >> 2) & 1u, &abort_flag, spin)) { alive = false; break; }
            phases ^= 4u;
        }
        {
            // 16-byte chunks of 8 bf16; 16 chunks = one k-block of one token: Q = rne(x 2^s), the block's largest magnitude in [2^14, 2^15)
            const int cpt = k_pad / 8, total = cpt * m;
            auto convert = [&](const uint4 v, const bool in, const int r, const int k0) {
                const uint32_t in32[4] = {v.x, v.y, v.z, v.w};
                uint32_t amax = 0;
#pragma unroll
                for (int j = 0; j < 4; ++j) amax = max(amax, max(in32[j] & 0x7FFFu, (in32[j] >> 16) & 0x7FFFu));
#pragma unroll
                for (int o = 1; o < 16; o <<= 1) amax = max(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, o));
                int sfield = 268 - (int)(amax >> 7);
                sfield = sfield < 1 ? 1 : (sfield > 253 ? 253 : sfield);
                const float mult = __uint_as_float((uint32_t)sfield << 23);
                // Q = rne(x 2^s) without a convert: adding 1.5 * 2^23 leaves the integer in the low mantissa bits. With 128 more in
                // the constant the low 16 bits are 256 hi + (lo + 128) for the split Q = 256 hi + lo, lo in [-128, 127]: the high
                // byte is hi as it stands and the low byte is lo with its top bit flipped. Clamped as raw bits (monotonic):
                // Q = 32640 (all-ones mantissa at the block's top exponent) would need hi = 128; inf and nan saturate.
                uint32_t v16[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const uint32_t bits = (j & 1) ? (in32[j >> 1] & 0xFFFF0000u) : (in32[j >> 1] << 16);
                    const int raw = __float_as_int(fmaf(__uint_as_float(bits), mult, 12582912.0f + 128.0f));
                    v16[j] = (uint32_t)max(0x4B400000 + 128 - 32640, min(0x4B400000 + 128 + 32639, raw));
                }
                uint32_t q0[2], q1[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t t01 = prmt_b32(v16[4 * h], v16[4 * h + 1], 0x5410u), t23 = prmt_b32(v16[4 * h + 2], v16[4 * h + 3], 0x5410u);
                    q0[h] = prmt_b32(t01, t23, 0x7531u);                   // the four high bytes
                    q1[h] = prmt_b32(t01, t23, 0x6420u) ^ 0x80808080u;     // the four low bytes, as signed
                }
                if (in) {
                    *reinterpret_cast<uint2*>(xb + (size_t)(2 * r) * plane + k0) = make_uint2(q0[0], q0[1]);
                    *reinterpret_cast<uint2*>(xb + (size_t)(2 * r + 1) * plane + k0) = make_uint2(q1[0], q1[1]);
                    // 2^-s, and 2^-emax for the integer weights
                    if ((lane & 15) == 0) xsc[(k0 >> 7) * (4 * NG) + r] = __uint_as_float((uint32_t)(254 - sfield) << 23) * (1.0f / (float)(1 << ((1 << (WB - 1)) - 1)));
                }
            };
            if (it.xsrc < 0) {   // activations from outside the chain, or ordered by the counter wait above
                for (int c0 = warp * 32; c0 < total; c0 += kNW * 32) {
                    const int c = c0 + lane;
                    const bool in = c < total;
                    const int r = in ? (int)mul_shift32((unsigned)c >> 4, it.kb_magic) : 0, k0 = in ? (c - r * cpt) * 8 : 0;   // cpt = 16 k_blocks
                    uint4 v = make_uint4(0u, 0u, 0u, 0u);
                    if (in && k0 < it.k_in) v = __ldcg(reinterpret_cast<const uint4*>(it.x + (size_t)r * it.k_in + k0));   // L2: written by other SMs
                    convert(v, in, r, k0);
                }
            } else {
                // Activations that an earlier linear of this launch produces: read from its tagged copy, word by word,
                // until every word carries this launch's tag. That is the whole dependency wait: a chunk is converted as soon
                // as the tiles it comes from are finished, wherever they were finished.
                const unsigned tag = tag_s;
                const uint2* tg = p.tags + (size_t)it.xsrc * kTagWords + it.xoff;
                const int tstride = p.item[it.xsrc].n_tiles * 8;
                const int bound = spin < kGlobalSpin ? spin : kGlobalSpin;
                for (int cb = warp * 32; cb < total && alive; cb += kNW * 32 * kXBatch) {
                    uint4 v[kXBatch];
                    bool need[kXBatch];
#pragma unroll
                    for (int u = 0; u < kXBatch; ++u) {
                        const int c = cb + u * (kNW * 32) + lane;
                        const int r = c < total ? (int)mul_shift32((unsigned)c >> 4, it.kb_magic) : 0, k0 = c < total ? (c - r * cpt) * 8 : 0;
                        need[u] = c < total && k0 < it.k_in;
                        v[u] = make_uint4(0u, 0u, 0u, 0u);
                    }
                    int spins = 0;
                    for (;;) {
                        bool ok = true;
#pragma unroll
                        for (int u = 0; u < kXBatch; ++u)
                            if (need[u]) {
                                const int c = cb + u * (kNW * 32) + lane;
                                const int r = (int)mul_shift32((unsigned)c >> 4, it.kb_magic), k0 = (c - r * cpt) * 8;
                                const uint2* src = tg + (size_t)r * tstride + (k0 >> 1);
                                unsigned long long w0, w1, w2, w3;
                                asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(w0), "=l"(w1) : "l"(src) : "memory");
                                asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(w2), "=l"(w3) : "l"(src + 2) : "memory");
                                if ((unsigned)(w0 >> 32) == tag && (unsigned)(w1 >> 32) == tag && (unsigned)(w2 >> 32) == tag && (unsigned)(w3 >> 32) == tag) {
                                    v[u] = make_uint4((unsigned)w0, (unsigned)w1, (unsigned)w2, (unsigned)w3);
                                    need[u] = false;
                                } else {
                                    ok = false;
                                }
                            }
                        if (__all_sync(0xFFFFFFFFu, ok)) break;
                        ++spins;
                        if (__any_sync(0xFFFFFFFFu, abort_flag != 0) || spins > bound) { abort_flag = 1; alive = false; break; }   // the whole warp or nobody
                    }
                    if (!alive) break;
#pragma unroll
                    for (int u = 0; u < kXBatch; ++u) {
                        const int c = cb + u * (kNW * 32) + lane;
                        const bool in = c < total;
                        const int r = in ? (int)mul_shift32((unsigned)c >> 4, it.kb_magic) : 0, k0 = in ? (c - r * cpt) * 8 : 0;
                        if (cb + u * (kNW * 32) < total) convert(v[u], in, r, k0);   // warp-uniform: the conversion shuffles
                    }
                }
                if (!alive) break;
            }
            __syncwarp();
            if (lane == 0) arrive_a(xbar_addr);
            if (!wait_a(xbar_addr, (phases >> 1) & 1u, &abort_flag, spin)) { alive = false; break; }
            phases ^= 2u;
        }
        // B fragment of lane (g, t): column g of column group cg = plane 8 cg + g (token 4 cg + g/2, slice g&1), k bytes t*8..t*8+7 of a chunk.
        // Planes of tokens that do not exist alias the last real plane: an output column depends on its own B column only.
        uint32_t xrow[NG];
        uint32_t xs_tok[NG];
#pragma unroll
        for (int cg = 0; cg < NG; ++cg) {
            xrow[cg] = order_after_wait(smem_u32(xb) + (uint32_t)(min(8 * cg + g, 2 * m - 1) * plane + t * 8));
            xs_tok[cg] = smem_u32(xsc + min(cg * 4 + t, m - 1));
        }
        FlushCtx fc;
        fc.red_addr = smem_u32(red); fc.part_bar_addr = smem_u32(part_bar); fc.done_gen = done_gen; fc.abort_flag = &abort_flag; fc.spin = spin;

        int cur_q = 0;                         // tile part this warp is accumulating
        float acc[NG][2];
#pragma unroll
        for (int cg = 0; cg < NG; ++cg) acc[cg][0] = acc[cg][1] = 0.f;
        bool tail_open = false;
        // hand over the parts this warp has passed (or never touched: zeros) up to part qn
        auto flush_to = [&](int qn) {
            for (; cur_q < qn && alive; ++cur_q) {
                Sums4 sums;
#pragma unroll
                for (int cg = 0; cg < 2; ++cg) { sums.v[2 * cg] = cg < NG ? acc[cg < NG ? cg : 0][0] : 0.f; sums.v[2 * cg + 1] = cg < NG ? acc[cg < NG ? cg : 0][1] : 0.f; }
                if (!flush_part<NG>(fc, seq + (unsigned)cur_q, sums)) alive = false;
#pragma unroll
                for (int cg = 0; cg < NG; ++cg) acc[cg][0] = acc[cg][1] = 0.f;
            }
        };
        // ---- full stages: record st*16 + warp of the walk, one per pass of ONE loop. Its k-block and tile part are carried
        //      along (16 records further each stage: a compare and a subtract), found afresh only at the turn of the walk ----
        {
            unsigned j = (unsigned)warp;
            int kbi = 0, q = 0;
            bool locate = true;
            for (unsigned st = 0; st < n_full && alive; ++st) {
                if (locate) {
                    const unsigned rho = walk_record(wk, j);
                    const int T = (int)mul_shift32(rho, it.kb_magic);
                    kbi = (int)(rho - (unsigned)T * (unsigned)kb);
                    q = walk_part_of_tile(wk, T);
                    locate = false;
                }
                if (cur_q < q) { flush_to(q); if (!alive) break; }
                const uint32_t koff = (uint32_t)kbi * kBlockK, ksc = (uint32_t)kbi * (16 * NG);
                {   // bounded wait for the stage, written out so that the record loop contains no call
                    int polls = 0;
                    while (!try_wait_a(full_addr + bar_off, phase)) {
                        if (++polls >= spin || ((polls & 255) == 0 && abort_flag)) {
                            abort_flag = 1;
                            alive = false;   // give up after this iteration (whatever it computes is never stored)
                            break;
                        }
                    }
                }
                const uint32_t unit = order_after_wait(unit0 + stage_off);
                const uint4 wv0 = lds128(unit), wv1 = lds128(unit + 512);
                const uint32_t coef_addr = unit - lane * 16 + kCodeBytesPerUnit + g * 4;
                const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
                int s1[NG][4], s2[NG][4], s3[NG][4];
                float rec[NG][2];
#pragma unroll
                for (int cg = 0; cg < NG; ++cg) {
                    rec[cg][0] = rec[cg][1] = 0.f;
#pragma unroll
                    for (int r = 0; r < 4; ++r) s1[cg][r] = s2[cg][r] = s3[cg][r] = 0;
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t pa0, pb0, qa0, qb0, fa0, fb0, pa1, pb1, qa1, qb1, fa1, fb1;
                    decode_word<WB, K1>(w0[c], lut_lane, pa0, pb0, qa0, qb0, fa0, fb0);
                    decode_word<WB, K1>(w1[c], lut_lane, pa1, pb1, qa1, qb1, fa1, fb1);
#pragma unroll
                    for (int cg = 0; cg < NG; ++cg) {
                        const uint2 xf = lds64(xrow[cg] + koff + c * 32);
                        mma_s8(s1[cg], pa0, pa1, pb0, pb1, xf.x, xf.y);
                        if constexpr (!K1) {
                            mma_s8(s2[cg], qa0, qa1, qb0, qb1, xf.x, xf.y);
                            mma_s8(s3[cg], fa0, fa1, fb0, fb1, xf.x, xf.y);
                        }
                    }
                    if (((c + 1) % CPG) == 0) group_end<NG, K1>(s1, s2, s3, lds32(coef_addr + (c / CPG) * 64), lds32(coef_addr + (c / CPG) * 64 + 32), rec);
                }
#pragma unroll
                for (int cg = 0; cg < NG; ++cg) {
                    const float sv = lds_f32(xs_tok[cg] + ksc);   // undo the activation scale of this k-block
                    acc[cg][0] = fmaf(sv, rec[cg][0], acc[cg][0]);
                    acc[cg][1] = fmaf(sv, rec[cg][1], acc[cg][1]);
                }
                __syncwarp();
                if (lane == 0) arrive_a(empty_addr + bar_off);
                stage_off += (uint32_t)stage_bytes; bar_off += 8;
                if (++slot == p.n_stages) { slot = 0; phase ^= 1; stage_off = 0; bar_off = 0; }
                // the next record is 16 further in the same linear order, unless the walk turns in between
                const bool before_turn = j < wk.L1;
                j += kStageRecs;
                kbi += kStageRecs;
                while (kbi >= kb) { kbi -= kb; ++q; }   // it has left the tile; a tile narrower than a stage may be skipped altogether
                if (before_turn && j >= wk.L1) locate = true;
            }
        }
        // ---- the last stage of the range, n_tail < 16 records: 16 / n_tail warps share each record, each warp a run of its four
        //      32-wide chunks (the sums are linear in the chunks), so that no warp visits more than one record; the shares come
        //      from a constant table and nothing here divides ----
        if (n_tail && alive) {
            const unsigned share = c_tail_share.v[n_tail][warp];   // record, first and end chunk of this warp
            const unsigned rloc = share & 15u, cb = (share >> 4) & 7u, ce = (share >> 7) & 7u;
            if (rloc < n_tail && cb < ce) {
                const unsigned rho = walk_record(wk, n_full * kStageRecs + rloc);
                const unsigned T = mul_shift32(rho, it.kb_magic);
                const int kbi = (int)(rho - T * (unsigned)kb);
                flush_to(walk_part_of_tile(wk, (int)T));
                if (alive && !wait_a(full_addr + bar_off, phase, &abort_flag, spin)) alive = false;
                if (alive) {
                    tail_open = true;
                    const uint32_t unit = order_after_wait(ring_addr + slot * stage_bytes + rloc * unit_bytes + lane * 16);
                    const uint4 wv0 = lds128(unit), wv1 = lds128(unit + 512);
                    const uint32_t coef_addr = unit - lane * 16 + kCodeBytesPerUnit + g * 4;
                    const uint32_t w0[4] = {wv0.x, wv0.y, wv0.z, wv0.w}, w1[4] = {wv1.x, wv1.y, wv1.z, wv1.w};
                    int s1[NG][4], s2[NG][4], s3[NG][4];
                    float rec[NG][2];
#pragma unroll
                    for (int cg = 0; cg < NG; ++cg) {
                        rec[cg][0] = rec[cg][1] = 0.f;
#pragma unroll
                        for (int r = 0; r < 4; ++r) s1[cg][r] = s2[cg][r] = s3[cg][r] = 0;
                    }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if ((unsigned)c >= cb && (unsigned)c < ce) {   // warp-uniform
                            uint32_t pa0, pb0, qa0, qb0, fa0, fb0, pa1, pb1, qa1, qb1, fa1, fb1;
                            decode_word<WB, K1>(w0[c], lut_lane, pa0, pb0, qa0, qb0, fa0, fb0);
                            decode_word<WB, K1>(w1[c], lut_lane, pa1, pb1, qa1, qb1, fa1, fb1);
#pragma unroll
                            for (int cg = 0; cg < NG; ++cg) {
                                const uint2 xf = lds64(xrow[cg] + (uint32_t)kbi * kBlockK + c * 32);
                                mma_s8(s1[cg], pa0, pa1, pb0, pb1, xf.x, xf.y);
                                if constexpr (!K1) {
                                    mma_s8(s2[cg], qa0, qa1, qb0, qb1, xf.x, xf.y);
                                    mma_s8(s3[cg], fa0, fa1, fb0, fb1, xf.x, xf.y);
                                }
                            }
                            if (((c + 1) % CPG) == 0 || (unsigned)(c + 1) == ce)   // end of a macro-block, or of this warp's share of it
                                group_end<NG, K1>(s1, s2, s3, lds32(coef_addr + (c / CPG) * 64), lds32(coef_addr + (c / CPG) * 64 + 32), rec);
                        }
                    }
#pragma unroll
                    for (int cg = 0; cg < NG; ++cg) {
                        const float sv = lds_f32(xs_tok[cg] + kbi * (16 * NG));
                        acc[cg][0] = fmaf(sv, rec[cg][0], acc[cg][0]);
                        acc[cg][1] = fmaf(sv, rec[cg][1], acc[cg][1]);
                    }
                }
            }
        }
        flush_to(wk.P);   // every part has been handed over
        if (!alive) break;
        if (n_tail) {   // every warp takes part in the tail stage's hand-shake, with or without chunks of its own
            if (!tail_open && !wait_a(full_addr + bar_off, phase, &abort_flag, spin)) { alive = false; break; }
            __syncwarp();
            if (lane == 0) arrive_a(empty_addr + bar_off);
            stage_off += (uint32_t)stage_bytes; bar_off += 8;
            if (++slot == p.n_stages) { slot = 0; phase ^= 1; stage_off = 0; bar_off = 0; }
        }
        seq += (unsigned)wk.P;
    }
    if (lane == 0 && abort_flag) atomicExch(p.status, (int)GOQ_ERR_TIMEOUT);
}

}  // namespace chain
}  // namespace goq

// ---- host side -------------------------------------------------------------------------------------
namespace goq {

static int chain_sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 148;
    return n > 0 ? n : 148;
}

static constexpr size_t kChainSmemMax = 226 * 1024;   // the opt-in limit is 227 KiB per CTA, static shared variables included

static size_t chain_fixed_smem(int ng) {
    return 8192 /* alignment slack */ + (size_t)kLutBytes + (size_t)chain::kTileSlots * chain::kNW * ng * 64 * sizeof(float) +
           (size_t)2 * chain::kMaxKBlocks * 4 * ng * sizeof(float) + (size_t)(2 * chain::kMaxStages + 4 + chain::kTileSlots) * sizeof(uint64_t);
}
static size_t chain_xbuf_bytes(int m, int k_pad) { return ((size_t)2 * m * (k_pad + chain::kXPad) + 127) & ~(size_t)127; }

bool gemv_seq_supported(const Geometry& g, int m) {
    if (!(g.group >= 32 && g.wbits <= 3 && m >= 1 && m <= 8 && g.k_blocks <= chain::kMaxKBlocks)) return false;
    if ((unsigned long long)g.n_units * (unsigned)g.k_blocks >= (1ull << 32)) return false;   // record -> tile by multiply and shift
    if (g.n_tiles > (1 << 21)) return false;   // tile parts per CTA stay far below 2^15 (packed beside the tail stage's chunk range)
    // at least two ring stages beside one activation buffer
    return chain_fixed_smem(m <= 4 ? 1 : 2) + chain_xbuf_bytes(m, g.k_pad) + (size_t)2 * chain::kStageRecs * g.unit_bytes <= kChainSmemMax;
}
// Scratch: [status word and, in its second word, the launch count, 256 B][done: n ints - zero on entry, left zero] then the
// posted partial sums, placed behind the counter area every kernel of the library keeps zero, so that a buffer laid out
// for goq_gemv can serve a one-linear chain. The whole buffer starts zero-filled (goq_workspace_init): a posted value is
// valid when it carries the current launch's tag, and zero is never a tag.
size_t gemv_seq_zeroed_prefix(int n_items) {
    const size_t n = (size_t)(n_items > 0 ? n_items : 0);
    const size_t z = kWsStatusBytes + align_up(n * sizeof(int), 256);
    return z > kWsScratchOff ? z : kWsScratchOff;
}
static size_t chain_parts_bytes(int n_items) {
    return (size_t)(n_items > 0 ? n_items : 0) * (size_t)chain_sm_count() * 2 * chain::kPartWords * sizeof(uint2);
}
size_t gemv_seq_workspace(int n_items) {
    // a single linear feeds nobody: no tagged copies
    const size_t tags = n_items > 1 ? (size_t)n_items * chain::kTagWords * sizeof(uint2) : 0;
    return gemv_seq_zeroed_prefix(n_items) + chain_parts_bytes(n_items) + tags;
}

template <int WB, int CPG, int NG, bool K1>
static cudaError_t launch_chain_cfg(chain::Params& p, size_t x_need, cudaStream_t st) {
    auto kernel = chain::gemv_chain_kernel<WB, CPG, NG, K1>;
    const size_t stage_bytes = (size_t)chain::kStageRecs * p.unit_bytes;
    const size_t fixed = chain_fixed_smem(NG);
    // two activation buffers when they leave room for four ring stages, else one
    p.x_double = (fixed + 2 * x_need + 4 * stage_bytes <= kChainSmemMax) ? 1 : 0;
    p.xbuf_bytes = (int)x_need;
    const size_t xtotal = (size_t)(p.x_double ? 2 : 1) * x_need;
    if (fixed + xtotal + 2 * stage_bytes > kChainSmemMax) return cudaErrorInvalidConfiguration;
    int n_stages = (int)((kChainSmemMax - fixed - xtotal) / stage_bytes);
    if (n_stages > chain::kMaxStages) n_stages = chain::kMaxStages;
    p.n_stages = n_stages;
    const size_t smem = fixed + xtotal + (size_t)n_stages * stage_bytes;
    static SmemAttrCache smem_attr;
    if (cudaError_t e = ensure_dynamic_smem(kernel, smem, smem_attr)) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(chain_sm_count());   // every CTA must be resident: the completion counters are waited on
    cfg.blockDim = dim3(chain::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// How the items of one launch are ordered (host only, no CUDA call). An item flagged `depends` waits for every earlier
// item (counter wait). An unflagged item whose activations lie inside ONE earlier bf16 output reads that output's tagged
// copy and waits word by word; any other overlap with what earlier items read or write falls back to the counter wait;
// an item that overlaps nothing does not wait.
void plan_sequence(const SeqCall* calls, int n, SeqOrder* out) {
    auto overlaps = [](const void* a, size_t an, const void* b, size_t bn) {
        const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
        return a0 < b0 + bn && b0 < a0 + an;
    };
    auto x_bytes = [&](int i) { return (size_t)calls[i].m * calls[i].g.k_in * 2; };
    auto y_bytes = [&](int i) { return (size_t)calls[i].m * calls[i].g.n_out * (calls[i].y_dtype == GOQ_F32 ? 4 : 2); };
    for (int j = 0; j < n; ++j) {
        out[j].kind = kSeqOrderNone; out[j].source = -1; out[j].word_offset = 0;
        if (j == 0) continue;
        if (calls[j].depends) { out[j].kind = kSeqOrderBarrier; continue; }
        int src = -1, hits = 0;
        bool clash = false;
        for (int i = 0; i < j; ++i) {
            if (overlaps(calls[j].x, x_bytes(j), calls[i].y, y_bytes(i))) { src = i; ++hits; }
            if (overlaps(calls[j].y, y_bytes(j), calls[i].y, y_bytes(i)) || overlaps(calls[j].y, y_bytes(j), calls[i].x, x_bytes(i))) clash = true;
        }
        if (!clash && hits == 0) continue;   // independent of everything before it
        out[j].kind = kSeqOrderBarrier;
        if (!clash && hits == 1 && calls[src].y_dtype == GOQ_BF16) {
            const Geometry& gs = calls[src].g;
            const Geometry& gj = calls[j].g;
            const int ms = calls[src].m, mj = calls[j].m;
            const uintptr_t x0 = (uintptr_t)calls[j].x, y0 = (uintptr_t)calls[src].y;
            const size_t stride = (size_t)gs.n_tiles * 8;   // words per token of the copy
            if (x0 >= y0 && (x0 - y0) % 2 == 0 && (size_t)ms * stride <= (size_t)chain::kTagWords && gj.k_in % 8 == 0) {
                const size_t e = (x0 - y0) / 2, tok0 = e / (size_t)gs.n_out, off = e % (size_t)gs.n_out;
                const bool rows_ok = (mj == 1) ? (off + (size_t)gj.k_in <= (size_t)gs.n_out)
                                               : (off == 0 && gj.k_in == gs.n_out && tok0 + (size_t)mj <= (size_t)ms);
                if (off % 8 == 0 && rows_ok && tok0 < (size_t)ms) {
                    out[j].kind = kSeqOrderData;
                    out[j].source = src;
                    out[j].word_offset = (unsigned)(tok0 * stride + off / 2);
                }
            }
        }
    }
}

cudaError_t launch_gemv_seq(const SeqCall* calls, int n, int wbits, int group, int unit_bytes, void* ws, int spin_limit, cudaStream_t st) {
    static thread_local chain::Params p;   // ~17 KB: kept off the stack
    auto* wsb = (uint8_t*)ws;
    p.n_items = n;
    p.unit_bytes = unit_bytes;
    p.spin_limit = spin_limit > 0 ? spin_limit : kSpinLimit;
    p.status = (int*)wsb;
    p.done = (int*)(wsb + 256);
    p.epoch = (unsigned*)(wsb + 4);
    p.parts = (uint2*)(wsb + gemv_seq_zeroed_prefix(n));
    p.tags = (uint2*)(wsb + gemv_seq_zeroed_prefix(n) + chain_parts_bytes(n));
    const int G = chain_sm_count();   // the grid
    p.g_magic = ((1ull << 32) + (unsigned)G - 1) / (unsigned)G;
    int m_max = 1;
    bool k1 = true;
    size_t x_need = 0;
    for (int i = 0; i < n; ++i) {
        chain::Item& it = p.item[i];
        const Geometry& g = calls[i].g;
        it.packed = (const uint8_t*)calls[i].packed;
        it.x = (const uint16_t*)calls[i].x;
        it.y = calls[i].y;
        it.kb_magic = ((1ull << 32) + (unsigned)g.k_blocks - 1) / (unsigned)g.k_blocks;
        it.units = (unsigned)g.n_units;
        it.n_tiles = g.n_tiles;
        it.k_blocks = g.k_blocks;
        it.k_in = g.k_in;
        it.n_out = g.n_out;
        it.m = calls[i].m;
        it.y_dtype = calls[i].y_dtype;
        it.depends = calls[i].depends;
        it.xsrc = -1; it.xoff = 0; it.tag_out = 0;
        it.uq = it.units / (unsigned)G;
        it.ur = it.units % (unsigned)G;
        if (calls[i].m > m_max) m_max = calls[i].m;
        k1 = k1 && g.k1;
        const size_t b = chain_xbuf_bytes(calls[i].m, g.k_pad);
        if (b > x_need) x_need = b;
    }
    // Ordering between the items of one launch, from the address ranges (plan_sequence).
    {
        static thread_local std::vector<SeqOrder> order;
        order.resize((size_t)n);
        plan_sequence(calls, n, order.data());
        for (int j = 0; j < n; ++j) {
            chain::Item& it = p.item[j];
            if (order[(size_t)j].kind == kSeqOrderBarrier) it.depends = 1;
            else it.depends = 0;
            if (order[(size_t)j].kind == kSeqOrderData) {
                it.xsrc = order[(size_t)j].source;
                it.xoff = order[(size_t)j].word_offset;
                p.item[it.xsrc].tag_out = 1;
            }
        }
    }
    const int cpg = group / 32;
#define GOQ_CHAIN(WB_, NG_, K1_)                                                                             \
    (cpg == 1 ? launch_chain_cfg<WB_, 1, NG_, K1_>(p, x_need, st) : cpg == 2 ? launch_chain_cfg<WB_, 2, NG_, K1_>(p, x_need, st) \
                                                                             : launch_chain_cfg<WB_, 4, NG_, K1_>(p, x_need, st))
    if (m_max <= 4) {
        if (k1) return wbits == 3 ? GOQ_CHAIN(3, 1, true) : GOQ_CHAIN(2, 1, true);   // every linear single-basis: the second operand is skipped
        return wbits == 3 ? GOQ_CHAIN(3, 1, false) : GOQ_CHAIN(2, 1, false);
    }
    return wbits == 3 ? GOQ_CHAIN(3, 2, false) : GOQ_CHAIN(2, 2, false);
#undef GOQ_CHAIN
}

}  // namespace goq
