// The steps either side of the inner product, on the device:
//   quantize_geo_kernel      Sections 3.2-3.4 (GEO mode): primary PoT code by round-to-nearest, orthogonal residual (Eq. 1),
//                            analytical sign inference and pattern selection per micro-block (Section 3.3, steps 1-3),
//                            decoupled least-squares coefficients (Eq. 2). One warp per macro-block.
//   solve_ref_kernel         Section 3.4, REF mode (Eq. 3): 2 x 2 ridge regression per macro-block on calibration inputs.
//   quantize_act_kernel      Section 3.5: X~ and s_x of Eq. 4 (per-token symmetric 8-bit integers).
// All decisions that end in an integer (a code, a pattern, a sign, a quantised activation) are taken in float64, the
// precision of the reference they are checked against; the work is bound by reading the inputs once.
#include <cuda_fp16.h>
#include "goq_common.cuh"
#include "goq_internal.h"

namespace goq {
namespace quant {

constexpr int kWarps = 8;
constexpr unsigned kFull = 0xFFFFFFFFu;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmax(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

// value of code c on the b-bit asymmetric lattice (Section 3.2): (-1)^sign 2^-e, the smallest positive bin being zero
__device__ __forceinline__ double lattice_value(int c, int wbits) {
    const int emax = (1 << (wbits - 1)) - 1, sg = c >> (wbits - 1), e = c & emax;
    if (!sg && e == emax) return 0.0;
    const double mag = __longlong_as_double((long long)(1023 - e) << 52);   // 2^-e
    return sg ? -mag : mag;
}
// Nearest lattice state in linear distance; exact ties go to the state of smaller magnitude. |v| <= 1. Between two
// neighbouring magnitudes 2^E and 2^(E+1) the midpoint is 1.5 * 2^E, so the choice is read off the exponent field and the
// top of the mantissa of |v|; below the smallest magnitude the neighbours are that state and zero. The positive side has
// no +2^-emax (that bin is the zero): its smallest state is 2^-(emax-1), met by zero at the midpoint 2^-emax.
__device__ __forceinline__ int rtn_code(double v, int wbits) {
    const int emax = (1 << (wbits - 1)) - 1;
    const long long bits = __double_as_longlong(fabs(v));
    const int E = (int)((bits >> 52) & 0x7FF) - 1023;                              // |v| = m 2^E, 1 <= m < 2
    const bool upper = (bits & 0xFFFFFFFFFFFFFll) > (1ll << 51);                   // m > 1.5: the larger neighbour
    const int e = -E - (upper ? 1 : 0);                                            // magnitude 2^-e
    const double a = fabs(v);
    if (v < 0.0) {
        if (!(a > __longlong_as_double((long long)(1023 - emax - 1) << 52))) return emax;   // at or below 2^-(emax+1): zero
        return (1 << (wbits - 1)) | min(e, emax);
    }
    if (!(a > __longlong_as_double((long long)(1023 - emax) << 52))) return emax;           // at or below 2^-emax: zero
    return min(e, emax - 1);
}

// b2 of the four elements a lane holds (elements 4*(lane&1) .. +3 of its micro-block) under record (s, flags):
// for each pair (i, j = i XOR s), i < j, with flag f (1 iff eta = -1):  y_i = -eta x_j,  y_j = eta x_i   (Theorem 1)
__device__ __forceinline__ void exchange4(const double (&x)[4], int s, unsigned flags, int half, double (&y)[4]) {
    double xo[4];   // the neighbouring lane's elements (the other half of the micro-block): fetched by every lane, whatever its pattern
#pragma unroll
    for (int a = 0; a < 4; ++a) xo[a] = __shfl_xor_sync(kFull, x[a], 1);
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        if (s < 4) {   // the partner stays inside the lane's half of the micro-block
            const int b = a ^ s;
            const int i = min(a, b) + 4 * half;                 // lower index of the pair inside the micro-block
            int p = 0;                                          // pairs are numbered in ascending order of their lower index
            for (int q = 0; q < i; ++q) p += (q < (q ^ s));
            const double eta = ((flags >> p) & 1u) ? -1.0 : 1.0;
            const double xb = (b == 0) ? x[0] : (b == 1) ? x[1] : (b == 2) ? x[2] : x[3];
            y[a] = (a < b) ? -eta * xb : eta * xb;
        } else {       // s = 4: the partner is the same position in the other half
            const double eta = ((flags >> a) & 1u) ? -1.0 : 1.0;
            y[a] = half ? eta * xo[a] : -eta * xo[a];
        }
    }
}

// One warp per macro-block of `group` weights (lane l holds elements 4l .. 4l+3; lanes beyond group/4 idle).
__global__ void __launch_bounds__(kWarps * 32)
quantize_geo_kernel(const float* __restrict__ w, uint8_t* __restrict__ codes, uint8_t* __restrict__ meta,
                    uint16_t* __restrict__ coef, int n_out, int k_in, int group, int wbits, int k1) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nj = k_in / group;
    const long long blk = (long long)blockIdx.x * kWarps + warp;
    if (blk >= (long long)n_out * nj) return;
    const int row = (int)(blk / nj), j = (int)(blk % nj);
    const bool on = lane * 4 < group;
    const size_t base = (size_t)row * k_in + (size_t)j * group + lane * 4;
    const int emax = (1 << (wbits - 1)) - 1, half = lane & 1;
    double wv[4] = {0, 0, 0, 0};
    if (on) {
        const float4 f = *reinterpret_cast<const float4*>(w + base);
        wv[0] = f.x; wv[1] = f.y; wv[2] = f.z; wv[3] = f.w;
    }
    // Section 3.2: s_norm = ||w||_inf, v = w / s_norm, b1 = Q(v)
    const double s_norm = warp_max(fmax(fmax(fabs(wv[0]), fabs(wv[1])), fmax(fabs(wv[2]), fabs(wv[3]))));
    int cd[4];
    double x[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) {
        cd[a] = (s_norm == 0.0) ? emax : rtn_code(wv[a] / s_norm, wbits);
        x[a] = on ? lattice_value(cd[a], wbits) : 0.0;
    }
    // Eq. 1: r = w - (<w, b1> / ||b1||^2) b1 (zero-norm bypass: an all-zero block keeps c1 = 0)
    const double nb1 = warp_sum(x[0] * x[0] + x[1] * x[1] + x[2] * x[2] + x[3] * x[3]);
    const double wb1 = warp_sum(wv[0] * x[0] + wv[1] * x[1] + wv[2] * x[2] + wv[3] * x[3]);
    const double c1 = nb1 == 0.0 ? 0.0 : wb1 / nb1;
    double r[4];
#pragma unroll
    for (int a = 0; a < 4; ++a) r[a] = wv[a] - c1 * x[a];

    unsigned rec = 0;
    double c2 = 0.0;
    if (!k1) {
        // Section 3.3, steps 1-2: d = x_i r_j - x_j r_i per pair, eta* = sgn d, A_s = sum |d|, s* = first maximiser
        double d[4][2];     // patterns 1..3: the two pairs inside this half; pattern 4: handled below
        double a_s[4];
#pragma unroll
        for (int s = 1; s <= 3; ++s) {
            int n = 0;
            double sum = 0.0;
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int b = a ^ s;
                if (a < b) { d[s - 1][n] = x[a] * r[b] - x[b] * r[a]; sum += fabs(d[s - 1][n]); ++n; }
            }
            // the micro-block's four pairs: two here, two in the neighbouring lane; added in pair order
            const double other = __shfl_xor_sync(kFull, sum, 1);
            a_s[s - 1] = half ? other + sum : sum + other;
        }
        double d4[4];
        {
            double sum = 0.0;
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const double xo = __shfl_xor_sync(kFull, x[a], 1), ro = __shfl_xor_sync(kFull, r[a], 1);
                d4[a] = half ? (xo * r[a] - x[a] * ro) : (x[a] * ro - xo * r[a]);   // (i, j) = (lower half, upper half)
                sum += fabs(d4[a]);
            }
            a_s[3] = sum;
        }
        int s_star = 0;
#pragma unroll
        for (int s = 1; s < 4; ++s) if (a_s[s] > a_s[s_star]) s_star = s;
        // sign flags of the chosen pattern. The exchange with the neighbouring lane is made by every lane (patterns differ
        // from micro-block to micro-block, and a warp-wide shuffle must not sit in a branch only some lanes take).
        unsigned mine = 0;
#pragma unroll
        for (int s = 0; s < 3; ++s)
            if (s == s_star) mine = (d[s][0] < 0.0 ? 1u : 0u) | (d[s][1] < 0.0 ? 2u : 0u);
        const unsigned other = __shfl_xor_sync(kFull, mine, 1);
        unsigned flags = half ? (other | (mine << 2)) : (mine | (other << 2));
        if (s_star == 3) {
            flags = 0;
#pragma unroll
            for (int a = 0; a < 4; ++a) flags |= (d4[a] < 0.0 ? 1u : 0u) << a;
        }
        rec = (s_norm == 0.0) ? 0u : ((unsigned)s_star | (flags << 2));
        // step 3 and Eq. 2: b2 from the record, c2 = <w, b2> / ||b2||^2
        double y[4];
        exchange4(x, (int)(rec & 3u) + 1, rec >> 2, half, y);
        const double nb2 = warp_sum(y[0] * y[0] + y[1] * y[1] + y[2] * y[2] + y[3] * y[3]);
        const double wb2 = warp_sum(wv[0] * y[0] + wv[1] * y[1] + wv[2] * y[2] + wv[3] * y[3]);
        c2 = nb2 == 0.0 ? 0.0 : wb2 / nb2;
    }
    if (on) {
        *reinterpret_cast<uint32_t*>(codes + base) = (uint32_t)cd[0] | ((uint32_t)cd[1] << 8) | ((uint32_t)cd[2] << 16) | ((uint32_t)cd[3] << 24);
        if (!half) meta[((size_t)row * k_in + (size_t)j * group) / 8 + lane / 2] = (uint8_t)rec;
    }
    if (lane == 0) {
        uint16_t* c = coef + ((size_t)row * nj + j) * 2;
        c[0] = __half_as_ushort(__double2half(c1));
        c[1] = __half_as_ushort(__double2half(c2));
    }
}

// ---- REF mode (Eq. 3) --------------------------------------------------------------------------------------
// c* = (A^T A + lambda I)^-1 A^T Y with A = [X_q b1, X_q b2] (M x 2), Y = X_q w, per row and macro-block.
// CTA = 8 warps = 8 rows of one macro-block column j: the calibration tile X_q[m0 .. m0+31][j g .. (j+1) g) is staged
// in shared memory once per 32 observations and shared by the 8 rows; lane l of a warp owns observation m0 + l and
// runs the three g-long dot products; the five entries of the normal equations accumulate in float64.
constexpr int kRefObs = 32;
__global__ void __launch_bounds__(kWarps * 32)
solve_ref_kernel(const float* __restrict__ w, const uint8_t* __restrict__ codes, const uint8_t* __restrict__ meta,
                 const float* __restrict__ xc, int m, double lambda, uint16_t* __restrict__ coef, double* __restrict__ c_out,
                 int n_out, int k_in, int group, int wbits) {
    __shared__ float xs[kRefObs][kBlockK + 1];
    __shared__ float ws[kWarps][kBlockK], b1s[kWarps][kBlockK], b2s[kWarps][kBlockK];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nj = k_in / group, j = blockIdx.x, row = blockIdx.y * kWarps + warp;
    const bool row_ok = row < n_out;
    // this row's w, b1, b2 of the macro-block (b2 by the recorded exchange, Section 3.3)
    for (int t = lane; t < group / 8; t += 32) {
        double x[8], y[8];
        const size_t o = (size_t)(row_ok ? row : 0) * k_in + (size_t)j * group + t * 8;
        for (int i = 0; i < 8; ++i) x[i] = lattice_value(codes[o + i], wbits);
        const unsigned rec = meta[o / 8];
        const int s = (int)(rec & 3u) + 1;
        int p = 0;
        for (int i = 0; i < 8; ++i) {
            const int q = i ^ s;
            if (i < q) {
                const double eta = ((rec >> (2 + p)) & 1u) ? -1.0 : 1.0;
                y[i] = -eta * x[q];
                y[q] = eta * x[i];
                ++p;
            }
        }
        for (int i = 0; i < 8; ++i) {
            ws[warp][t * 8 + i] = row_ok ? w[o + i] : 0.f;
            b1s[warp][t * 8 + i] = (float)x[i];   // PoT values: exact in float
            b2s[warp][t * 8 + i] = (float)y[i];
        }
    }
    double g11 = 0, g12 = 0, g22 = 0, r1 = 0, r2 = 0;
    for (int m0 = 0; m0 < m; m0 += kRefObs) {
        __syncthreads();
        for (int i = threadIdx.x; i < kRefObs * group; i += kWarps * 32) {
            const int o = i / group, k = i - o * group;
            xs[o][k] = (m0 + o < m) ? xc[(size_t)(m0 + o) * k_in + (size_t)j * group + k] : 0.f;
        }
        __syncthreads();
        double u1 = 0, u2 = 0, t = 0;
        for (int k = 0; k < group; ++k) {
            const double xv = xs[lane][k];
            u1 += xv * b1s[warp][k];
            u2 += xv * b2s[warp][k];
            t += xv * ws[warp][k];
        }
        g11 += u1 * u1; g12 += u1 * u2; g22 += u2 * u2; r1 += u1 * t; r2 += u2 * t;
    }
    g11 = warp_sum(g11); g12 = warp_sum(g12); g22 = warp_sum(g22); r1 = warp_sum(r1); r2 = warp_sum(r2);
    if (lane == 0 && row_ok) {
        const double a = g11 + lambda, d = g22 + lambda, det = a * d - g12 * g12;
        const double c1 = (d * r1 - g12 * r2) / det, c2 = (a * r2 - g12 * r1) / det;
        const size_t o = ((size_t)row * nj + j) * 2;
        coef[o] = __half_as_ushort(__double2half(c1));
        coef[o + 1] = __half_as_ushort(__double2half(c2));
        if (c_out) { c_out[o] = c1; c_out[o + 1] = c2; }
    }
}

// ---- activation quantizer (Section 3.5: X~, s_x) -----------------------------------------------------------
// Per token: s_x = max |x| / q_max (1 for an all-zero token), x~ = clamp(rne(x / s_x), +-q_max), q_max = 2^(bits-1) - 1,
// in int8 containers whatever the width. One CTA per token; when the
// caller already has the token's largest magnitude (the integer GEMM's epilogue can record it) the first pass is skipped.
template <typename T> __device__ __forceinline__ double load_act(const T* p);
template <> __device__ __forceinline__ double load_act<float>(const float* p) { return (double)*p; }
template <> __device__ __forceinline__ double load_act<uint16_t>(const uint16_t* p) { return (double)bf16_to_f32(*p); }

template <typename T>
__global__ void __launch_bounds__(256)
quantize_act_kernel(const T* __restrict__ x, int k, const float* __restrict__ amax_in, int8_t* __restrict__ xq, float* __restrict__ sx,
                    double qmax) {
    __shared__ double red[8];
    __shared__ double s_amax;
    const int tok = blockIdx.x, tid = threadIdx.x;
    const T* row = x + (size_t)tok * k;
    if (amax_in) {
        if (tid == 0) s_amax = (double)amax_in[tok];
    } else {
        double a = 0.0;
        for (int i = tid; i < k; i += 256) a = fmax(a, fabs(load_act<T>(row + i)));
        a = warp_max(a);
        if ((tid & 31) == 0) red[tid >> 5] = a;
        __syncthreads();
        if (tid == 0) {
            double v = red[0];
            for (int i = 1; i < 8; ++i) v = fmax(v, red[i]);
            s_amax = v;
        }
    }
    __syncthreads();
    const double s = s_amax == 0.0 ? 1.0 : s_amax / qmax;
    for (int i = tid; i < k; i += 256) {
        double q = rint(load_act<T>(row + i) / s);   // round half to even
        q = fmin(qmax, fmax(-qmax, q));
        xq[(size_t)tok * k + i] = (int8_t)(int)q;
    }
    if (tid == 0) sx[tok] = (float)s;
}

}  // namespace quant

// ---- launchers -----------------------------------------------------------------------------------------------
cudaError_t launch_quantize_geo(const Geometry& g, const float* w, uint8_t* codes, uint8_t* meta, uint16_t* coef, cudaStream_t st) {
    const long long blocks = (long long)g.n_out * (g.k_in / g.group);
    quant::quantize_geo_kernel<<<(unsigned)((blocks + quant::kWarps - 1) / quant::kWarps), quant::kWarps * 32, 0, st>>>(
        w, codes, meta, coef, g.n_out, g.k_in, g.group, g.wbits, g.k1);
    return cudaGetLastError();
}
cudaError_t launch_solve_ref(const Geometry& g, const float* w, const uint8_t* codes, const uint8_t* meta, const float* x_calib,
                             int m, double lambda, uint16_t* coef, double* c_out, cudaStream_t st) {
    dim3 grid(g.k_in / g.group, (g.n_out + quant::kWarps - 1) / quant::kWarps);
    quant::solve_ref_kernel<<<grid, quant::kWarps * 32, 0, st>>>(w, codes, meta, x_calib, m, lambda, coef, c_out, g.n_out, g.k_in,
                                                                 g.group, g.wbits);
    return cudaGetLastError();
}
cudaError_t launch_quantize_act(const void* x, int x_dtype, int m, int k, int abits, const float* amax, int8_t* xq, float* sx,
                                cudaStream_t st) {
    const double qmax = (double)((1 << (abits - 1)) - 1);
    if (x_dtype == GOQ_F32) quant::quantize_act_kernel<float><<<m, 256, 0, st>>>((const float*)x, k, amax, xq, sx, qmax);
    else quant::quantize_act_kernel<uint16_t><<<m, 256, 0, st>>>((const uint16_t*)x, k, amax, xq, sx, qmax);
    return cudaGetLastError();
}

}  // namespace goq
