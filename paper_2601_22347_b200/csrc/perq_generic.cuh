// Generic rotate+quantize kernel: any supported (d, b, fmt, group, perm) combination.
//
// One CTA owns one token row at a time (grid-stride over rows).  The (permuted) bf16 row
// stays in shared memory for the whole row so that single output coordinates can be
// re-evaluated exactly; the butterfly runs in fp32 through registers and shared memory.
//
// Numerical contract (what makes scales and codes reproducible against exact arithmetic):
//   * the fp32 butterfly result u32 carries a small rounding error, bounded here by
//     ERR_K * log2(b) * 2^-24 * (largest |u32| of the Hadamard block);
//   * every quantity that decides an output bit is therefore re-derived in fp64 from the
//     bf16 inputs whenever the fp32 value is within that bound of a decision boundary:
//       - the absmax of an INT4 scale range (always: the stored scale must be exact),
//       - the absmax of an MX group when it is close to a power-of-two boundary,
//       - any element whose scaled value is close to a rounding tie.
//     An fp64 sum of <= 32768 bf16 terms is exact unless their exponents span more than
//     ~30 binades, so these re-derived values are the true ones.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace perq {

constexpr int GEN_THREADS = 256;
constexpr int GEN_WARPS = GEN_THREADS / 32;
constexpr int TIE_CAP = 1024;
constexpr float ERR_K = 8.0f;                 // safety factor on the fp32 butterfly error model
constexpr float TWO_M24 = 5.9604644775390625e-8f;
constexpr int GEN_MAX_BASE = 76;              // largest base matrix of a non-power-of-2 rotation (3 words of sign bits)

struct GenParams {
    const uint16_t *x;
    const int32_t *perm;
    long long T;
    int d;
    int log2b;
    int fmt;          // 0 INT4, 1 MXFP4, 2 F32 debug, 3 E2M1 with a per-token fp32 scale, 4 asymmetric INT4 per token
    int g;            // effective scale-range length (d for per-token, 32 for MX)
    void *out_codes;
    void *out_scales;
    float inv_sqrt_b;
    double sqrt_b;
    // Full-vector rotation of a row whose length is not a power of two: d = 2^log2b * base_n, H_d =
    // H_{2^log2b} (x) H_{base_n} (rotations of base_n ADJACENT inputs, then butterflies over strides of base_n).
    // base_n = 0: Sylvester blocks of 2^log2b.  hrow[r] holds row r of the +-1 base matrix, bit c set = -1.
    int base_n;
    uint32_t hrow[GEN_MAX_BASE][3];
};

// Base matrix in shared memory for the tensor-core stage: NP output columns (a multiple of 8), rows of KP + 8
// bf16 (KP = inputs padded to a multiple of 16; the 8 extra keep the fragment loads off one bank).
__host__ __device__ constexpr int gen_base_np(int n0) { return (n0 + 7) / 8 * 8; }
__host__ __device__ constexpr int gen_base_ldk(int n0) { return (n0 + 15) / 16 * 16 + 8; }

// Shared-memory carve-up, computed identically on host (for the launch) and device.
struct GenSmem {
    size_t xs, ub, ub2, bmat, codes, r_max, r_thr, r_mul, r_aux, r_E, b_max, ties, asym, total;
    __host__ __device__ GenSmem(int d, int g, int log2b, int base_n)
    {
        const size_t nr = (size_t)(d / g), nb = base_n ? 1 : (size_t)(d >> log2b);
        size_t o = 0;
        xs = o;    o += (size_t)d * 2;
        ub = o;    o += (size_t)d * 4;
        ub2 = o;   o += base_n ? (size_t)d * 4 : 0;      // transposed copy for the butterflies over strides of base_n
        bmat = o;  o += base_n ? (size_t)gen_base_np(base_n) * gen_base_ldk(base_n) * 2 : 0;   // base matrix, bf16, [n][k]
        codes = o; o += (size_t)d / 2;
        o = (o + 15) & ~(size_t)15;
        r_aux = o; o += nr * 8;
        r_max = o; o += nr * 4;
        r_thr = o; o += nr * 4;
        r_mul = o; o += nr * 4;
        r_E = o;   o += nr * 4;
        b_max = o; o += nb * 4;
        ties = o;  o += (size_t)TIE_CAP * 4 + 16;
        o = (o + 7) & ~(size_t)7;   // 64-bit atomics below
        asym = o;  o += 4 * 8;      // asymmetric INT4: exact max, exact min (order-preserving codes), step, zero point
        total = o;
    }
};

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ double bf16_to_f64(uint16_t h) { return (double)__uint_as_float((uint32_t)h << 16); }

// Order-preserving unsigned codes of signed floating-point values (for atomicMax / atomicMin).
__device__ __forceinline__ uint32_t ord32(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float unord32(uint32_t c)
{
    return __uint_as_float((c & 0x80000000u) ? (c & 0x7fffffffu) : ~c);
}
__device__ __forceinline__ unsigned long long ord64(double f)
{
    const unsigned long long u = (unsigned long long)__double_as_longlong(f);
    return (u >> 63) ? ~u : (u | 0x8000000000000000ull);
}
__device__ __forceinline__ double unord64(unsigned long long c)
{
    return __longlong_as_double((long long)((c >> 63) ? (c & 0x7fffffffffffffffull) : ~c));
}

// In-register butterfly over the low `R` index bits of v[0..2^R).
template <int R>
__device__ __forceinline__ void butterfly_regs(float (&v)[1 << R])
{
#pragma unroll
    for (int t = 0; t < R; ++t) {
#pragma unroll
        for (int e = 0; e < (1 << R); ++e) {
            if ((e & (1 << t)) == 0) {
                const float a = v[e], c = v[e | (1 << t)];
                v[e] = a + c;
                v[e | (1 << t)] = a - c;
            }
        }
    }
}

// One pass of R butterfly stages on index bits [s, s+R) of the fp32 row in shared memory.
template <int R>
__device__ __forceinline__ void radix_pass(float *ub, int d, int s, int tid)
{
    const int nsets = d >> R;
    for (int q = tid; q < nsets; q += GEN_THREADS) {
        const int base = ((q >> s) << (s + R)) | (q & ((1 << s) - 1));
        float v[1 << R];
#pragma unroll
        for (int e = 0; e < (1 << R); ++e) v[e] = ub[base + (e << s)];
        butterfly_regs<R>(v);
#pragma unroll
        for (int e = 0; e < (1 << R); ++e) ub[base + (e << s)] = v[e];
    }
}

// d += a * b, one m16n8k16 tile: bf16 operands (a: 16 x 16 row-major fragment, b: 16 x 8), fp32 accumulators.
__device__ __forceinline__ void gen_mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Exact value of one unnormalised output coordinate, sum_k H[k][ii] x'_k over the coordinate's block,
// evaluated by a whole warp in fp64.  Sylvester blocks: H[k][ii] = (-1)^{popcount(ii & k)}.  With a base
// matrix of order n0 (one block: the row): H[k][ii] = (-1)^{popcount(k / n0 & ii / n0)} * base[ii % n0][k % n0].
__device__ __forceinline__ double exact_coord_warp(const GenParams &p, const uint16_t *xs, int blk_base, int b, int ii, int lane)
{
    double acc = 0.0;
    if (p.base_n == 0) {
        for (int k = lane; k < b; k += 32) {
            const double v = bf16_to_f64(xs[blk_base + k]);
            acc += (__popc(ii & k) & 1) ? -v : v;
        }
    } else {
        const int n0 = p.base_n, i2 = ii / n0, r = ii - i2 * n0;
        const uint32_t h0 = p.hrow[r][0], h1 = p.hrow[r][1], h2 = p.hrow[r][2];
        int k2 = lane / n0, c = lane - k2 * n0;
        for (int k = lane; k < b; k += 32) {
            const double v = bf16_to_f64(xs[k]);
            const uint32_t hw = c < 32 ? h0 : (c < 64 ? h1 : h2);
            const uint32_t neg = (__popc(i2 & k2) ^ (hw >> (c & 31))) & 1u;
            acc += neg ? -v : v;
            c += 32;
            while (c >= n0) { c -= n0; ++k2; }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

__device__ __forceinline__ double exact_coord_thread(const GenParams &p, const uint16_t *xs, int blk_base, int b, int ii)
{
    double acc = 0.0;
    if (p.base_n == 0) {
        for (int k = 0; k < b; ++k) {
            const double v = bf16_to_f64(xs[blk_base + k]);
            acc += (__popc(ii & k) & 1) ? -v : v;
        }
    } else {
        const int n0 = p.base_n, i2 = ii / n0, r = ii - i2 * n0;
        int k2 = 0, c = 0;
        for (int k = 0; k < b; ++k) {
            const double v = bf16_to_f64(xs[k]);
            const uint32_t neg = (__popc(i2 & k2) ^ (p.hrow[r][c >> 5] >> (c & 31))) & 1u;
            acc += neg ? -v : v;
            if (++c == n0) { c = 0; ++k2; }
        }
    }
    return acc;
}

// E2M1 code (sign << 3 | magnitude index) of an exactly known scaled value; ties to the even index.
__device__ __forceinline__ uint32_t e2m1_code_exact(double v, bool negative)
{
    const double m = fabs(v);
    uint32_t k;
    if (m <= 0.25) k = 0;
    else if (m < 0.75) k = 1;
    else if (m <= 1.25) k = 2;
    else if (m < 1.75) k = 3;
    else if (m <= 2.5) k = 4;
    else if (m < 3.5) k = 5;
    else if (m <= 5.0) k = 6;
    else k = 7;
    return (negative ? 8u : 0u) | k;
}

// Distance from |v| to the nearest E2M1 rounding midpoint {.25,.75,1.25,1.75,2.5,3.5,5}.
__device__ __forceinline__ float e2m1_tie_distance(float m)
{
    if (m < 2.0f) {
        const float t = 2.0f * m - 0.5f;             // midpoints at t = 0, 1, 2, 3
        const float r = fminf(rintf(t), 3.0f);
        return 0.5f * fabsf(t - r);
    }
    if (m < 4.0f) {
        const float t = m - 0.5f;                    // midpoints at t = 2, 3
        const float r = fminf(fmaxf(rintf(t), 2.0f), 3.0f);
        return fabsf(t - r);
    }
    return fabsf(m - 5.0f);
}

// Two fp32 values -> one byte of two E2M1 codes (first operand in the low nibble), RNE, saturating.
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi)
{
    uint16_t r;
    asm("{ .reg .b8 t; cvt.rn.satfinite.e2m1x2.f32 t, %1, %2; cvt.u16.u8 %0, t; }" : "=h"(r) : "f"(hi), "f"(lo));
    return (uint32_t)r;
}

// Exact code of element i (row-relative index) from its exact unnormalised value u.
__device__ __forceinline__ uint32_t exact_code(const GenParams &p, double u, double s64, int E, double z64 = 0.0)
{
    const double y = u / p.sqrt_b;
    if (p.fmt == 4) {
        if (s64 == 0.0) return 0u;
        const double q = fmin(fmax(rint(y / s64) - z64, 0.0), 15.0);
        return (uint32_t)((int)q);
    }
    if (p.fmt == 0) {
        if (s64 == 0.0) return 0u;
        double q = rint(y / s64);
        q = fmin(fmax(q, -8.0), 7.0);
        return (uint32_t)((int)q) & 0xFu;
    }
    if (p.fmt == 3) return e2m1_code_exact((s64 == 0.0) ? 0.0 : y / s64, signbit(y));
    return e2m1_code_exact(scalbn(y, -E), signbit(y));
}

__global__ void __launch_bounds__(GEN_THREADS) perq_generic_kernel(GenParams p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int d = p.d, L = p.log2b, n0 = p.base_n, b = n0 ? d : 1 << L, g = p.g;
    const int LB = n0 ? 30 : L;               // shift from an element index to its Hadamard block (one block with a base matrix)
    const int bmask = n0 ? 0x3fffffff : b - 1;
    const int nr = d / g, nb = n0 ? 1 : d >> L, nchunks = d >> 3;
    const GenSmem lay(d, g, L, n0);
    uint16_t *xs = (uint16_t *)(smem + lay.xs);
    float *ub = (float *)(smem + lay.ub);
    uint32_t *codes = (uint32_t *)(smem + lay.codes);
    unsigned long long *r_aux = (unsigned long long *)(smem + lay.r_aux);  // exact amax bits, then s64 bits
    uint32_t *r_max = (uint32_t *)(smem + lay.r_max);
    float *r_thr = (float *)(smem + lay.r_thr);
    float *r_mul = (float *)(smem + lay.r_mul);
    int *r_E = (int *)(smem + lay.r_E);
    uint32_t *b_max = (uint32_t *)(smem + lay.b_max);
    int *tie_list = (int *)(smem + lay.ties);
    int *tie_count = tie_list + TIE_CAP;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // |u32 - u| <= err_rel * (block max |u32|); a base matrix adds a sequential sum of n0 terms to the L stages
    const float err_rel = ERR_K * (float)(n0 ? L + n0 - 1 : L) * TWO_M24;

    if (n0) {   // base matrix as bf16 +-1 (0 in the padding), [output n][input k]: B[k][n] = base[n][k] (symmetric)
        uint16_t *bmw = (uint16_t *)(smem + lay.bmat);
        const int NP = gen_base_np(n0), LDK = gen_base_ldk(n0);
        for (int e = tid; e < NP * LDK; e += GEN_THREADS) {
            const int n = e / LDK, k = e - n * LDK;
            uint16_t v = 0;
            if (n < n0 && k < n0) v = ((p.hrow[n][k >> 5] >> (k & 31)) & 1u) ? 0xBF80 : 0x3F80;
            bmw[e] = v;
        }
        __syncthreads();
    }
    for (long long row = blockIdx.x; row < p.T; row += gridDim.x) {
        // ---- A. row -> shared memory, through the permutation gather if there is one
        const uint4 *src = (const uint4 *)(p.x + (size_t)row * d);
        if (p.perm == nullptr) {
            for (int c = tid; c < nchunks; c += GEN_THREADS) ((uint4 *)xs)[c] = __ldcs(src + c);
        } else {
            uint16_t *raw = (uint16_t *)ub;
            for (int c = tid; c < nchunks; c += GEN_THREADS) ((uint4 *)raw)[c] = __ldcs(src + c);
            __syncthreads();
            for (int i = tid; i < d; i += GEN_THREADS) {
                int q = __ldg(p.perm + i);
                q = min(max(q, 0), d - 1);
                xs[i] = raw[q];
            }
        }
        for (int r = tid; r < nr; r += GEN_THREADS) { r_max[r] = 0u; r_aux[r] = 0ull; }
        for (int j = tid; j < nb; j += GEN_THREADS) b_max[j] = 0u;
        if (tid == 0) *tie_count = 0;
        __syncthreads();

        // ---- B. butterfly: index bits 0..2 in registers, the rest in passes over shared memory
        if (n0 == 0) {
            for (int c = tid; c < nchunks; c += GEN_THREADS) {
                const uint4 w = ((const uint4 *)xs)[c];
                float v[8] = {bf16lo(w.x), bf16hi(w.x), bf16lo(w.y), bf16hi(w.y),
                              bf16lo(w.z), bf16hi(w.z), bf16lo(w.w), bf16hi(w.w)};
                butterfly_regs<3>(v);
                ((float4 *)ub)[2 * c] = make_float4(v[0], v[1], v[2], v[3]);
                ((float4 *)ub)[2 * c + 1] = make_float4(v[4], v[5], v[6], v[7]);
            }
            __syncthreads();
            for (int s = 3; s < L; s += 3) {
                const int R = min(3, L - s);
                if (R == 3) radix_pass<3>(ub, d, s, tid);
                else if (R == 2) radix_pass<2>(ub, d, s, tid);
                else radix_pass<1>(ub, d, s, tid);
                __syncthreads();
            }
        } else {
            // ---- B'. base matrix: the groups of n0 adjacent inputs times the +-1 base matrix -- a dense contraction,
            // on the tensor cores: m16n8k16 tiles over 16 groups x 8 outputs, bf16 operands (products exact), fp32
            // accumulators.  A warp takes 16 groups at a time, keeps their input fragments (the bf16 row in shared
            // memory read as 32-bit pairs, zero beyond n0) and walks the output tiles; results are stored
            // transposed (output r of all groups contiguous).  Then the L butterfly stages over the group index,
            // and the transpose back.
            float *ub2 = (float *)(smem + lay.ub2);
            const uint16_t *bm = (const uint16_t *)(smem + lay.bmat);
            const int K = 1 << L;
            const int KT = (n0 + 15) >> 4, NT = (n0 + 7) >> 3, LDK = gen_base_ldk(n0);
            const int fg = lane >> 2, fq = lane & 3;
            for (int mt = warp; mt * 16 < K; mt += GEN_WARPS) {
                uint32_t afr[(GEN_MAX_BASE + 15) / 16][4];
#pragma unroll
                for (int kt = 0; kt < (GEN_MAX_BASE + 15) / 16; ++kt) {
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const int grp = mt * 16 + fg + 8 * (h & 1), kk = kt * 16 + 2 * fq + 8 * (h >> 1);
                        afr[kt][h] = (kt < KT && grp < K && kk < n0) ? *(const uint32_t *)(xs + grp * n0 + kk) : 0u;
                    }
                }
                for (int nt = 0; nt < NT; ++nt) {
                    float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                    const uint16_t *brow = bm + (nt * 8 + fg) * LDK + 2 * fq;
#pragma unroll
                    for (int kt = 0; kt < (GEN_MAX_BASE + 15) / 16; ++kt) {
                        if (kt < KT) gen_mma_bf16(c, afr[kt], *(const uint32_t *)(brow + kt * 16), *(const uint32_t *)(brow + kt * 16 + 8));
                    }
#pragma unroll
                    for (int h = 0; h < 4; ++h) {
                        const int grp = mt * 16 + fg + 8 * (h >> 1), r = nt * 8 + 2 * fq + (h & 1);
                        if (grp < K && r < n0) ub2[r * K + grp] = c[h];
                    }
                }
            }
            __syncthreads();
            for (int s = 0; s < L; s += 3) {
                const int R = min(3, L - s);
                if (R == 3) radix_pass<3>(ub2, d, s, tid);
                else if (R == 2) radix_pass<2>(ub2, d, s, tid);
                else radix_pass<1>(ub2, d, s, tid);
                __syncthreads();
            }
            for (int j = tid; j < d; j += GEN_THREADS) ub[(j & (K - 1)) * n0 + (j >> L)] = ub2[j];
            __syncthreads();
        }

        if (p.fmt == 2) {   // debug: the rotated row itself
            float4 *dst = (float4 *)((float *)p.out_codes + (size_t)row * d);
            const float k = p.inv_sqrt_b;
            for (int c = tid; c < d / 4; c += GEN_THREADS) {
                float4 v = ((const float4 *)ub)[c];
                dst[c] = make_float4(v.x * k, v.y * k, v.z * k, v.w * k);
            }
            __syncthreads();
            continue;
        }

        unsigned long long *asym = (unsigned long long *)(smem + lay.asym);
        if (p.fmt == 4) {
            // ---- C'-E'. asymmetric INT4 (one range: the row): signed fp32 extremes, their exact values, step and zero point
            uint32_t *cmin = (uint32_t *)r_thr;     // (the threshold slot is free in this mode)
            if (tid == 0) { r_max[0] = 0u; cmin[0] = 0xffffffffu; asym[0] = 0ull; asym[1] = ~0ull; }
            __syncthreads();
            for (int c = tid; c < nchunks; c += GEN_THREADS) {
                const float4 a = ((const float4 *)ub)[2 * c], e = ((const float4 *)ub)[2 * c + 1];
                const float hi = fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(e.x, e.y), fmaxf(e.z, e.w)));
                const float lo = fminf(fminf(fminf(a.x, a.y), fminf(a.z, a.w)), fminf(fminf(e.x, e.y), fminf(e.z, e.w)));
                atomicMax(&r_max[0], ord32(hi));
                atomicMin(&cmin[0], ord32(lo));
                atomicMax(&b_max[(c * 8) >> LB], __float_as_uint(fmaxf(fabsf(hi), fabsf(lo))));
            }
            __syncthreads();
            const float mx32 = unord32(r_max[0]), mn32 = unord32(cmin[0]);
            const float err_row = err_rel * fmaxf(fabsf(mx32), fabsf(mn32));     // every block maximum is below this
            const float thr_hi = mx32 - 2.0f * err_row, thr_lo = mn32 + 2.0f * err_row;
            for (int i0 = warp * 32; i0 < d; i0 += GEN_THREADS) {
                const float ui = ub[i0 + lane];
                unsigned m = __ballot_sync(0xffffffffu, ui >= thr_hi || ui <= thr_lo);
                while (m) {
                    const int ic = i0 + (__ffs(m) - 1);
                    m &= m - 1;
                    const double u = exact_coord_warp(p, xs, (ic >> LB) << LB, b, ic & bmask, lane);
                    if (lane == 0) { atomicMax(&asym[0], ord64(u)); atomicMin(&asym[1], ord64(u)); }
                }
            }
            __syncthreads();
            if (tid == 0) {
                const double mxy = unord64(asym[0]) / p.sqrt_b, mny = unord64(asym[1]) / p.sqrt_b;
                const double s = (mxy - mny) / 15.0;
                const double z = (s == 0.0) ? 0.0 : rint(mny / s);
                ((float *)p.out_scales)[(size_t)row * 2] = (float)s;
                ((float *)p.out_scales)[(size_t)row * 2 + 1] = (float)z;
                r_mul[0] = (s == 0.0) ? 0.0f : fminf((float)(1.0 / (s * p.sqrt_b)), 3.0e38f);
                asym[2] = (unsigned long long)__double_as_longlong(s);
                asym[3] = (unsigned long long)__double_as_longlong(z);
            }
            __syncthreads();
        }
        // ---- C. fp32 absmax per scale range and per Hadamard block
        for (int c = tid; p.fmt != 4 && c < nchunks; c += GEN_THREADS) {
            const float4 a = ((const float4 *)ub)[2 * c], e = ((const float4 *)ub)[2 * c + 1];
            const float m = fmaxf(fmaxf(fmaxf(fabsf(a.x), fabsf(a.y)), fmaxf(fabsf(a.z), fabsf(a.w))),
                                  fmaxf(fmaxf(fabsf(e.x), fabsf(e.y)), fmaxf(fabsf(e.z), fabsf(e.w))));
            atomicMax(&r_max[(c * 8) / g], __float_as_uint(m));
            atomicMax(&b_max[(c * 8) >> LB], __float_as_uint(m));
        }
        __syncthreads();

        // ---- D. which ranges need their absmax re-derived exactly, and from which elements
        for (int r = tid; p.fmt != 4 && r < nr; r += GEN_THREADS) {
            const float rm = __uint_as_float(r_max[r]);
            const float bm = (g >= b) ? rm : __uint_as_float(b_max[(r * g) >> LB]);
            const float err = err_rel * bm;
            bool need = rm > 0.0f;
            if (need && p.fmt == 1) {
                // MX only needs floor(log2(amax / sqrt(b))): exact only near a power of two
                int e;
                const double mant = frexp((double)rm / p.sqrt_b, &e);       // [0.5, 1)
                const double rho = (double)err / (double)rm + 2.4e-7;
                need = (mant * (1.0 + rho) >= 1.0) || (mant * (1.0 - rho) < 0.5);
            }
            r_thr[r] = need ? fmaxf(rm - 2.0f * err, 0.0f) : __int_as_float(0x7f800000);
        }
        __syncthreads();
        {
            const int parts = (g + 255) >> 8;
            const int units = nr * parts;
            for (int unit = warp; p.fmt != 4 && unit < units; unit += GEN_WARPS) {
                const int r = unit / parts, part = unit - r * parts;
                const float thr = r_thr[r];
                if (!(thr < __int_as_float(0x7f800000))) continue;
                const int start = r * g + (part << 8);
                const int end = min(r * g + g, start + 256);
                for (int i0 = start; i0 < end; i0 += 32) {
                    const int i = i0 + lane;
                    const bool cand = (i < end) && (fabsf(ub[i]) >= thr);
                    unsigned m = __ballot_sync(0xffffffffu, cand);
                    while (m) {
                        const int ic = i0 + (__ffs(m) - 1);
                        m &= m - 1;
                        const double u = exact_coord_warp(p, xs, (ic >> LB) << LB, b, ic & bmask, lane);
                        if (lane == 0) atomicMax(&r_aux[r], (unsigned long long)__double_as_longlong(fabs(u)));
                    }
                }
            }
        }
        __syncthreads();

        // ---- E. scales
        for (int r = tid; p.fmt != 4 && r < nr; r += GEN_THREADS) {
            const float rm = __uint_as_float(r_max[r]);
            const bool exact = r_thr[r] < __int_as_float(0x7f800000);
            const double au = exact ? __longlong_as_double((long long)r_aux[r]) : (double)rm;
            const double yd = au / p.sqrt_b;
            if (p.fmt != 1) {
                const double s = yd / 7.0;
                ((float *)p.out_scales)[(size_t)row * nr + r] = (au == 0.0) ? 0.0f : (float)s;
                r_mul[r] = (au == 0.0) ? 0.0f : fminf((float)(7.0 / au), 3.0e38f);
                r_aux[r] = (unsigned long long)__double_as_longlong(s);
            } else {
                int E = -127;
                if (au != 0.0) {
                    int e;
                    (void)frexp(yd, &e);
                    E = min(max(e - 3, -127), 127);
                }
                ((uint8_t *)p.out_scales)[(size_t)row * nr + r] = (au == 0.0) ? 0 : (uint8_t)(E + 127);
                r_mul[r] = (au == 0.0) ? 0.0f : (float)(scalbn(1.0, -E) / p.sqrt_b);
                r_E[r] = E;
            }
        }
        __syncthreads();

        // ---- F. quantise in fp32, flagging elements too close to a rounding tie
        for (int c = tid; c < nchunks; c += GEN_THREADS) {
            const int i0 = c * 8, r = i0 / g;
            const float mul = r_mul[r];
            const float tau_abs = err_rel * __uint_as_float(b_max[i0 >> LB]) * mul;
            const float4 a = ((const float4 *)ub)[2 * c], e = ((const float4 *)ub)[2 * c + 1];
            const float u[8] = {a.x, a.y, a.z, a.w, e.x, e.y, e.z, e.w};
            uint32_t word = 0u, flags = 0u;
            if (p.fmt == 4) {
                const float zf = (float)__longlong_as_double((long long)asym[3]);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float v = u[k] * mul;
                    const float rq = rintf(v);
                    if (fabsf(v - rq) > 0.5f - (tau_abs + (fabsf(v) + 8.0f) * 5.0e-7f)) flags |= 1u << k;
                    word |= (uint32_t)((int)fminf(fmaxf(rq - zf, 0.0f), 15.0f)) << (4 * k);
                }
            } else if (p.fmt == 0) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    const float v = u[k] * mul;
                    const float q = fminf(fmaxf(rintf(v), -8.0f), 7.0f);
                    if (fabsf(v - q) > 0.5f - (tau_abs + 4.0e-6f)) flags |= 1u << k;
                    word |= ((uint32_t)((int)q) & 0xFu) << (4 * k);
                }
            } else {
#pragma unroll
                for (int k = 0; k < 8; k += 2) {
                    const float v0 = fmaf(u[k], mul, 0.0f), v1 = fmaf(u[k + 1], mul, 0.0f);
                    word |= cvt_e2m1x2(v0, v1) << (4 * k);
                    // (a value within the error bound of zero may have the wrong sign bit: flagged too)
                    if (fminf(e2m1_tie_distance(fabsf(v0)), fabsf(v0)) < tau_abs + fabsf(v0) * 1.0e-6f) flags |= 1u << k;
                    if (fminf(e2m1_tie_distance(fabsf(v1)), fabsf(v1)) < tau_abs + fabsf(v1) * 1.0e-6f) flags |= 2u << k;
                }
            }
            while (flags) {
                const int k = __ffs(flags) - 1;
                flags &= flags - 1;
                const int pos = atomicAdd(tie_count, 1);
                if (pos < TIE_CAP) {
                    tie_list[pos] = i0 + k;
                } else {   // list full: resolve here, single-threaded
                    const int i = i0 + k;
                    const double ue = exact_coord_thread(p, xs, (i >> LB) << LB, b, i & bmask);
                    const uint32_t code = (p.fmt == 4)
                        ? exact_code(p, ue, __longlong_as_double((long long)asym[2]), 0, __longlong_as_double((long long)asym[3]))
                        : exact_code(p, ue, __longlong_as_double((long long)r_aux[r]), r_E[r]);
                    word = (word & ~(0xFu << (4 * k))) | (code << (4 * k));
                }
            }
            codes[c] = word;
        }
        __syncthreads();

        // ---- G. resolve the flagged elements exactly
        {
            const int n = min(*tie_count, TIE_CAP);
            for (int t = warp; t < n; t += GEN_WARPS) {
                const int i = tie_list[t], r = i / g;
                const double ue = exact_coord_warp(p, xs, (i >> LB) << LB, b, i & bmask, lane);
                if (lane == 0) {
                    const uint32_t code = (p.fmt == 4)
                        ? exact_code(p, ue, __longlong_as_double((long long)asym[2]), 0, __longlong_as_double((long long)asym[3]))
                        : exact_code(p, ue, __longlong_as_double((long long)r_aux[r]), r_E[r]);
                    const int sh = 4 * (i & 7);
                    atomicAnd(&codes[i >> 3], ~(0xFu << sh));
                    atomicOr(&codes[i >> 3], code << sh);
                }
            }
        }
        __syncthreads();

        // ---- H. packed codes out
        {
            uint4 *dst = (uint4 *)((uint8_t *)p.out_codes + (size_t)row * (d / 2));
            for (int c = tid; c < d / 32; c += GEN_THREADS) __stcs(dst + c, ((const uint4 *)codes)[c]);
        }
        __syncthreads();
    }
}

}  // namespace perq
