// Per-token diagnostics: the quantities the paper plots per token (delta, the block bound, the outlier
// suppression ratio, the 4-bit quantization error), before their normalisation by ||X||_inf.
// One CTA per row at a time; calibration-time work, so the simple structure of the generic kernel:
// row (gathered through the permutation) in shared memory, fp32 butterfly over shared memory, fixed-order
// reductions (deterministic outputs).
#pragma once
#include "perq_generic.cuh"

namespace perq {

struct DiagParams {
    const uint16_t *x;
    const int32_t *perm;     // or null
    float *out;              // [T, 5]
    long long T;
    int d;
    int log2b;
    float inv_sqrt_b;
};

struct DiagSmem {
    size_t xs, ub, red, total;
    __host__ __device__ DiagSmem(int d)
    {
        size_t o = 0;
        xs = o;  o += (size_t)d * 2;
        ub = o;  o += (size_t)d * 4;
        red = o; o += 2 * GEN_WARPS * 4;
        total = o;
    }
};

__device__ __forceinline__ float warp_sum_tree(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max_tree(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
// Sum and maximum over the CTA, the same in every thread, combined in a fixed order.
__device__ __forceinline__ void cta_sum_max(float &s, float &m, float *red, int lane, int warp)
{
    s = warp_sum_tree(s);
    m = warp_max_tree(m);
    __syncthreads();                       // (red may still be read from the previous use)
    if (lane == 0) { red[warp] = s; red[GEN_WARPS + warp] = m; }
    __syncthreads();
    s = 0.0f;
    m = 0.0f;
#pragma unroll
    for (int w = 0; w < GEN_WARPS; ++w) { s += red[w]; m = fmaxf(m, red[GEN_WARPS + w]); }
}

__global__ void __launch_bounds__(GEN_THREADS) perq_diag_kernel(DiagParams p)
{
    extern __shared__ __align__(16) unsigned char dsmem[];
    const int d = p.d, L = p.log2b, b = 1 << L, nb = d >> L, nchunks = d >> 3;
    const DiagSmem lay(d);
    uint16_t *xs = (uint16_t *)(dsmem + lay.xs);
    float *ub = (float *)(dsmem + lay.ub);
    float *red = (float *)(dsmem + lay.red);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (long long row = blockIdx.x; row < p.T; row += gridDim.x) {
        // ---- the row, through the permutation gather if there is one
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
        __syncthreads();

        // ---- ||x||_inf and ||x||_1; the butterfly's first three stages on the way
        float x1 = 0.0f, xinf = 0.0f;
        for (int c = tid; c < nchunks; c += GEN_THREADS) {
            const uint4 w = ((const uint4 *)xs)[c];
            float v[8] = {bf16lo(w.x), bf16hi(w.x), bf16lo(w.y), bf16hi(w.y),
                          bf16lo(w.z), bf16hi(w.z), bf16lo(w.w), bf16hi(w.w)};
#pragma unroll
            for (int e = 0; e < 8; ++e) { x1 += fabsf(v[e]); xinf = fmaxf(xinf, fabsf(v[e])); }
            butterfly_regs<3>(v);
            ((float4 *)ub)[2 * c] = make_float4(v[0], v[1], v[2], v[3]);
            ((float4 *)ub)[2 * c + 1] = make_float4(v[4], v[5], v[6], v[7]);
        }
        cta_sum_max(x1, xinf, red, lane, warp);

        // ---- largest block l1 norm: a warp per block, lanes over its elements
        float bmax = 0.0f, unused = 0.0f;
        for (int j = warp; j < nb; j += GEN_WARPS) {
            float s = 0.0f;
            for (int i = lane; i < b; i += 32) s += fabsf(__uint_as_float((uint32_t)xs[(size_t)j * b + i] << 16));
            bmax = fmaxf(bmax, warp_sum_tree(s));
        }
        cta_sum_max(unused, bmax, red, lane, warp);

        // ---- the remaining butterfly stages
        for (int s = 3; s < L; s += 3) {
            const int R = min(3, L - s);
            if (R == 3) radix_pass<3>(ub, d, s, tid);
            else if (R == 2) radix_pass<2>(ub, d, s, tid);
            else radix_pass<1>(ub, d, s, tid);
            __syncthreads();
        }

        // ---- ||u||_inf, then the error of the symmetric 4-bit quantiser with one step per token
        float umax = 0.0f;
        unused = 0.0f;
        for (int c = tid; c < d / 4; c += GEN_THREADS) {
            const float4 v = ((const float4 *)ub)[c];
            umax = fmaxf(umax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
        }
        cta_sum_max(unused, umax, red, lane, warp);
        float e2 = 0.0f;
        unused = 0.0f;
        if (umax > 0.0f) {
            const float step = umax / 7.0f, inv = 7.0f / umax;
            for (int c = tid; c < d / 4; c += GEN_THREADS) {
                const float4 v = ((const float4 *)ub)[c];
                const float u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float qf = fminf(fmaxf(rintf(u[e] * inv), -8.0f), 7.0f);
                    const float er = fmaf(-step, qf, u[e]);
                    e2 = fmaf(er, er, e2);
                }
            }
        }
        cta_sum_max(e2, unused, red, lane, warp);
        if (tid == 0) {
            float *o = p.out + (size_t)row * 5;
            o[0] = xinf;
            o[1] = x1;
            o[2] = bmax;
            o[3] = umax * p.inv_sqrt_b;
            o[4] = sqrtf(e2) * p.inv_sqrt_b;
        }
        __syncthreads();                   // the next row overwrites the shared row
    }
}

}  // namespace perq
