// Calibration statistic kernels: per-channel sum of |x|, per-block mean l1 norm and
// per-token max block l1 norm under an optional permutation.
//
// Phase 1: each CTA walks a contiguous slab of rows with the whole row in shared memory,
// keeps per-channel and per-block partial sums in registers (every thread owns fixed
// columns / blocks), and writes them to its own slice of the workspace.
// Phase 2: one thread per output adds the CTA slices in CTA order.  All additions happen
// in a fixed order, so the results are bit-identical from run to run.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace perq {

constexpr int ST_THREADS = 512;
constexpr int ST_MAX_CHUNKS = 8;    // 8 * 512 threads * 8 channels = 32768 channels

struct StatsParams {
    const uint16_t *x;
    const int32_t *perm;
    long long T;
    int d;
    int log2b;
    int rows_per_cta;
    float *ws_chan;      // [n_cta, d]
    float *ws_block;     // [n_cta, d/b]
    float *token_max;    // [T] or null
};

__device__ __forceinline__ float abs_bf16(uint16_t h) { return __uint_as_float(((uint32_t)h & 0x7fffu) << 16); }

__global__ void __launch_bounds__(ST_THREADS) perq_stats_partial_kernel(StatsParams p)
{
    extern __shared__ __align__(16) unsigned char smem[];
    const int d = p.d, L = p.log2b, nb = d >> L, nchunks = d >> 3;
    uint16_t *raw = (uint16_t *)smem;                         // [d] one row, original order
    uint16_t *sperm = raw + d;                                // [d] permutation (d <= 32768 fits 16 bits)
    float *cs = (float *)(smem + (size_t)d * 4);              // [d/8] per-chunk l1 of the permuted row
    float *red = cs + nchunks;                                // [32]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int i = tid; i < d; i += ST_THREADS) {
        int q = p.perm ? __ldg(p.perm + i) : i;
        sperm[i] = (uint16_t)min(max(q, 0), d - 1);
    }
    float csum[ST_MAX_CHUNKS][8];
    float bsum[ST_MAX_CHUNKS];
#pragma unroll
    for (int k = 0; k < ST_MAX_CHUNKS; ++k) {
        bsum[k] = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) csum[k][e] = 0.0f;
    }
    const long long t0 = (long long)blockIdx.x * p.rows_per_cta;
    const long long t1 = min(p.T, t0 + p.rows_per_cta);
    const bool want_blocks = (p.ws_block != nullptr) || (p.token_max != nullptr);
    __syncthreads();

    for (long long t = t0; t < t1; ++t) {
        const uint4 *src = (const uint4 *)(p.x + (size_t)t * d);
#pragma unroll
        for (int k = 0; k < ST_MAX_CHUNKS; ++k) {
            const int c = tid + k * ST_THREADS;
            if (c < nchunks) {
                const uint4 w = __ldcs(src + c);
                ((uint4 *)raw)[c] = w;
                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    csum[k][2 * e] += __uint_as_float((ww[e] << 16) & 0x7fffffffu);
                    csum[k][2 * e + 1] += __uint_as_float(ww[e] & 0x7fff0000u);
                }
            }
        }
        if (want_blocks) {
            __syncthreads();
#pragma unroll
            for (int k = 0; k < ST_MAX_CHUNKS; ++k) {
                const int c = tid + k * ST_THREADS;
                if (c < nchunks) {
                    const uint4 pi = ((const uint4 *)sperm)[c];
                    const uint32_t pp[4] = {pi.x, pi.y, pi.z, pi.w};
                    float s = 0.0f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        s += abs_bf16(raw[pp[e] & 0xffffu]);
                        s += abs_bf16(raw[pp[e] >> 16]);
                    }
                    cs[c] = s;
                }
            }
            __syncthreads();
            float mx = 0.0f;
            const int cpb = 1 << (L - 3);          // chunks per block
#pragma unroll
            for (int k = 0; k < ST_MAX_CHUNKS; ++k) {
                const int j = tid + k * ST_THREADS;
                if (j < nb) {
                    float s = 0.0f;
                    for (int c = 0; c < cpb; ++c) s += cs[j * cpb + c];
                    bsum[k] += s;
                    mx = fmaxf(mx, s);
                }
            }
            if (p.token_max) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                if (lane == 0) red[warp] = mx;
                __syncthreads();
                if (tid == 0) {
                    float m = red[0];
                    for (int w = 1; w < ST_THREADS / 32; ++w) m = fmaxf(m, red[w]);
                    p.token_max[t] = m;
                }
            }
            __syncthreads();
        } else {
            __syncthreads();
        }
    }

    if (p.ws_chan) {
        float4 *dst = (float4 *)(p.ws_chan + (size_t)blockIdx.x * d);
#pragma unroll
        for (int k = 0; k < ST_MAX_CHUNKS; ++k) {
            const int c = tid + k * ST_THREADS;
            if (c < nchunks) {
                dst[2 * c] = make_float4(csum[k][0], csum[k][1], csum[k][2], csum[k][3]);
                dst[2 * c + 1] = make_float4(csum[k][4], csum[k][5], csum[k][6], csum[k][7]);
            }
        }
    }
    if (p.ws_block) {
#pragma unroll
        for (int k = 0; k < ST_MAX_CHUNKS; ++k) {
            const int j = tid + k * ST_THREADS;
            if (j < nb) p.ws_block[(size_t)blockIdx.x * nb + j] = bsum[k];
        }
    }
}

__global__ void perq_stats_reduce_kernel(const float *ws_chan, const float *ws_block, int n_cta, int d, int nb,
                                         float inv_T, float *chan_abs_sum, float *block_l1_mean)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (chan_abs_sum && i < d) {
        float s = 0.0f;
        for (int c = 0; c < n_cta; ++c) s += ws_chan[(size_t)c * d + i];
        chan_abs_sum[i] = s;
    }
    if (block_l1_mean && i < nb) {
        float s = 0.0f;
        for (int c = 0; c < n_cta; ++c) s += ws_block[(size_t)c * nb + i];
        block_l1_mean[i] = s * inv_T;
    }
}

// perm[0..d) is a permutation?  status: bit0 = out of range, bit1 = duplicate.
__global__ void perq_validate_perm_kernel(const int32_t *perm, int d, int32_t *status)
{
    extern __shared__ uint32_t bitmap[];
    __shared__ int bad;
    for (int w = threadIdx.x; w < (d + 31) / 32; w += blockDim.x) bitmap[w] = 0u;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const int q = perm[i];
        if (q < 0 || q >= d) {
            atomicOr(&bad, 1);
        } else {
            const uint32_t bit = 1u << (q & 31);
            if (atomicOr(&bitmap[q >> 5], bit) & bit) atomicOr(&bad, 2);
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) *status = bad;
}

}  // namespace perq
