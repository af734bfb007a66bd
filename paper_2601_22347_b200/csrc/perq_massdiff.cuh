// Algorithm 1 (MassDiff) on the device, so that a calibration pass (statistic -> permutation -> permuted
// rotate+quantize) never leaves the GPU.  Same rules as the host function: channels in descending mass
// (equal masses: lower channel first), each to the open block with the smallest running sum (equal sums:
// lower block first), running sums in double, perm = the blocks concatenated.
//
// Two kernels: ranks by counting (every CTA ranks 256 channels against all d: d^2 comparisons spread over the
// grid), then the greedy itself, which is sequential in the channels: one warp scans the open blocks for the
// minimum (lanes over blocks, integer warp reductions), d times.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace perq {

constexpr int MD_THREADS = 256;
constexpr int MD_TILE = 1024;
constexpr int MD_MAX_BLOCKS = 4096;      // running sums and fill counts live in shared memory

// order[r] = the channel of rank r (rank = number of channels that come before it)
__global__ void __launch_bounds__(MD_THREADS) perq_massdiff_rank_kernel(const float *a, int d, int32_t *order)
{
    __shared__ float tile[MD_TILE];
    const int i = blockIdx.x * MD_THREADS + threadIdx.x;
    const float ai = (i < d) ? a[i] : 0.0f;
    int rank = 0;
    for (int k0 = 0; k0 < d; k0 += MD_TILE) {
        __syncthreads();
        for (int k = threadIdx.x; k < MD_TILE; k += MD_THREADS) tile[k] = (k0 + k < d) ? a[k0 + k] : 0.0f;
        __syncthreads();
        const int kn = min(MD_TILE, d - k0);
        for (int k = 0; k < kn; ++k) {
            const float ak = tile[k];
            rank += (ak > ai || (ak == ai && k0 + k < i)) ? 1 : 0;
        }
    }
    if (i < d) order[rank] = i;
}

// one warp; n = d / b <= MD_MAX_BLOCKS.  Running sums are non-negative doubles, so their bit patterns order
// like the values: the minimum over the warp is three integer warp reductions (high word, low word among
// the lanes that hold the minimal high word, block index among the lanes that hold the minimal sum).  A full
// block's sum is replaced by +infinity.
__global__ void __launch_bounds__(32) perq_massdiff_greedy_kernel(const float *a, const int32_t *order, int d, int b,
                                                                  int32_t *perm)
{
    __shared__ unsigned long long sum[MD_MAX_BLOCKS];      // bit patterns of the doubles
    __shared__ int fill[MD_MAX_BLOCKS];
    const int lane = threadIdx.x, n = d / b;
    for (int j = lane; j < n; j += 32) { sum[j] = 0ull; fill[j] = 0; }
    __syncwarp();
    const unsigned long long INF = 0x7ff0000000000000ull;
    for (int s0 = 0; s0 < d; s0 += 32) {
        // the next 32 channels and their masses, one per lane
        const int cl = (s0 + lane < d) ? order[s0 + lane] : 0;
        const float al = (s0 + lane < d) ? a[cl] : 0.0f;
        const int steps = min(32, d - s0);
        for (int t = 0; t < steps; ++t) {
            const int c = __shfl_sync(0xffffffffu, cl, t);
            const float ac = __shfl_sync(0xffffffffu, al, t);
            unsigned long long best = ~0ull;
            int bj = 0x7fffffff;
#pragma unroll 4
            for (int j = lane; j < n; j += 32) {
                const unsigned long long v = sum[j];
                if (v < best) { best = v; bj = j; }          // ascending j: equal sums keep the lower block
            }
            const uint32_t hi = (uint32_t)(best >> 32), lo = (uint32_t)best;
            const uint32_t mhi = __reduce_min_sync(0xffffffffu, hi);
            const uint32_t mlo = __reduce_min_sync(0xffffffffu, hi == mhi ? lo : 0xffffffffu);
            const int mj = (int)__reduce_min_sync(0xffffffffu, (hi == mhi && lo == mlo) ? (uint32_t)bj : 0x7fffffffu);
            if (lane == 0) {
                const int f = fill[mj];
                perm[(size_t)mj * b + f] = c;
                fill[mj] = f + 1;
                const double ns = __longlong_as_double((long long)(((unsigned long long)mhi << 32) | mlo)) + (double)ac;
                sum[mj] = (f + 1 < b) ? (unsigned long long)__double_as_longlong(ns) : INF;
            }
            __syncwarp();
        }
    }
}

}  // namespace perq
