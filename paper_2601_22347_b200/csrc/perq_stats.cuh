// Calibration statistic kernels: per-channel sum of |x|, per-block mean l1 norm and
// per-token max block l1 norm under an optional permutation.
//
// Phase 1: each CTA walks a contiguous slab of rows, 64 KB of rows at a time through a ring of
// bulk-copied shared-memory stages, keeps
// per-channel and per-block partial sums in registers (every thread owns fixed columns /
// blocks), and writes them to its own slice of the workspace.  Rows go through shared memory
// only when a block statistic needs the gather through the permutation.
// Phase 2: one thread per output adds the CTA slices in CTA order.  All additions happen
// in a fixed order, so the results are bit-identical from run to run.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "perq_fast.cuh"   // mbarrier / bulk-copy wrappers, device error word

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
    int n_stages;        // shared-memory stages of the row ring
};

__device__ __forceinline__ float abs_bf16(uint16_t h) { return __uint_as_float(((uint32_t)h & 0x7fffu) << 16); }

// KC = 16-byte chunks of a row per thread (d <= KC * 4096); R = rows per batch (64 KB).  Batches of
// consecutive rows are contiguous in global memory: one elected thread fetches each with a single
// cp.async.bulk into a ring of shared-memory stages (bulk copies are not limited by the load
// queue of the SM the way per-thread loads are), everybody reads its columns from there.
// CL >= 0 selects a specialised variant: rows of exactly KC * 4096 channels, no permutation, blocks of
// 2^CL chunks (CL <= 5: summed by shuffles), block statistics wanted (WB) or not -- the flags the general
// variant (CL = -1) tests at run time inside its unrolled loops are constants there.
template <int KC, int CL, bool WB>
__global__ void __launch_bounds__(ST_THREADS) perq_stats_partial_kernel(StatsParams p)
{
    constexpr int R = 8 / KC;
    constexpr bool FAST = CL >= 0;
    static_assert(CL <= 5, "shuffle sums need a block inside a warp");
    const int NST = p.n_stages;                   // 3, or 2 where 3 stages would not fit
    extern __shared__ __align__(128) unsigned char smem[];
    const int d = p.d, L = p.log2b, nb = d >> L, nchunks = d >> 3;
    const size_t stage_bytes = (size_t)R * d * 2;
    uint16_t *stages = (uint16_t *)smem;                                 // [NST][R][d] rows, original order
    uint16_t *sperm = (uint16_t *)(smem + NST * stage_bytes);            // [d] permutation (d <= 32768 fits 16 bits)
    float *cs = (float *)(smem + NST * stage_bytes + (size_t)d * 2);     // [R][d/8] per-chunk l1 of the permuted rows
    float *red = cs + (size_t)R * nchunks;                               // [2][R][16]
    uint64_t *full = (uint64_t *)(red + 2 * R * 16);                     // [NST] mbarriers
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int i = tid; i < d; i += ST_THREADS) {
        int q = p.perm ? __ldg(p.perm + i) : i;
        sperm[i] = (uint16_t)min(max(q, 0), d - 1);
    }
    float2 csum[KC][4];      // per-channel sums of |x|, as pairs for the packed fp32 add
    float bsum[KC];
#pragma unroll
    for (int k = 0; k < KC; ++k) {
        bsum[k] = 0.0f;
#pragma unroll
        for (int e = 0; e < 4; ++e) csum[k][e] = make_float2(0.0f, 0.0f);
    }
    const long long t0 = (long long)blockIdx.x * p.rows_per_cta;
    const long long t1 = min(p.T, t0 + p.rows_per_cta);
    const bool want_blocks = FAST ? WB : ((p.ws_block != nullptr) || (p.token_max != nullptr));
    const bool use_perm = FAST ? false : (p.perm != nullptr);
    const int cpb = FAST ? (1 << (CL < 0 ? 0 : CL)) : (1 << (L - 3));   // 16-byte chunks per block
    const bool shuffle_blocks = FAST ? true : cpb <= 32;                // a block's chunks sit in adjacent lanes of one warp

    auto fetch = [&](int stage, long long t) {      // one thread: rows t .. t+R-1 (those below t1) into a stage
        if (t < t1) {
            const uint32_t bytes = (uint32_t)(min((long long)R, t1 - t) * d * 2);
            mbar_expect_tx(smem_u32(&full[stage]), bytes);
            bulk_load(smem_u32(stages + (size_t)stage * R * d), p.x + (size_t)t * d, bytes, smem_u32(&full[stage]));
        }
    };
    if (tid == 0) {
        for (int s = 0; s < NST; ++s) mbar_init(smem_u32(&full[s]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        for (int s = 0; s < NST; ++s) fetch(s, t0 + (long long)s * R);
    }
    __syncthreads();

    uint32_t it = 0;
    for (long long t = t0; t < t1; t += R, ++it) {
        const int stage = (int)(it % NST);
        if (!mbar_wait(smem_u32(&full[stage]), (it / NST) & 1u)) {
            if (tid == 0) atomicOr(&g_perq_device_error, 8u);
            return;
        }
        const uint16_t *rows = stages + (size_t)stage * R * d;
        // ---- channel sums; chunk l1 norms (directly, or through the permutation gather); blocks of up
        // to 256 channels are summed with shuffles over the adjacent lanes that hold their chunks
        float mx[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            mx[r] = 0.0f;
            const bool live = t + r < t1;
#pragma unroll
            for (int k = 0; k < KC; ++k) {
                const int c = tid + k * ST_THREADS;
                float s = 0.0f;
                if (live && (FAST || c < nchunks)) {
                    const uint4 w = ((const uint4 *)(rows + (size_t)r * d))[c];
                    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
                    float2 m[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const uint32_t a = ww[e] & 0x7fff7fffu;                 // |.| of both halves
                        m[e] = make_float2(__uint_as_float(a << 16), __uint_as_float(a & 0xffff0000u));
                        csum[k][e] = __fadd2_rn(csum[k][e], m[e]);
                    }
                    if (want_blocks) {
                        if (use_perm) {
                            const uint4 pi = ((const uint4 *)sperm)[c];
                            const uint32_t pp[4] = {pi.x, pi.y, pi.z, pi.w};
                            const uint16_t *row = rows + (size_t)r * d;
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                s += abs_bf16(row[pp[e] & 0xffffu]);
                                s += abs_bf16(row[pp[e] >> 16]);
                            }
                        } else {
                            const float2 h = __fadd2_rn(__fadd2_rn(m[0], m[1]), __fadd2_rn(m[2], m[3]));
                            s = h.x + h.y;
                        }
                    }
                }
                if (want_blocks) {
                    if (shuffle_blocks) {
#pragma unroll
                        for (int o = 1; o < cpb; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                        if ((c & (cpb - 1)) == 0) bsum[k] += s;       // the block's first chunk keeps its sum
                        mx[r] = fmaxf(mx[r], s);
                    } else if (live && c < nchunks) {
                        cs[(size_t)r * nchunks + c] = s;
                    }
                }
            }
        }
        float *redp = red + (it & 1u) * (R * 16);        // double-buffered: one barrier per batch suffices
        if (shuffle_blocks && p.token_max) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], o));
                if (lane == 0) redp[r * 16 + warp] = mx[r];
            }
        }
        __syncthreads();                                 // every thread is done with the stage; cs / red are complete
        if (tid == 0) fetch(stage, t + (long long)NST * R);
        if (!want_blocks) continue;
        if (shuffle_blocks) {
            if (p.token_max && tid < R && t + tid < t1) {
                float m = redp[tid * 16];
                for (int wv = 1; wv < ST_THREADS / 32; ++wv) m = fmaxf(m, redp[tid * 16 + wv]);
                p.token_max[t + tid] = m;
            }
            continue;
        }
        // ---- long blocks (more than 256 channels): per-chunk sums through shared memory
#pragma unroll
        for (int r = 0; r < R; ++r) {
            mx[r] = 0.0f;
            const bool live = t + r < t1;
#pragma unroll
            for (int k = 0; k < KC; ++k) {
                const int j = tid + k * ST_THREADS;
                if (j < nb && live) {
                    float sb = 0.0f;
                    for (int c = 0; c < cpb; ++c) sb += cs[(size_t)r * nchunks + j * cpb + c];
                    bsum[k] += sb;
                    mx[r] = fmaxf(mx[r], sb);
                }
            }
        }
        if (p.token_max) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], o));
                if (lane == 0) redp[r * 16 + warp] = mx[r];
            }
            __syncthreads();
            if (tid < R && t + tid < t1) {
                float m = redp[tid * 16];
                for (int wv = 1; wv < ST_THREADS / 32; ++wv) m = fmaxf(m, redp[tid * 16 + wv]);
                p.token_max[t + tid] = m;
            }
        }
        __syncthreads();                                 // cs may be overwritten by the next batch
    }

    if (p.ws_chan) {
        float4 *dst = (float4 *)(p.ws_chan + (size_t)blockIdx.x * d);
#pragma unroll
        for (int k = 0; k < KC; ++k) {
            const int c = tid + k * ST_THREADS;
            if (c < nchunks) {
                dst[2 * c] = make_float4(csum[k][0].x, csum[k][0].y, csum[k][1].x, csum[k][1].y);
                dst[2 * c + 1] = make_float4(csum[k][2].x, csum[k][2].y, csum[k][3].x, csum[k][3].y);
            }
        }
    }
    if (p.ws_block) {
#pragma unroll
        for (int k = 0; k < KC; ++k) {
            const int c = tid + k * ST_THREADS;
            if (shuffle_blocks) {      // the thread of a block's first chunk holds its sum
                if (c < nchunks && (c & (cpb - 1)) == 0) p.ws_block[(size_t)blockIdx.x * nb + (c >> (L - 3))] = bsum[k];
            } else if (c < nb) {
                p.ws_block[(size_t)blockIdx.x * nb + c] = bsum[k];
            }
        }
    }
}

// 256 threads: 64 outputs, each summed by 4 threads over a quarter of the CTA slices, then
// combined in a fixed order (deterministic).
__global__ void __launch_bounds__(256) perq_stats_reduce_kernel(const float *ws_chan, const float *ws_block, int n_cta, int d,
                                                                int nb, float inv_T, float *chan_abs_sum, float *block_l1_mean)
{
    __shared__ float part[2][4][64];
    const int o = threadIdx.x & 63, quarter = threadIdx.x >> 6;
    const int i = blockIdx.x * 64 + o;
    const int per = (n_cta + 3) / 4;
    const int c0 = quarter * per, c1 = min(n_cta, c0 + per);
    float sc = 0.0f, sb = 0.0f;
    // eight independent loads at a time, added in slice order (x + 0 is exact, so padding is harmless)
    if (chan_abs_sum && i < d) {
        for (int c = c0; c < c1; c += 8) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (c + j < c1) ? ws_chan[(size_t)(c + j) * d + i] : 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) sc += v[j];
        }
    }
    if (block_l1_mean && i < nb) {
        for (int c = c0; c < c1; c += 8) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = (c + j < c1) ? ws_block[(size_t)(c + j) * nb + i] : 0.0f;
#pragma unroll
            for (int j = 0; j < 8; ++j) sb += v[j];
        }
    }
    part[0][quarter][o] = sc;
    part[1][quarter][o] = sb;
    __syncthreads();
    if (quarter == 0) {
        if (chan_abs_sum && i < d) chan_abs_sum[i] = ((part[0][0][o] + part[0][1][o]) + part[0][2][o]) + part[0][3][o];
        if (block_l1_mean && i < nb)
            block_l1_mean[i] = (((part[1][0][o] + part[1][1][o]) + part[1][2][o]) + part[1][3][o]) * inv_T;
    }
}

// perm[0..d) is a permutation?  status: bit0 = out of range, bit1 = duplicate.
// Per-channel maximum magnitude over the rows: chan_abs_max[c] = max_t |x[t, c]| (the statistic of the absmax and
// zigzag comparison permutations).  A CTA takes a slab of rows and 2048 channels; a thread keeps the maxima of
// eight adjacent channels as bf16 magnitude patterns (which order like the values), two per word, and merges
// them into the output with atomicMax on the fp32 bit patterns (non-negative floats order like unsigned
// integers; a maximum does not depend on the order of its operands: deterministic).  out must be zero on entry.
__global__ void __launch_bounds__(256) perq_chan_abs_max_kernel(const uint16_t *x, long long T, int d, int rows_per_cta, float *out)
{
    const int c0 = (blockIdx.x * 256 + threadIdx.x) * 8;
    if (c0 >= d) return;
    const long long t0 = (long long)blockIdx.y * rows_per_cta;
    const long long t1 = min(T, t0 + rows_per_cta);
    uint32_t m[4] = {0u, 0u, 0u, 0u};
    const uint4 *src = reinterpret_cast<const uint4 *>(x + t0 * d + c0);
    const size_t step = (size_t)d / 8;
#pragma unroll 4
    for (long long t = t0; t < t1; ++t, src += step) {
        const uint4 w = __ldg(src);
        m[0] = __vmaxu2(m[0], w.x & 0x7fff7fffu);
        m[1] = __vmaxu2(m[1], w.y & 0x7fff7fffu);
        m[2] = __vmaxu2(m[2], w.z & 0x7fff7fffu);
        m[3] = __vmaxu2(m[3], w.w & 0x7fff7fffu);
    }
    uint32_t *o = reinterpret_cast<uint32_t *>(out) + c0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        atomicMax(o + 2 * k, m[k] << 16);
        atomicMax(o + 2 * k + 1, m[k] & 0xffff0000u);
    }
}

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
