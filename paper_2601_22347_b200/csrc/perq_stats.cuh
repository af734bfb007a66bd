// Calibration statistic kernels: per-channel sum of |x|, per-block mean l1 norm and
// per-token max block l1 norm under an optional permutation.
//
// Phase 1: each CTA walks a contiguous slab of rows, a few rows at a time (64 KB of loads in
// flight per CTA, the next batch being fetched while the current one is reduced), keeps
// per-channel and per-block partial sums in registers (every thread owns fixed columns /
// blocks), and writes them to its own slice of the workspace.  Rows go through shared memory
// only when a block statistic needs the gather through the permutation.
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

// KC = 16-byte chunks of a row per thread (d <= KC * 4096); R = rows in flight per CTA, chosen so
// that every thread always has 8 loads of 16 bytes outstanding (64 KB per CTA).
template <int KC>
__global__ void __launch_bounds__(ST_THREADS) perq_stats_partial_kernel(StatsParams p)
{
    constexpr int R = 8 / KC;
    extern __shared__ __align__(16) unsigned char smem[];
    const int d = p.d, L = p.log2b, nb = d >> L, nchunks = d >> 3;
    uint16_t *sperm = (uint16_t *)smem;                                  // [d] permutation (d <= 32768 fits 16 bits)
    uint16_t *raw = sperm + d;                                           // [R][d] rows, original order
    float *cs = (float *)(smem + (size_t)(R + 1) * d * 2);               // [R][d/8] per-chunk l1 of the permuted rows
    float *red = cs + (size_t)R * nchunks;                               // [R][16]
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    for (int i = tid; i < d; i += ST_THREADS) {
        int q = p.perm ? __ldg(p.perm + i) : i;
        sperm[i] = (uint16_t)min(max(q, 0), d - 1);
    }
    float csum[KC][8];
    float bsum[KC];
#pragma unroll
    for (int k = 0; k < KC; ++k) {
        bsum[k] = 0.0f;
#pragma unroll
        for (int e = 0; e < 8; ++e) csum[k][e] = 0.0f;
    }
    const long long t0 = (long long)blockIdx.x * p.rows_per_cta;
    const long long t1 = min(p.T, t0 + p.rows_per_cta);
    const bool want_blocks = (p.ws_block != nullptr) || (p.token_max != nullptr);
    const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);

    // two batches of rows in flight in registers: while one is reduced the other is still arriving
    constexpr int NBUF = KC >= 8 ? 1 : 2;      // (the widest rows leave registers for one batch only)
    uint4 wbuf[NBUF][R][KC];
    auto load_batch = [&](uint4 (&w)[R][KC], long long t) {
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const uint4 *src = (const uint4 *)(p.x + (size_t)(t + r) * d);
#pragma unroll
            for (int k = 0; k < KC; ++k) {
                const int c = tid + k * ST_THREADS;
                w[r][k] = (t + r < t1 && c < nchunks) ? __ldcs(src + c) : zero4;
            }
        }
    };
    load_batch(wbuf[0], t0);
    if (NBUF == 2) load_batch(wbuf[NBUF - 1], t0 + R);
    __syncthreads();

    auto process = [&](uint4 (&w)[R][KC], long long t) {
        // ---- channel sums from the registers; rows to shared memory for the gather
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
            for (int k = 0; k < KC; ++k) {
                const uint32_t ww[4] = {w[r][k].x, w[r][k].y, w[r][k].z, w[r][k].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    csum[k][2 * e] += __uint_as_float((ww[e] << 16) & 0x7fffffffu);
                    csum[k][2 * e + 1] += __uint_as_float(ww[e] & 0x7fff0000u);
                }
                const int c = tid + k * ST_THREADS;
                if (want_blocks && c < nchunks) {
                    if (p.perm) {
                        ((uint4 *)(raw + (size_t)r * d))[c] = w[r][k];
                    } else {      // identity: the chunk's l1 norm is this thread's own eight values
                        float s = 0.0f;
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            s += __uint_as_float((ww[e] << 16) & 0x7fffffffu);
                            s += __uint_as_float(ww[e] & 0x7fff0000u);
                        }
                        cs[(size_t)r * nchunks + c] = s;
                    }
                }
            }
        }
        // ---- refill these registers with the batch after next
        load_batch(w, t + NBUF * R);
        if (!want_blocks) return;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < R; ++r) {
            if (!p.perm) break;
            const uint16_t *row = raw + (size_t)r * d;
#pragma unroll
            for (int k = 0; k < KC; ++k) {
                const int c = tid + k * ST_THREADS;
                if (c < nchunks) {
                    const uint4 pi = ((const uint4 *)sperm)[c];
                    const uint32_t pp[4] = {pi.x, pi.y, pi.z, pi.w};
                    float s = 0.0f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        s += abs_bf16(row[pp[e] & 0xffffu]);
                        s += abs_bf16(row[pp[e] >> 16]);
                    }
                    cs[(size_t)r * nchunks + c] = s;
                }
            }
        }
        if (p.perm) __syncthreads();
        const int cpb = 1 << (L - 3);          // chunks per block
        float mx[R];
#pragma unroll
        for (int r = 0; r < R; ++r) {
            mx[r] = 0.0f;
            const bool live = t + r < t1;
#pragma unroll
            for (int k = 0; k < KC; ++k) {
                const int j = tid + k * ST_THREADS;
                if (j < nb && live) {
                    float s = 0.0f;
                    for (int c = 0; c < cpb; ++c) s += cs[(size_t)r * nchunks + j * cpb + c];
                    bsum[k] += s;
                    mx[r] = fmaxf(mx[r], s);
                }
            }
        }
        if (p.token_max) {
#pragma unroll
            for (int r = 0; r < R; ++r) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], o));
                if (lane == 0) red[r * 16 + warp] = mx[r];
            }
            __syncthreads();
            if (tid < R && t + tid < t1) {
                float m = red[tid * 16];
                for (int wv = 1; wv < ST_THREADS / 32; ++wv) m = fmaxf(m, red[tid * 16 + wv]);
                p.token_max[t + tid] = m;
            }
        }
        __syncthreads();
    };
    for (long long t = t0; t < t1; t += NBUF * R) {
        process(wbuf[0], t);
        if (NBUF == 2 && t + R < t1) process(wbuf[NBUF - 1], t + R);
    }

    if (p.ws_chan) {
        float4 *dst = (float4 *)(p.ws_chan + (size_t)blockIdx.x * d);
#pragma unroll
        for (int k = 0; k < KC; ++k) {
            const int c = tid + k * ST_THREADS;
            if (c < nchunks) {
                dst[2 * c] = make_float4(csum[k][0], csum[k][1], csum[k][2], csum[k][3]);
                dst[2 * c + 1] = make_float4(csum[k][4], csum[k][5], csum[k][6], csum[k][7]);
            }
        }
    }
    if (p.ws_block) {
#pragma unroll
        for (int k = 0; k < KC; ++k) {
            const int j = tid + k * ST_THREADS;
            if (j < nb) p.ws_block[(size_t)blockIdx.x * nb + j] = bsum[k];
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
