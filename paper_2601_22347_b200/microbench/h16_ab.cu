// A/B timing: the H_16 stage of a b = 32 rotation on the tensor cores (ldmatrix + mma.sync, then one packed
// add/sub stage) against five add/sub stages on registers, both from bf16 in shared memory and both followed by
// the pair maxima; 148 CTAs of 16 warps, CUDA events.  Not part of the library.  Build and run:
//   nvcc -gencode arch=compute_100a,code=sm_100a -O3 -std=c++17 -I paper_2601_22347_b200/csrc \
//        -o h16_ab paper_2601_22347_b200/microbench/h16_ab.cu && ./h16_ab
#include <cuda_runtime.h>
#include <cstdio>
#include "perq_tok.cuh"
using namespace perq;
constexpr int ITERS = 4000;

template <int WHAT>
__global__ void __launch_bounds__(512, 1) ab_kernel(const uint16_t *x, float *out)
{
    extern __shared__ __align__(128) unsigned char sm_raw[];
    unsigned char *sm = sm_raw + ((1024u - (smem_u32(sm_raw) & 1023u)) & 1023u);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t *mine = reinterpret_cast<uint32_t *>(sm + warp * 2048);
    for (int i = lane; i < 512; i += 32) mine[i] = reinterpret_cast<const uint32_t *>(x)[(warp * 512 + i) & 4095];
    __syncwarp();
    const uint32_t seg_addr = smem_u32(sm + warp * 2048);
    TokLane<5> L;
    L.init(lane);
    float acc = 0.0f;
    for (int it = 0; it < ITERS; ++it) {
        f32x2 v[8][2];
        if (WHAT == 0) {
            tok_rotate<5>(seg_addr, L, v);
        } else {
            // lane holds the 32 consecutive elements of one block: 4 x 16 bytes, converted, five stages
            float f[32];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                uint32_t w[4];
                asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "r"(seg_addr + (uint32_t)(lane * 64 + r * 16)) : "memory");
#pragma unroll
                for (int k = 0; k < 4; ++k) { f[8 * r + 2 * k] = __uint_as_float(w[k] << 16); f[8 * r + 2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
            }
            // stage over bit 0 inside pairs (scalar), then bits 1..4 on packed pairs
#pragma unroll
            for (int e = 0; e < 32; e += 2) { const float a = f[e], c = f[e + 1]; f[e] = a + c; f[e + 1] = a - c; }
            f32x2 pv[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) pv[e] = pack2(f[2 * e], f[2 * e + 1]);
#pragma unroll
            for (int t = 0; t < 4; ++t) {
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    if ((e & (1 << t)) == 0) { const f32x2 a = pv[e], c = pv[e | (1 << t)]; pv[e] = add2(a, c); pv[e | (1 << t)] = sub2(a, c); }
                }
            }
#pragma unroll
            for (int s = 0; s < 8; ++s) { v[s][0] = pv[2 * s]; v[s][1] = pv[2 * s + 1]; }
        }
        float gm[4];
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            float a = max3abs(fabsf(v[2 * m][0].x), v[2 * m][0].y, v[2 * m][1].x);
            a = max3abs(a, v[2 * m][1].y, v[2 * m + 1][0].x);
            a = max3abs(a, v[2 * m + 1][0].y, v[2 * m + 1][1].x);
            gm[m] = fmaxf(a, fabsf(v[2 * m + 1][1].y));
        }
        acc += fmaxf(fmaxf(gm[0], gm[1]), fmaxf(gm[2], gm[3]));
        __syncwarp();
    }
    out[blockIdx.x * 512 + tid] = acc;
}

int main()
{
    uint16_t *x; float *out;
    cudaMalloc(&x, 16384); cudaMemset(x, 0x3f, 16384);
    cudaMalloc(&out, 148 * 512 * 4);
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    auto run = [&](auto k, const char *name) {
        cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 32768 + 1024);
        for (int w = 0; w < 2; ++w) k<<<148, 512, 32768 + 1024>>>(x, out);
        cudaEventRecord(e0);
        for (int r = 0; r < 5; ++r) k<<<148, 512, 32768 + 1024>>>(x, out);
        cudaEventRecord(e1); cudaEventSynchronize(e1);
        float ms; cudaEventElapsedTime(&ms, e0, e1);
        printf("%-40s %.3f ns per 1024-element segment and SM (16 warps)\n", name, ms / 5 * 1e6 / ITERS / 16);
    };
    run(ab_kernel<0>, "H_16 on tensor cores + 1 packed stage");
    run(ab_kernel<1>, "5 add/sub stages on registers");
    cudaError_t e = cudaDeviceSynchronize();
    printf("%s\n", cudaGetErrorString(e));
    return e != cudaSuccess;
}
