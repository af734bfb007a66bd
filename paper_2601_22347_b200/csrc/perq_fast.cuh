// Fast rotate+quantize kernel for the common cases: no permutation, b in {16,32,64,128},
// d a multiple of 1024, scales per token (d/1024 in {1,2,4,8}), per 128 (INT4) or per 32 (MXFP4).
//
// Data path (HBM-bound, one pass):
//   global --cp.async.bulk + mbarrier--> shared memory ring (bf16 rows, as stored)
//   --ldmatrix--> tensor-core H_16 (mma.sync bf16 x (+-1) -> fp32; products are exact)
//   --packed fp32 add/sub on registers--> remaining log2(b)-4 butterfly stages
//   --absmax / scale / round / pack in registers--> shared staging --cp.async.bulk--> global
//
// Work is split into segments of 1024 consecutive elements, one warp each.  Within a warp,
// lane = (g, q) with g = lane / 4 the "lane group" and q = lane % 4.  Lane group g owns the
// 8 chunks (16 elements each) g*8 .. g*8+7 of the segment; the lane holds outputs
// 4q .. 4q+3 of each chunk, in "slots" s = 0..7.
//
// Slot relabelling.  To make the ldmatrix reads bank-conflict free, slot s of lane group g
// is loaded from chunk s ^ f(g), f(g) = g & 3, and the two 8-element halves of every chunk
// are swapped when g & 4.  For a Sylvester Hadamard transform an XOR shift of the input
// index only flips signs of outputs:  H(x[. ^ f])[i] = (-1)^{popcount(i & f)} H(x)[i].
// So after the butterfly over the slot bits inside a block (mask PM), slot s holds
// (-1)^{popcount(s & f & PM)} * out[chunk s ^ (f & ~PM)], and the half swap negates the
// outputs 8..15 of a chunk.  Signs are folded into the quantisation multiplier, positions
// into the store addresses; no data is moved to undo the relabelling.
//
// Exactness: see perq_generic.cuh.  The same rules apply here: range maxima of INT4 scales
// are re-derived exactly in fp64 from the bf16 inputs in shared memory, MX exponents when
// the fp32 maximum is close to a power-of-two boundary, and single elements when their
// scaled value is close to a rounding tie.
//
// Per-token scales: the G = d/1024 warps of a row exchange their fp32 maxima through one
// named barrier.  Only the warps whose maximum is within the error bound of the row's
// (normally one) derive exact values; with one such warp it stores the scale itself, with
// several the last one to add its value to a shared accumulator does.  Warps that need the
// exact maximum for a tie fix-up (rare) wait for it on a flag, with a bounded spin.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "perq_generic.cuh"

namespace perq {

constexpr int FAST_WARPS = 16;
constexpr int FAST_THREADS = FAST_WARPS * 32;
constexpr int FAST_NSTAGE = 4;
constexpr int SEG_ELEMS = 1024;
constexpr int SEG_BYTES = 2048;
constexpr int SEG_CODE_BYTES = 512;
constexpr float FAST_ERR_K = 4.0f;
constexpr uint32_t WAIT_SPIN_LIMIT = 1u << 22;

enum FastMode { MODE_TOKEN = 0, MODE_G128 = 1, MODE_MX = 2 };

struct FastParams {
    const uint16_t *x;
    uint8_t *out_codes;
    void *out_scales;
    uint32_t units_total;    // units of G = 2^LOG2G segments (fewer than 2^31)
    double sqrt_b;
    double inv_7_sqrt_b;     // 1 / (7 sqrt(b)): INT4 scale = exact |u|max times this
};

// Set (never cleared by kernels) when a bounded wait inside a kernel ran out.
__device__ unsigned int g_perq_device_error = 0u;

// Shared-memory carve-up, relative to a 1024-byte aligned base.
struct FastSmem {
    static constexpr size_t stages = 0;
    static constexpr size_t codes = stages + (size_t)FAST_WARPS * FAST_NSTAGE * SEG_BYTES;
    static constexpr size_t full = codes + (size_t)FAST_WARPS * 2 * SEG_CODE_BYTES;
    static constexpr size_t wacc = full + (size_t)FAST_WARPS * FAST_NSTAGE * 8;     // [2][FAST_WARPS] u64 accumulators
    static constexpr size_t wpub = wacc + (size_t)FAST_WARPS * 2 * 8;               // [2][FAST_WARPS] u64 published row maxima
    static constexpr size_t wmax = wpub + (size_t)FAST_WARPS * 2 * 8;               // [2][FAST_WARPS] f32 warp maxima
    static constexpr size_t wcnt = wmax + (size_t)FAST_WARPS * 2 * 4;               // [2][FAST_WARPS] u32 arrival counts
    static constexpr size_t wflag = wcnt + (size_t)FAST_WARPS * 2 * 4;              // [2][FAST_WARPS] u32 publication flags
    static constexpr size_t used = wflag + (size_t)FAST_WARPS * 2 * 4;
    static constexpr size_t total = used + 1024;                                    // room to align the base
};

// ---------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait: false if the phase did not complete within WAIT_SPIN_LIMIT polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < WAIT_SPIN_LIMIT; ++spin) {
        uint32_t done;
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// c = a * b with a zero accumulator input (no registers are cleared for it)
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
        : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}
__device__ __forceinline__ void named_barrier(int id, int threads)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void sts_u16(uint32_t addr, uint32_t v)
{
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"((uint16_t)v) : "memory");
}
__device__ __forceinline__ uint32_t ld_volatile_shared_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.volatile.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}

// Two fp32 values per operand: the packed add / fma of sm_100 (half the issue slots of scalar code).
typedef float2 f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) { return make_float2(lo, hi); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) { return __ffma2_rn(b, make_float2(-1.0f, -1.0f), a); }
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) { return __fmul2_rn(a, b); }
// max over the warp of a non-negative fp32 value (one instruction on sm_100a)
__device__ __forceinline__ float warp_max_f32(float v)
{
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
// max over the warp of a non-negative double, on its bit pattern
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v)
{
    const uint32_t hi = __reduce_max_sync(0xffffffffu, (uint32_t)(v >> 32));
    const uint32_t lo = __reduce_max_sync(0xffffffffu, ((uint32_t)(v >> 32) == hi) ? (uint32_t)v : 0u);
    return ((unsigned long long)hi << 32) | lo;
}
__device__ __forceinline__ float max3abs(float acc, float a, float b) { return fmaxf(fmaxf(acc, fabsf(a)), fabsf(b)); }

__device__ __forceinline__ uint32_t hadamard_bf16(int k, int n) { return (__popc(k & n) & 1) ? 0xBF80u : 0x3F80u; }
